/*
 * Seeded synthetic-input generator: counter-based random numbers only.
 *
 * Every value is a pure function of (seed, stream id, element index), so any
 * slice of any tensor can be regenerated alone and the same bits reach every
 * consumer.  This file holds no arithmetic of the decoding method itself: it
 * produces bf16 Gaussian tensors and uniform integer streams, nothing else.
 *
 * Recipe
 *   key   = mix64(seed * 0x9E3779B97F4A7C15 + stream * 0xD1B54A32D192ED03 + 1)
 *   bits  = mix64(key + (counter + 1) * 0x9E3779B97F4A7C15)
 *   Gaussian pair p (elements 2p, 2p+1): u1 = (hi32(bits)+1) / 2^32 in (0,1],
 *   u2 = lo32(bits) / 2^32; r = sqrt(-2 ln u1); z0 = r cos(2 pi u2),
 *   z1 = r sin(2 pi u2) (Box-Muller), scaled by std, rounded once to bf16
 *   with round-to-nearest-even.
 *   Uniform integer i: lo + (bits(counter=i) >> 11) mod (hi - lo).
 */
#include <math.h>
#include <stdint.h>

static inline uint64_t mix64(uint64_t z) {
  z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ULL;
  z ^= z >> 27; z *= 0x94D049BB133111EBULL;
  z ^= z >> 31;
  return z;
}

static inline uint64_t stream_key(uint64_t seed, uint64_t stream) {
  return mix64(seed * 0x9E3779B97F4A7C15ULL + stream * 0xD1B54A32D192ED03ULL + 1ULL);
}

static inline uint64_t draw(uint64_t key, uint64_t counter) {
  return mix64(key + (counter + 1ULL) * 0x9E3779B97F4A7C15ULL);
}

static inline uint16_t f32_to_bf16_rne(float f) {
  union { float f; uint32_t u; } v; v.f = f;
  uint32_t u = v.u;
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x0040u); /* NaN */
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7FFFu + lsb;
  return (uint16_t)(u >> 16);
}

/* out[i] = bf16(std * z_{first+i}) for i in [0, count). */
void synth_normal_bf16(uint64_t seed, uint64_t stream, uint64_t first, uint64_t count,
                       double std, uint16_t *out) {
  const uint64_t key = stream_key(seed, stream);
  const double two_pi = 6.283185307179586476925286766559;
  const uint64_t p0 = first >> 1, p1 = (first + count + 1) >> 1;
#pragma omp parallel for schedule(static)
  for (uint64_t p = p0; p < p1; ++p) {
    uint64_t b = draw(key, p);
    double u1 = ((double)(uint32_t)(b >> 32) + 1.0) * (1.0 / 4294967296.0);
    double u2 = (double)(uint32_t)(b & 0xFFFFFFFFu) * (1.0 / 4294967296.0);
    double r = sqrt(-2.0 * log(u1));
    double z0 = r * cos(two_pi * u2), z1 = r * sin(two_pi * u2);
    uint64_t e0 = 2 * p, e1 = 2 * p + 1;
    if (e0 >= first && e0 < first + count) out[e0 - first] = f32_to_bf16_rne((float)(std * z0));
    if (e1 >= first && e1 < first + count) out[e1 - first] = f32_to_bf16_rne((float)(std * z1));
  }
}

/* out[i] = lo + draw(first+i) mod (hi-lo), hi exclusive. */
void synth_uniform_i32(uint64_t seed, uint64_t stream, uint64_t first, uint64_t count,
                       int32_t lo, int32_t hi, int32_t *out) {
  const uint64_t key = stream_key(seed, stream);
  const uint64_t span = (uint64_t)((int64_t)hi - (int64_t)lo);
  for (uint64_t i = 0; i < count; ++i)
    out[i] = (int32_t)((int64_t)lo + (int64_t)((draw(key, first + i) >> 11) % span));
}
