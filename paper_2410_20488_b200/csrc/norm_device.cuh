// Device bodies of the residual-update + RMSNorm pass and of the operand split for Eq. 3, shared by their own
// kernels and by the fused decoder kernel.
//   rmsnorm_item:  h[r] += the partial tiles a residual GEMM left in scratch (fixed order: ascending CTA index);
//                  x[r] = h[r] * g as bf16 planes (hi, lo; plus a third plane on request) -- NOT yet divided by the
//                  row's RMS; ss[r][w] = sum of h[r][c]^2 over the 128 columns of warp w.  The division by
//                  sqrt(mean(h^2) + eps) commutes with the GEMM that consumes x, so that GEMM's finisher applies it
//                  to the fp32 sums (it adds the ss[r][*] in a fixed order).  No reduction beyond a warp, no barrier.
//   root_split_item: the fp32 residual rows Eq. 3 reads (raw, or times a gain for the pre-norm variant), as (hi, lo)
//                  bf16 planes.
#pragma once
#include "firp_kernels.cuh"

namespace firp {

// item t = (row of the range, float4 of the row); a warp's 32 items are 128 neighbouring columns of one row
__device__ __forceinline__ void rmsnorm_item(const Rows &rw, int v0, int nv, float *h, const Partials &pend, const bf16 *g,
                                             int d, bf16 *x, size_t x_lo_off, int planes, float *ss, unsigned t) {
  const int nvec = d >> 2;                                  // float4 per row, a multiple of 32
  if (t >= (unsigned)(rw.n_seq * nv * nvec)) return;        // whole warps drop out together
  const int rowi = (int)(t / (unsigned)nvec), idx = (int)(t % (unsigned)nvec);
  const int s = rowi / nv, v = v0 + rowi % nv;
  const int r = s * rw.Ms + v;
  float4 *hr = reinterpret_cast<float4 *>(h + (size_t)r * d);
  float4 a = __ldcg(hr + idx);
  if (pend.sk.U > 0) {
    const size_t plane_elems = (size_t)pend.ws_rows * 128;
    const int n = idx * 4, st = n >> 8, tl = (n >> 7) & 1, i = n & 127;
    const SkContrib k = sk_contributors(pend.sk, st);
    const float *base = pend.ws + (size_t)tl * plane_elems + (size_t)r * 128 + i;
    for (int c0 = k.c_first; c0 <= k.c_last; c0 += 12) {    // 12 contributors' loads in flight together
      float4 p[12];
#pragma unroll
      for (int j = 0; j < 12; ++j) {      // unconditional loads (index clamped) so that they issue back to back
        const int c = min(c0 + j, k.c_last);
        p[j] = __ldcg(reinterpret_cast<const float4 *>(
            base + (size_t)(c * kGemmSlots + (c == k.c_first ? k.ord_first : 0)) * 2 * plane_elems));
      }
#pragma unroll
      for (int j = 0; j < 12; ++j) {
        if (c0 + j <= k.c_last) { a.x += p[j].x; a.y += p[j].y; a.z += p[j].z; a.w += p[j].w; }
      }
    }
    hr[idx] = a;
  }
  float sq = a.x * a.x + a.y * a.y + a.z * a.z + a.w * a.w;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
  if ((threadIdx.x & 31) == 0) ss[(size_t)r * kNormMaxWarps + (idx >> 5)] = sq;
  const __nv_bfloat162 g01 = reinterpret_cast<const __nv_bfloat162 *>(g)[2 * idx];
  const __nv_bfloat162 g23 = reinterpret_cast<const __nv_bfloat162 *>(g)[2 * idx + 1];
  const float2 ga = __bfloat1622float2(g01), gb = __bfloat1622float2(g23);
  const float y0 = a.x * ga.x, y1 = a.y * ga.y, y2 = a.z * gb.x, y3 = a.w * gb.y;
  const __nv_bfloat162 o01 = __floats2bfloat162_rn(y0, y1), o23 = __floats2bfloat162_rn(y2, y3);
  const float2 f01 = __bfloat1622float2(o01), f23 = __bfloat1622float2(o23);
  const __nv_bfloat162 l01 = __floats2bfloat162_rn(y0 - f01.x, y1 - f01.y);     // lo plane: what the hi half lost
  const __nv_bfloat162 l23 = __floats2bfloat162_rn(y2 - f23.x, y3 - f23.y);
  uint2 hi2, lo2;
  hi2.x = *reinterpret_cast<const uint32_t *>(&o01); hi2.y = *reinterpret_cast<const uint32_t *>(&o23);
  lo2.x = *reinterpret_cast<const uint32_t *>(&l01); lo2.y = *reinterpret_cast<const uint32_t *>(&l23);
  *reinterpret_cast<uint2 *>(x + (size_t)r * d + 4 * idx) = hi2;
  *reinterpret_cast<uint2 *>(x + x_lo_off + (size_t)r * d + 4 * idx) = lo2;
  if (planes == 3) {   // third plane on request: what hi + mid still miss (measured: it changes no logit)
    const float2 m01 = __bfloat1622float2(l01), m23 = __bfloat1622float2(l23);
    const __nv_bfloat162 t01 = __floats2bfloat162_rn(y0 - f01.x - m01.x, y1 - f01.y - m01.y);
    const __nv_bfloat162 t23 = __floats2bfloat162_rn(y2 - f23.x - m23.x, y3 - f23.y - m23.y);
    uint2 t2;
    t2.x = *reinterpret_cast<const uint32_t *>(&t01); t2.y = *reinterpret_cast<const uint32_t *>(&t23);
    *reinterpret_cast<uint2 *>(x + 2 * x_lo_off + (size_t)r * d + 4 * idx) = t2;
  }
}


// g != NULL: the planes hold h * g (the pre-norm variant of Eq. 3; the division by the row's RMS is applied by
// the finisher of the GEMM, as for every other normalised operand)
__device__ __forceinline__ void root_split_item(const Rows &rw, const float *h, const bf16 *g, int d, bf16 *xp, size_t xp_lo_off, unsigned t) {
  const int nvec = d >> 2;
  const int per_seq = rw.chains ? rw.T : 1;                 // source rows per sequence
  if (t >= (unsigned)(rw.n_seq * per_seq * nvec)) return;
  const int m = (int)(t / (unsigned)nvec), idx = (int)(t % (unsigned)nvec);
  const int sq = m / per_seq, v = rw.chains ? m - sq * per_seq : rw.anchor;
  const int s = m;                                          // destination row in xp
  float4 a = __ldcg(reinterpret_cast<const float4 *>(h + (size_t)(sq * rw.Ms + v) * d) + idx);
  if (g != nullptr) {
    const float2 ga = __bfloat1622float2(reinterpret_cast<const __nv_bfloat162 *>(g)[2 * idx]);
    const float2 gb = __bfloat1622float2(reinterpret_cast<const __nv_bfloat162 *>(g)[2 * idx + 1]);
    a.x *= ga.x; a.y *= ga.y; a.z *= gb.x; a.w *= gb.y;
  }
  const __nv_bfloat162 o01 = __floats2bfloat162_rn(a.x, a.y), o23 = __floats2bfloat162_rn(a.z, a.w);
  const float2 f01 = __bfloat1622float2(o01), f23 = __bfloat1622float2(o23);
  const __nv_bfloat162 l01 = __floats2bfloat162_rn(a.x - f01.x, a.y - f01.y), l23 = __floats2bfloat162_rn(a.z - f23.x, a.w - f23.y);
  uint2 hi2, lo2;
  hi2.x = *reinterpret_cast<const uint32_t *>(&o01); hi2.y = *reinterpret_cast<const uint32_t *>(&o23);
  lo2.x = *reinterpret_cast<const uint32_t *>(&l01); lo2.y = *reinterpret_cast<const uint32_t *>(&l23);
  *reinterpret_cast<uint2 *>(xp + (size_t)s * d + 4 * idx) = hi2;
  *reinterpret_cast<uint2 *>(xp + xp_lo_off + (size_t)s * d + 4 * idx) = lo2;
}


}  // namespace firp
