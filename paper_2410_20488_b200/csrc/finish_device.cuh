// Device bodies of the finishers of the stream-K GEMMs: each sums the partial tiles a GEMM left in scratch
// (fixed order: ascending CTA index) and applies the elementwise step that follows the contraction:
//   qkv     rotary embedding at the row's tree position (Section 3.4: a tree token keeps its
//           positional index), queries as (hi, lo) bf16 planes, keys / values into the bf16 cache
//   swiglu  silu(gate) * up as (hi, lo) bf16 planes
//   logits  fp32 logits of the lm-head (Section 3.2: the original lm-head on every row)
//   pseudo  Eq. 3: bias and the store of the new residual rows
// An item (flat index t) owns 4 neighbouring lanes (weight rows) of one token row of one supertile, so partial
// tiles are read as float4 and results leave as 8- or 16-byte stores.  Callers hand every warp 32 consecutive
// items (one token row of one supertile).
#pragma once
#include "firp_kernels.cuh"

namespace firp {

struct Item { int st, m, i4; };

// flat item t -> (supertile, token row, lane quad); quads vary fastest (coalesced float4 reads), so the 32 lanes
// of a warp share one (supertile, token row) as long as t is the warp's base + lane
__device__ __forceinline__ bool item_of(unsigned t, int n_st, int R, Item &it) {
  if (t >= (unsigned)(n_st * R * 32)) return false;
  it.i4 = (int)(t & 31u) * 4;
  const unsigned r = t >> 5;
  it.m = (int)(r % (unsigned)R);
  it.st = (int)(r / (unsigned)R);
  return true;
}

// sums of tile 0 and tile 1 of supertile st for token row m, lanes i4 .. i4+3
__device__ __forceinline__ void sum_partials(const Partials &p, int st, int m, int i4, float4 &v0, float4 &v1) {
  const size_t plane = (size_t)p.ws_rows * 128, slot = 2 * plane;
  const SkContrib k = sk_contributors(p.sk, st);
  const float *base = p.ws + (size_t)m * 128 + i4;
  v0 = v1 = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int c0 = k.c_first; c0 <= k.c_last; c0 += 4) {      // 4 contributors' loads in flight together
    float4 a[4], b[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {         // unconditional loads (index clamped) so that they issue back to back
      const int c = min(c0 + j, k.c_last);
      const float *src = base + (size_t)(c * kGemmSlots + (c == k.c_first ? k.ord_first : 0)) * slot;
      a[j] = __ldcg(reinterpret_cast<const float4 *>(src));
      b[j] = __ldcg(reinterpret_cast<const float4 *>(src + plane));
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (c0 + j <= k.c_last) {
        v0.x += a[j].x; v0.y += a[j].y; v0.z += a[j].z; v0.w += a[j].w;
        v1.x += b[j].x; v1.y += b[j].y; v1.z += b[j].z; v1.w += b[j].w;
      }
    }
  }
}

// 1 / sqrt(mean(h^2) + eps) of token row m from the per-warp sums of squares the RMSNorm kernel left;
// all 32 lanes of a warp work on the same row, and the butterfly adds in a fixed order
__device__ __forceinline__ float row_rms_scale(const GemmArgs &a, int m) {
  if (a.ss == nullptr) return 1.f;
  const int lane = threadIdx.x & 31, nw = a.K >> 7;
  const float *p = a.ss + (size_t)m * kNormMaxWarps;
  float v = (lane < nw ? __ldcg(p + lane) : 0.f) + (lane + 32 < nw ? __ldcg(p + lane + 32) : 0.f);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return rsqrtf(v / (float)a.K + a.eps);
}

__device__ __forceinline__ void split4(const float v[4], uint2 &hi, uint2 &lo) {
  const __nv_bfloat162 h01 = __floats2bfloat162_rn(v[0], v[1]), h23 = __floats2bfloat162_rn(v[2], v[3]);
  const float2 f01 = __bfloat1622float2(h01), f23 = __bfloat1622float2(h23);
  const __nv_bfloat162 l01 = __floats2bfloat162_rn(v[0] - f01.x, v[1] - f01.y);
  const __nv_bfloat162 l23 = __floats2bfloat162_rn(v[2] - f23.x, v[3] - f23.y);
  hi = make_uint2(*reinterpret_cast<const uint32_t *>(&h01), *reinterpret_cast<const uint32_t *>(&h23));
  lo = make_uint2(*reinterpret_cast<const uint32_t *>(&l01), *reinterpret_cast<const uint32_t *>(&l23));
}
__device__ __forceinline__ uint2 round4(const float v[4]) {
  const __nv_bfloat162 h01 = __floats2bfloat162_rn(v[0], v[1]), h23 = __floats2bfloat162_rn(v[2], v[3]);
  return make_uint2(*reinterpret_cast<const uint32_t *>(&h01), *reinterpret_cast<const uint32_t *>(&h23));
}

// ---- q, k, v: rotary embedding, query planes, cache rows --------------------------------------
// Supertile st holds the first halves (c < dh/2) of 128 / (dh/2) heads in tile 0 and their second
// halves in tile 1, so lanes i4..i4+3 of the two tiles are 4 rotary pairs (c, c + dh/2) of one head.
__device__ __forceinline__ void qkv_finish_item(const Partials &p, const GemmArgs &a, int n_st, unsigned t) {
  Item it;
  if (!item_of(t, n_st, a.R, it)) return;
  const int half = a.dh >> 1, hp = 128 / half;
  const int unit = it.st * hp + it.i4 / half, c = it.i4 % half;
  const int s = it.m / a.rw.Ms, v = it.m - s * a.rw.Ms;
  const float rs = row_rms_scale(a, it.m);          // before any lane drops out: the warp adds together
  if (unit >= a.H + 2 * a.Hkv || v >= a.rows_active) return;
  float4 v0, v1;
  sum_partials(p, it.st, it.m, it.i4, v0, v1);
  float x1[4] = {v0.x * rs, v0.y * rs, v0.z * rs, v0.w * rs}, x2[4] = {v1.x * rs, v1.y * rs, v1.z * rs, v1.w * rs};
  if (unit < a.H + a.Hkv) {     // queries and keys are rotated at the row's tree position
    const float4 *cs = reinterpret_cast<const float4 *>(a.rope + (size_t)it.m * half + c);
    const float4 cs01 = __ldcg(cs), cs23 = __ldcg(cs + 1);
    const float co[4] = {cs01.x, cs01.z, cs23.x, cs23.z}, si[4] = {cs01.y, cs01.w, cs23.y, cs23.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float y1 = x1[j] * co[j] - x2[j] * si[j], y2 = x2[j] * co[j] + x1[j] * si[j];
      x1[j] = y1; x2[j] = y2;
    }
  }
  if (unit < a.H) {
    uint2 h1, l1, h2, l2;
    split4(x1, h1, l1); split4(x2, h2, l2);
    bf16 *dst = a.q + (size_t)it.m * a.H * a.dh + unit * a.dh + c;
    *reinterpret_cast<uint2 *>(dst) = h1;
    *reinterpret_cast<uint2 *>(dst + half) = h2;
    *reinterpret_cast<uint2 *>(dst + a.q_lo_off) = l1;
    *reinterpret_cast<uint2 *>(dst + a.q_lo_off + half) = l2;
  } else {                      // the cache stores bf16: one rounding, on store
    const int is_v = unit >= a.H + a.Hkv;
    const int kvh = unit - a.H - (is_v ? a.Hkv : 0);
    const int slot = a.seq_ids[s];
    const int pos = a.pos[s * a.rw.Ms] + v;        // committed length (position of the root row) + row index
    if (pos < a.max_ctx) {
      bf16 *dst = a.kcache + (is_v ? a.kv_stride : 0) + (kv_row(a.pages, slot, pos, a.max_ctx) * a.Hkv + kvh) * a.dh + c;
      *reinterpret_cast<uint2 *>(dst) = round4(x1);
      *reinterpret_cast<uint2 *>(dst + half) = round4(x2);
    }
  }
}

// ---- SwiGLU: tile 0 = gate rows st*128 .., tile 1 = the matching up rows ------------------------
__device__ __forceinline__ void swiglu_finish_item(const Partials &p, const GemmArgs &a, int n_st, unsigned t) {
  Item it;
  if (!item_of(t, n_st, a.R, it)) return;
  const int j0 = it.st * 128 + it.i4;
  const int v = it.m % a.rw.Ms;
  const float rs = row_rms_scale(a, it.m);
  if (j0 >= a.F || v >= a.rows_active) return;
  float4 g, u;
  sum_partials(p, it.st, it.m, it.i4, g, u);
  const float gg[4] = {g.x * rs, g.y * rs, g.z * rs, g.w * rs}, uu[4] = {u.x * rs, u.y * rs, u.z * rs, u.w * rs};
  float y[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) y[j] = gg[j] / (1.f + __expf(-gg[j])) * uu[j];
  uint2 hi, lo;
  split4(y, hi, lo);
  bf16 *dst = a.y + (size_t)it.m * a.F + j0;
  *reinterpret_cast<uint2 *>(dst) = hi;
  *reinterpret_cast<uint2 *>(dst + a.y_lo_off) = lo;
}

// ---- logits: tile 0 = rows st*256 .., tile 1 = rows st*256 + 128 .. -----------------------------
__device__ __forceinline__ void logits_finish_item(const Partials &p, const GemmArgs &a, int n_st, unsigned t) {
  Item it;
  if (!item_of(t, n_st, a.R, it)) return;
  const int n0 = it.st * 256 + it.i4, n1 = n0 + 128;
  const float rs = row_rms_scale(a, it.m);
  if (n0 >= a.N) return;
  float4 v0, v1;
  sum_partials(p, it.st, it.m, it.i4, v0, v1);
  v0.x *= rs; v0.y *= rs; v0.z *= rs; v0.w *= rs;
  v1.x *= rs; v1.y *= rs; v1.z *= rs; v1.w *= rs;
  float *row = a.logits + (size_t)it.m * a.N;
  if ((a.N & 3) == 0) {
    *reinterpret_cast<float4 *>(row + n0) = v0;
    if (n1 < a.N) *reinterpret_cast<float4 *>(row + n1) = v1;
  } else {
    const float e0[4] = {v0.x, v0.y, v0.z, v0.w}, e1[4] = {v1.x, v1.y, v1.z, v1.w};
    for (int j = 0; j < 4; ++j) {
      if (n0 + j < a.N) row[n0 + j] = e0[j];
      if (n1 + j < a.N) row[n1 + j] = e1[j];
    }
  }
}

// ---- Eq. 3: the k maps stacked into one [k d][d] matrix; token row m = sequence m ------------------------
__device__ __forceinline__ void pseudo_finish_item(const Partials &p, const GemmArgs &a, int n_st, unsigned t) {
  Item it;
  if (!item_of(t, n_st, a.R, it)) return;
  const int n0 = it.st * 256 + it.i4;
  // pre-norm variant (a.ss given): the operand was h * g; divide by the RMS of the source row of the residual stream
  int src_row;
  if (a.rw.chains) { const int s = it.m / a.rw.T; src_row = s * a.rw.Ms + (it.m - s * a.rw.T); }
  else src_row = it.m * a.rw.Ms + a.rw.anchor;
  const float rs = row_rms_scale(a, src_row);       // before any lane drops out: the warp adds together
  if (n0 >= a.N) return;
  float4 v0, v1;
  sum_partials(p, it.st, it.m, it.i4, v0, v1);
  const float e[2][4] = {{v0.x * rs, v0.y * rs, v0.z * rs, v0.w * rs}, {v1.x * rs, v1.y * rs, v1.z * rs, v1.w * rs}};
#pragma unroll
  for (int t = 0; t < 2; ++t) {
    const int n = n0 + 128 * t;                   // d is a multiple of 128: the 4 outputs belong to one map
    if (n >= a.N) continue;
    const int i = n / a.K, o = n - i * a.K;
    float4 r = make_float4(e[t][0], e[t][1], e[t][2], e[t][3]);
    if (a.pred_b) {
      r.x += __bfloat162float(a.pred_b[n]); r.y += __bfloat162float(a.pred_b[n + 1]);
      r.z += __bfloat162float(a.pred_b[n + 2]); r.w += __bfloat162float(a.pred_b[n + 3]);
    }
    size_t row;
    if (a.rw.chains) {
      const int s = it.m / a.rw.T, v = it.m - s * a.rw.T;
      row = (size_t)s * a.rw.Ms + a.rw.T + (size_t)(a.pseudo0 + i) * a.rw.T + v;
    } else {
      row = (size_t)it.m * a.rw.Ms + a.rw.T + a.pseudo0 + i;
    }
    *reinterpret_cast<float4 *>(a.h_rows + row * a.K + o) = r;
  }
}


}  // namespace firp
