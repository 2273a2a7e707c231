// Tile geometry and fused epilogues shared by the skinny GEMM kernels.
//
// A GEMM tile is BN weight rows x all token rows, handed over as an fp32 tile in shared memory,
// C[m * ldc + col] with col = tile-local weight row.  Activations leave every epilogue as a
// bf16 pair (hi, lo) with hi + lo = the fp32 value to ~16 mantissa bits: bf16 weights are exact,
// so feeding both halves to the tensor cores keeps GEMM inputs at near-fp32 precision.
#pragma once
#include "firp_kernels.cuh"

namespace firp {

__device__ __forceinline__ void split_bf16(float v, bf16 &hi, bf16 &lo) {
  hi = __float2bfloat16_rn(v);
  lo = __float2bfloat16_rn(v - __bfloat162float(hi));
}

// Which global weight rows a tile covers.
//   contiguous: rows tile*BN .. tile*BN+BN-1
//   paired:     two groups of BN/2 rows, pair_off apart: [g0, g0+BN/2) and [g0+pair_off, ...),
//               g0 = unit*unit_stride + sub*(BN/2); puts a rotary pair (c, c+dh/2) or a gate row
//               and its up row into one tile.
struct TileMap {
  int paired;
  int tiles_per_unit;  // paired: tiles per unit (a head, or the whole gate matrix)
  int unit_stride;     // paired: rows between units
  int pair_off;        // paired: distance between the two groups
  int group_rows;      // paired: valid rows per group within a unit (dh/2, or F)
};

template <int BN>
__device__ __forceinline__ int tile_row(const TileMap &tm, int tile, int i, int N, bool &valid) {
  if (!tm.paired) {
    const int r = tile * BN + i;
    valid = r < N;
    return r;
  }
  constexpr int G = BN / 2;
  const int unit = tile / tm.tiles_per_unit, sub = tile % tm.tiles_per_unit;
  const int grp = i / G, w = sub * G + (i % G);
  valid = w < tm.group_rows;
  return unit * tm.unit_stride + grp * tm.pair_off + w;
}

template <int EPI, int BN>
__device__ __forceinline__ void gemm_epilogue(const float *C, int ldc, int tile, int split, const GemmArgs &a,
                                              const TileMap &tm, int tid, int nthreads) {
  constexpr int G = BN / 2;
  if (EPI == EPI_RESIDUAL) {   // every k split adds its partial sums into the residual stream
    for (int idx = tid; idx < a.R * BN; idx += nthreads) {
      const int m = idx / BN, col = idx % BN, n = tile * BN + col;
      if (n < a.N && (m % a.rw.Ms) < a.rows_active) atomicAdd(a.h_out + (size_t)m * a.N + n, C[m * ldc + col]);
    }
  } else if (EPI == EPI_LOGITS) {
    for (int idx = tid; idx < a.R * BN; idx += nthreads) {
      const int m = idx / BN, col = idx % BN, n = tile * BN + col;
      if (n < a.N) a.logits[(size_t)m * a.N + n] = C[m * ldc + col];
    }
  } else if (EPI == EPI_SWIGLU) {   // paired tile: gate rows in [0, G), up rows in [G, BN)
    for (int idx = tid; idx < a.R * G; idx += nthreads) {
      const int m = idx / G, i = idx % G, j = tile * G + i;
      if (j < a.F) {
        const float g = C[m * ldc + i], u = C[m * ldc + G + i];
        bf16 hi, lo;
        split_bf16(g / (1.f + __expf(-g)) * u, hi, lo);
        a.y[(size_t)m * a.F + j] = hi;
        a.y[a.y_lo_off + (size_t)m * a.F + j] = lo;
      }
    }
  } else {  // EPI_QKV_ROPE: rotary pairs (c, c + dh/2) of one head are both in the tile
    const int half = a.dh >> 1;
    for (int idx = tid; idx < a.R * G; idx += nthreads) {
      const int m = idx / G, pi = idx % G;
      int unit, c, col1, col2;
      if (tm.paired) {            // tile = two half-groups of one head
        unit = tile / tm.tiles_per_unit; c = (tile % tm.tiles_per_unit) * G + pi; col1 = pi; col2 = G + pi;
      } else {                    // tile = BN / dh whole heads
        const int hd = pi / half;
        unit = tile * (BN / a.dh) + hd; c = pi % half; col1 = hd * a.dh + c; col2 = col1 + half;
      }
      const int s = m / a.rw.Ms, v = m % a.rw.Ms;
      if (c >= half || unit >= a.H + 2 * a.Hkv || v >= a.rows_active) continue;
      float x1 = C[m * ldc + col1], x2 = C[m * ldc + col2];
      if (unit < a.H + a.Hkv) {   // queries and keys are rotated at the row's tree position
        const float2 cs = a.rope[(size_t)m * half + c];
        const float y1 = x1 * cs.x - x2 * cs.y, y2 = x2 * cs.x + x1 * cs.y;
        x1 = y1; x2 = y2;
      }
      if (unit < a.H) {
        bf16 h1, l1, h2, l2;
        split_bf16(x1, h1, l1); split_bf16(x2, h2, l2);
        bf16 *dst = a.q + (size_t)m * a.H * a.dh + unit * a.dh + c;
        dst[0] = h1; dst[half] = h2;
        dst[a.q_lo_off] = l1; dst[a.q_lo_off + half] = l2;
      } else {                    // the cache stores bf16: one rounding, on store
        const int is_v = unit >= a.H + a.Hkv;
        const int kvh = unit - a.H - (is_v ? a.Hkv : 0);
        const int slot = a.seq_ids[s];
        const int p = a.ctx_len[slot] + v;
        if (p < a.max_ctx) {
          bf16 *dst = a.kcache + (size_t)slot * a.seq_stride + (is_v ? a.kv_stride : 0) +
                      ((size_t)p * a.Hkv + kvh) * a.dh + c;
          dst[0] = __float2bfloat16_rn(x1); dst[half] = __float2bfloat16_rn(x2);
        }
      }
    }
  }
}

}  // namespace firp
