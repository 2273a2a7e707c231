// Core of the tree-masked split-KV decode attention (Section 3.4 "Tree attention"; Section 3.3 for pseudo rows),
// shared by the stand-alone attention kernel and the fused decoder kernel.
//
// Every new row attends to the whole committed prefix [0, n) and, among the new rows of its own sequence (cache
// slots n .. n+rows-1), only to its ancestors and itself; the visibility bits come from the parent array (built
// once per step).  A work item stages 64-position K and V tiles of its split in shared memory (cp.async, double
// buffered), each warp owns 16 query rows (row x head-of-group for grouped-query attention), S = Q K^T and
// O += P V run on the tensor cores with an online softmax in fp32.  Queries and probabilities enter the tensor
// cores as bf16 (hi, lo) pairs accumulated into the same fp32 accumulators, so the only bf16 rounding on this
// path is the cache's own storage format.
#pragma once
#include "firp_kernels.cuh"

namespace firp {

constexpr int kAttnWarps = 4, kAttnThreads = kAttnWarps * 32, kAttnQRows = kAttnWarps * 16;   // threads and query rows of a work item

__device__ __forceinline__ uint32_t attn_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void *src, bool valid) {
  const int sz = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(sz));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }
__device__ __forceinline__ void ldmatrix_x4(uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float *c, const uint32_t *a, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}

// Row r of a [rows][DH] bf16 tile, 16-byte chunk c, XOR-swizzled within each 128-byte line.
template <int DH> __device__ __forceinline__ int tile_off(int r, int c) {
  return r * (DH * 2) + (((c & ~7) | ((c ^ r) & 7)) << 4);
}

// Shared memory of one work item: smem = [2 planes][kAttnQRows][DH] queries, [2][kAttnTile][DH] keys, [2][kAttnTile][DH] values
// (attn_smem_bytes<DH>() bytes, 128-byte aligned); s_mask [kAttnQRows][kMaskWords]; s_row [kAttnQRows].
template <int DH> __host__ __device__ constexpr int attn_smem_bytes() { return 2 * kAttnQRows * DH * 2 + 4 * kAttnTile * DH * 2; }

struct AttnCtaSync { static __device__ __forceinline__ void sync() { __syncthreads(); } };

// One work item = (sequence s, kv head, 64-row query block qb, kv split `split` of `nsplits`), computed by the
// 128 threads tid = 0..127 (4 warps) that share `smem`.  Leaves the split's unnormalised result -- per query
// row its running max (log2 units) m_out[i], its sum l_out[i] and o_out[i][DH] -- in the given arrays, which may
// live in shared or in global memory.  o_out may alias the key tiles of `smem` (it is written after the last
// tile has been consumed).  Sync::sync() is a barrier over exactly those 128 threads.
template <int DH, typename Sync>
__device__ __forceinline__ void attn_split_item(const AttnArgs &a, uint8_t *smem, uint32_t (*s_mask)[kMaskWords], int *s_row,
                                                int tid, int s, int kvh, int qb, int split, int nsplits,
                                                float *m_out, float *l_out, float *o_out) {
  constexpr int CH = DH / 8;          // 16-byte chunks per row
  constexpr int TILE_BYTES = kAttnTile * DH * 2;
  uint8_t *sQ = smem;                               // [2 planes][kAttnQRows][DH]
  constexpr int Q_BYTES = kAttnQRows * DH * 2;
  uint8_t *sK = sQ + 2 * Q_BYTES;                   // [2][kAttnTile][DH]
  uint8_t *sV = sK + 2 * TILE_BYTES;                // [2][kAttnTile][DH]
  const int warp = tid >> 5, lane = tid & 31;
  const int G = a.H / a.Hkv;
  const int qrows_total = a.rows_active * G;
  // the query tile does not depend on the context length: its loads go out first
  for (int ch = tid; ch < kAttnQRows * CH; ch += kAttnThreads) {
    const int i = ch / CH, c = ch % CH;
    const int qr = qb * kAttnQRows + i;
    const bool valid = qr < qrows_total;
    const bf16 *src = valid ? a.q + ((size_t)(s * a.rw.Ms + qr / G) * a.H + kvh * G + qr % G) * DH + c * 8 : a.q;
    cp_async_16(attn_smem_u32(sQ + tile_off<DH>(i, c)), src, valid);
    cp_async_16(attn_smem_u32(sQ + Q_BYTES + tile_off<DH>(i, c)), valid ? src + a.q_lo_off : a.q, valid);
  }
  const int slot = a.seq_ids[s];
  const int n = a.pos[s * a.rw.Ms];                 // position of the root row = committed length (no dependent load)
  const int kv_len = min(n + a.rows_active, a.max_ctx);
  const int tiles_total = (kv_len + kAttnTile - 1) / kAttnTile;
  // balanced ranges; a remainder goes to the first splits, the last one owns the (slower) masked tiles
  const int t0 = (split * tiles_total + nsplits - 1) / nsplits, t1 = ((split + 1) * tiles_total + nsplits - 1) / nsplits;

  const bf16 *kbase = a.kcache + (size_t)kvh * DH;       // row 0 of the plane; a tile's rows follow from kv_row()
  const bf16 *vbase = kbase + a.kv_stride;
  const size_t pos_stride = (size_t)a.Hkv * DH;
  auto load_kv = [&](int buf, int t) {
    const int p0 = t * kAttnTile;
    const size_t row0 = kv_row(a.pages, slot, p0, a.max_ctx);      // the tile lies inside one page
    for (int ch = tid; ch < kAttnTile * CH; ch += kAttnThreads) {
      const int i = ch / CH, c = ch % CH;
      const bool valid = (p0 + i) < kv_len;
      const size_t off = (row0 + i) * pos_stride + c * 8;
      cp_async_16(attn_smem_u32(sK + buf * TILE_BYTES + tile_off<DH>(i, c)), valid ? kbase + off : kbase, valid);
      cp_async_16(attn_smem_u32(sV + buf * TILE_BYTES + tile_off<DH>(i, c)), valid ? vbase + off : vbase, valid);
    }
  };
  if (t0 < t1) load_kv(0, t0);
  cp_async_commit();
  // query rows of this block: qr -> (tree row v = qr / G, head = kvh * G + qr % G), and their visibility words
  for (int i = tid; i < kAttnQRows; i += kAttnThreads) {
    const int qr = qb * kAttnQRows + i;
    int r = -1;
    if (qr < qrows_total) r = s * a.rw.Ms + qr / G;
    s_row[i] = r;
    for (int w = 0; w < kMaskWords; ++w) s_mask[i][w] = (r >= 0) ? a.mask[(size_t)r * kMaskWords + w] : 0u;
  }

  const int g = lane >> 2, t4 = lane & 3, mi = lane >> 3, r8 = lane & 7;
  const float scale_log2 = rsqrtf((float)DH) * 1.4426950408889634f;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  float o_acc[DH / 8][4];
#pragma unroll
  for (int i = 0; i < DH / 8; ++i) { o_acc[i][0] = o_acc[i][1] = o_acc[i][2] = o_acc[i][3] = 0.f; }

  for (int t = t0; t < t1; ++t) {
    const int buf = (t - t0) & 1;
    if (t + 1 < t1) load_kv(buf ^ 1, t + 1);
    cp_async_commit();
    cp_async_wait<1>();
    Sync::sync();
    const uint8_t *kt = sK + buf * TILE_BYTES, *vt = sV + buf * TILE_BYTES;
    // S = Q K^T over the 64 positions of the tile
    float sc[kAttnTile / 8][4];
#pragma unroll
    for (int i = 0; i < kAttnTile / 8; ++i) { sc[i][0] = sc[i][1] = sc[i][2] = sc[i][3] = 0.f; }
#pragma unroll
    for (int kk = 0; kk < DH / 16; ++kk) {
      uint32_t qh[4], ql[4];
      {
        const int row = warp * 16 + (mi & 1) * 8 + r8, chunk = kk * 2 + (mi >> 1);
        ldmatrix_x4(qh[0], qh[1], qh[2], qh[3], attn_smem_u32(sQ + tile_off<DH>(row, chunk)));
        ldmatrix_x4(ql[0], ql[1], ql[2], ql[3], attn_smem_u32(sQ + Q_BYTES + tile_off<DH>(row, chunk)));
      }
#pragma unroll
      for (int p = 0; p < kAttnTile / 16; ++p) {
        uint32_t b0, b1, b2, b3;
        const int row = p * 16 + (mi >> 1) * 8 + r8, chunk = kk * 2 + (mi & 1);
        ldmatrix_x4(b0, b1, b2, b3, attn_smem_u32(kt + tile_off<DH>(row, chunk)));
        mma_bf16(sc[2 * p], qh, b0, b1);
        mma_bf16(sc[2 * p + 1], qh, b2, b3);
        if (a.q_planes > 1) {
          mma_bf16(sc[2 * p], ql, b0, b1);
          mma_bf16(sc[2 * p + 1], ql, b2, b3);
        }
      }
    }
    // mask, scale, online softmax (rows g and g+8 of this warp's 16)
    const int p0 = t * kAttnTile;
    const bool need_mask = (p0 + kAttnTile > n);
    // visibility of the tile's 64 positions for this thread's two rows: bit j = position p0 + j;
    // positions below n are the committed prefix (visible), position n + u is new row u (mask bit u)
    uint32_t vis[2][2] = {{~0u, ~0u}, {~0u, ~0u}};
    if (need_mask) {
#pragma unroll
      for (int rr = 0; rr < 2; ++rr) {
        const uint32_t *mw = s_mask[warp * 16 + g + rr * 8];
#pragma unroll
        for (int hw = 0; hw < 2; ++hw) {
          const int sh = p0 + 32 * hw - n;             // mask bit of this word's bit 0
          uint32_t bits;
          if (sh <= -32) bits = ~0u;
          else if (sh < 0) bits = (mw[0] << (-sh)) | ((1u << (-sh)) - 1u);
          else {
            const int w = sh >> 5, bsh = sh & 31;
            const uint32_t lo = (w < kMaskWords) ? mw[w] : 0u, hi = (w + 1 < kMaskWords) ? mw[w + 1] : 0u;
            bits = bsh ? ((lo >> bsh) | (hi << (32 - bsh))) : lo;
          }
          vis[rr][hw] = bits;
        }
      }
    }
    float mx[2] = {m_run[0], m_run[1]};
#pragma unroll
    for (int nt = 0; nt < kAttnTile / 8; ++nt) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int rr = e >> 1, j = nt * 8 + t4 * 2 + (e & 1);
        float v = sc[nt][e] * scale_log2;
        if (!((vis[rr][j >> 5] >> (j & 31)) & 1u)) v = -INFINITY;
        sc[nt][e] = v;
        mx[rr] = fmaxf(mx[rr], v);
      }
    }
    float corr[2], msafe[2];
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      mx[rr] = fmaxf(mx[rr], __shfl_xor_sync(0xffffffffu, mx[rr], 1));
      mx[rr] = fmaxf(mx[rr], __shfl_xor_sync(0xffffffffu, mx[rr], 2));
      msafe[rr] = (mx[rr] == -INFINITY) ? 0.f : mx[rr];
      corr[rr] = exp2f(m_run[rr] - msafe[rr]);      // m_run = -inf -> 0
      m_run[rr] = mx[rr];
      l_run[rr] *= corr[rr];
    }
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) {
      o_acc[i][0] *= corr[0]; o_acc[i][1] *= corr[0]; o_acc[i][2] *= corr[1]; o_acc[i][3] *= corr[1];
    }
    uint32_t pf[kAttnTile / 16][4], pl[kAttnTile / 16][4];   // probabilities as bf16 hi and lo halves
#pragma unroll
    for (int nt = 0; nt < kAttnTile / 8; ++nt) {
      const float e0 = exp2f(sc[nt][0] - msafe[0]), e1 = exp2f(sc[nt][1] - msafe[0]);
      const float e2 = exp2f(sc[nt][2] - msafe[1]), e3 = exp2f(sc[nt][3] - msafe[1]);
      l_run[0] += e0 + e1; l_run[1] += e2 + e3;
      const __nv_bfloat162 h01 = __floats2bfloat162_rn(e0, e1), h23 = __floats2bfloat162_rn(e2, e3);
      const float2 f01 = __bfloat1622float2(h01), f23 = __bfloat1622float2(h23);
      pf[nt >> 1][(nt & 1) * 2 + 0] = *reinterpret_cast<const uint32_t *>(&h01);
      pf[nt >> 1][(nt & 1) * 2 + 1] = *reinterpret_cast<const uint32_t *>(&h23);
      pl[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(e0 - f01.x, e1 - f01.y);
      pl[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(e2 - f23.x, e3 - f23.y);
    }
    // O += P V
#pragma unroll
    for (int j = 0; j < kAttnTile / 16; ++j) {
#pragma unroll
      for (int d2 = 0; d2 < DH / 16; ++d2) {
        uint32_t b0, b1, b2, b3;
        const int row = j * 16 + (mi & 1) * 8 + r8, chunk = d2 * 2 + (mi >> 1);
        ldmatrix_x4_trans(b0, b1, b2, b3, attn_smem_u32(vt + tile_off<DH>(row, chunk)));
        mma_bf16(o_acc[2 * d2], pf[j], b0, b1);
        mma_bf16(o_acc[2 * d2 + 1], pf[j], b2, b3);
        if (a.p_planes > 1) {
          mma_bf16(o_acc[2 * d2], pl[j], b0, b1);
          mma_bf16(o_acc[2 * d2 + 1], pl[j], b2, b3);
        }
      }
    }
    Sync::sync();
  }
  cp_async_wait<0>();

  // this split's partial result (the key tiles are free now, should o_out alias them)
  static_assert(2 * TILE_BYTES >= kAttnQRows * DH * 4, "a partial O must fit the key tiles");
  Sync::sync();
#pragma unroll
  for (int rr = 0; rr < 2; ++rr) {
    float l = l_run[rr];
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    const int i = warp * 16 + g + rr * 8;
    if (t4 == 0) { m_out[i] = m_run[rr]; l_out[i] = l; }
#pragma unroll
    for (int nt = 0; nt < DH / 8; ++nt)
      *reinterpret_cast<float2 *>(o_out + i * DH + nt * 8 + t4 * 2) = make_float2(o_acc[nt][rr * 2], o_acc[nt][rr * 2 + 1]);
  }
}

}  // namespace firp
