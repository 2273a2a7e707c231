// Tree-masked split-KV decode attention on the tcgen05 tensor cores (Section 3.4 "Tree attention"; Section 3.3
// for the pseudo rows), head dimension 128.
//
// Roles are swapped as in the GEMMs: a tile of 128 cached positions is the MMA's M dimension, the query rows of
// the block (tree rows x heads of the group, <= 48) its N dimension.
//   S^T = K Q^T      K tile [128 pos][128 dh] K-major (TMA, 128-byte swizzle), Q [NQ][128] K-major (hi and lo
//                    bf16 planes, both accumulated into the same fp32 columns)           -> NQ TMEM columns
//   softmax          thread i of a warpgroup owns position i of the tile (= TMEM lane i): scale, visibility,
//                    column maxima and sums over the 128 positions (warp butterflies + shared memory), P = 2^(s - m)
//                    as bf16 (hi, lo) planes written to shared memory as [NQ][128 pos] K-major
//   O^T = V^T P^T    V tile [128 pos][128 dh] as the MN-major A operand (M = dh)         -> NQ TMEM columns
// A CTA keeps two tiles of its kv range in flight (tile groups 0 and 1 take the tiles in turn), each with its own
// K, V and P buffers, TMEM columns and running (max, sum, O^T), so that the tensor-core work of one overlaps the
// softmax of the other; the query columns of a tile are shared by two warpgroups (halves), which makes four
// softmax warpgroups: thread i of each keeps O^T[i][its columns] (dh index i) in registers.  One thread issues
// every MMA, two more feed the K and the V buffers by TMA.  The CTAs of one (kv head, query block) -- the kv
// splits -- form a cluster; every partial result (split, tile group) is pushed, four columns at a time, to the
// CTA that finalises those columns.  One CTA per SM (shared memory), so the 256 TMEM columns it allocates are
// never contended.  Every mbarrier wait is bounded; a wait that runs out sets the status word and the kernel runs to
// its end.
#include <cooperative_groups.h>

#include <map>
#include <tuple>

#include "firp_kernels.cuh"
#include "launch_util.cuh"
#include "tc_device.cuh"

namespace cg = cooperative_groups;

namespace firp {

namespace {

constexpr int kTcDh = 128;                  // head dimension this kernel is written for
constexpr int kTcTile = 128;                // cached positions per tile (MMA M)
constexpr int kTcWg = 128;                  // threads of a warpgroup
constexpr int kTcSoft = 4 * kTcWg;          // softmax threads: 2 tile groups x 2 column halves
constexpr int kTcThreads = kTcSoft + 96;    // + the MMA issuer's warp, the K and the V producer's
constexpr int kTcSlab = kTcTile * 128;      // bytes of one [128 rows][64 elements] slab
constexpr int kTcStage = 2 * kTcSlab;       // a K or V tile: two slabs (dh halves)
constexpr int kTcTmemCols = 256;

template <int NQ> struct TcLayout {
  static constexpr int Q_SLAB = NQ * 128;                 // [NQ rows][64 elements]
  static constexpr int K_OFF = 0;                         // [2 warpgroups][2 dh halves][128 pos][128 B]
  static constexpr int V_OFF = K_OFF + 2 * kTcStage;      // [2 warpgroups][2 dh halves][128 pos][128 B]
  static constexpr int Q_OFF = V_OFF + 2 * kTcStage;      // [2 planes][2 dh halves][NQ][128 B]
  static constexpr int P_OFF = Q_OFF + 4 * Q_SLAB;        // [2 warpgroups][2 planes][2 pos halves][NQ][128 B]
  static constexpr int BYTES = P_OFF + 8 * Q_SLAB;
  static_assert(NQ % 16 == 0 && NQ >= 16 && NQ <= 48 && 4 * NQ <= kTcTmemCols, "query columns per block");
  static_assert(2 * (NQ + 4 * 8) * kTcDh * 4 <= 4 * kTcStage, "the partials a CTA receives must fit the K and V buffers");
  static_assert(BYTES + 1024 + 6144 <= 227 * 1024, "shared memory budget (dynamic + alignment + static)");
};

// MN-major operand, 128-byte swizzle: 64 elements of M contiguous (128 bytes), the 8 rows of a K group 128 bytes
// apart, K groups `1024` bytes apart (stride offset), 64-element M blocks lbo_bytes apart (leading offset).
__device__ __forceinline__ uint64_t smem_desc_mn(uint32_t addr, uint32_t lbo_bytes) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void wg_sync(int w) { asm volatile("bar.sync %0, 128;" ::"r"(1 + w) : "memory"); }
__device__ __forceinline__ void tc_ld8(uint32_t taddr, float *r) {
  uint32_t *u = reinterpret_cast<uint32_t *>(r);
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7])
               : "r"(taddr) : "memory");
}
// N = 8, 16 or 24 consecutive columns of this warp's lanes (no wait)
template <int N> __device__ __forceinline__ void tc_ld_cols(uint32_t taddr, float *r) {
  static_assert(N == 8 || N == 16 || N == 24, "columns per warpgroup");
  if (N >= 16) tc_ld16(taddr, r);
  if (N == 8) tc_ld8(taddr, r);
  if (N == 24) tc_ld8(taddr + 16, r + 16);
}
// Reduction (max or sum) over the 32 lanes of N = 8 or 16 columns at once: in each butterfly step a lane keeps
// half of its columns and trades the other half with its partner, so N columns cost N + log2(32 / N) - 1 shuffles
// instead of 5 N.  Destroys v; lane L returns the result of column L * N / 32 (N = 16: L >> 1, N = 8: L >> 2).
template <int N, bool SUM> __device__ __forceinline__ float warp_col_reduce(float *v, int lane) {
  static_assert(N == 8 || N == 16, "columns per butterfly");
  int m = 16;
#pragma unroll
  for (int half = N / 2; half >= 1; half >>= 1, m >>= 1) {
    const bool up = (lane & m) != 0;
#pragma unroll
    for (int c = 0; c < half; ++c) {
      const float got = __shfl_xor_sync(0xffffffffu, up ? v[c] : v[c + half], m);
      const float kept = up ? v[c + half] : v[c];
      v[c] = SUM ? kept + got : fmaxf(kept, got);
    }
  }
#pragma unroll
  for (; m >= 1; m >>= 1) {
    const float got = __shfl_xor_sync(0xffffffffu, v[0], m);
    v[0] = SUM ? v[0] + got : fmaxf(v[0], got);
  }
  return v[0];
}
// The same for NH = 8, 16 or 24 columns (a block of 16, then one of 8); the results go to dst[column][slot].
template <int NH, bool SUM> __device__ __forceinline__ void warp_cols_to_smem(const float *v, float (*dst)[4], int slot, int lane) {
  if (NH >= 16) {
    float t[16];
#pragma unroll
    for (int c = 0; c < 16; ++c) t[c] = v[c];
    const float r = warp_col_reduce<16, SUM>(t, lane);
    if ((lane & 1) == 0) dst[lane >> 1][slot] = r;
  }
  if (NH == 8 || NH == 24) {
    constexpr int o = NH == 24 ? 16 : 0;
    float t[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) t[c] = v[o + c];
    const float r = warp_col_reduce<8, SUM>(t, lane);
    if ((lane & 3) == 0) dst[o + (lane >> 2)][slot] = r;
  }
}

#ifdef FIRP_ATTN_TRACE
__device__ unsigned long long g_attn_trace[16];
#define TC_STAMP(k) do { if (tid == 0 && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0) g_attn_trace[k] = globaltimer(); } while (0)
#else
#define TC_STAMP(k) do { } while (0)
#endif

template <int NQ>
__global__ void __launch_bounds__(kTcThreads, 1)
tree_attn_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, AttnArgs a,
                    int qper, int pdl) {
  using LY = TcLayout<NQ>;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(16) float s_red[2][NQ][4];   // per tile group and column: its four warps' maxima of the tile
  __shared__ __align__(16) float s_lred[2][NQ][4];  // and their sums of P, added to the running sum one tile later
  __shared__ __align__(16) float s_m[2][NQ];        // running max (log2 units)
  __shared__ __align__(16) float s_corr[2][NQ];     // 2^(old max - new max) of the current tile; merge weights at the end
  __shared__ __align__(16) float s_l[2][NQ];        // running sum
  __shared__ __align__(16) float s_pm[2 * (NQ + 4 * kAttnMaxSplits)], s_pl[2 * (NQ + 4 * kAttnMaxSplits)];   // (max, sum) received for the merge: [partial][slot][4 columns]
  __shared__ uint32_t s_oidx[NQ];                   // element offset of each column's output row
  // mbarriers: K landed [2], V landed [2], S^T complete [2], P written [2], O^T complete [2], Q written
  __shared__ __align__(8) uint64_t s_bar[11];
  __shared__ uint32_t s_tmem;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  TC_STAMP(0);
  uint8_t *base = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t sb = smem_u32(base);
  const uint32_t bar0 = smem_u32(s_bar);
  const uint32_t full_k = bar0, full_v = bar0 + 16, s_ready = bar0 + 32, p_ready = bar0 + 48, o_ready = bar0 + 64,
                 q_ready = bar0 + 80;               // [w] of a pair: + 8 w

  if (tid == 0) {
    for (int i = 0; i < 6; ++i) mbar_init(bar0 + 8 * i, 1);
    mbar_init(p_ready, 2 * kTcWg); mbar_init(p_ready + 8, 2 * kTcWg);
    mbar_init(o_ready, 1); mbar_init(o_ready + 8, 1);
    mbar_init(q_ready, kTcSoft);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int j = tid; j < 2 * NQ * 4; j += kTcThreads) (&s_lred[0][0][0])[j] = 0.f;
  for (int j = tid; j < 2 * NQ; j += kTcThreads) { (&s_m[0][0])[j] = -INFINITY; (&s_l[0][0])[j] = 0.f; }
  if (warp == 16) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(kTcTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem;
  if (pdl) { griddep_launch(); griddep_wait(); }
  TC_STAMP(1);

  const int kvh = blockIdx.y, G = a.H / a.Hkv;
  const int qblocks = gridDim.z / a.rw.n_seq;
  const int s = blockIdx.z / qblocks, qb = blockIdx.z % qblocks;
  const int split = blockIdx.x, nsplits = gridDim.x;
  const int qrows_total = a.rows_active * G, q0 = qb * qper;
  const int ncols = min(qper, qrows_total - q0);
  const int slot = a.seq_ids[s];
  const int n = a.pos[s * a.rw.Ms];                 // position of the root row = committed length
  // queries of this block (all softmax threads share the work): column j = query row q0 + j -> (tree row
  // (q0 + j) / G, head kvh G + (q0 + j) % G).  Their loads go out before the context length above is first used.
  constexpr int QIT = (NQ * 16 + kTcSoft - 1) / kTcSoft;
  uint4 qh[QIT], ql[QIT];
  if (warp < 16) {
#pragma unroll
    for (int it = 0; it < QIT; ++it) {
      const int idx = it * kTcSoft + tid, j = idx >> 4, c = idx & 15, qr = q0 + j;
      qh[it] = make_uint4(0u, 0u, 0u, 0u); ql[it] = qh[it];
      if (j < ncols) {
        const bf16 *src = a.q + ((size_t)(s * a.rw.Ms + qr / G) * a.H + kvh * G + qr % G) * kTcDh + c * 8;
        qh[it] = *reinterpret_cast<const uint4 *>(src);
        ql[it] = *reinterpret_cast<const uint4 *>(src + a.q_lo_off);
      }
    }
  }
  const int kv_len = min(n + a.rows_active, a.max_ctx);
  const int tiles_total = (kv_len + kTcTile - 1) / kTcTile;
  const int t0 = (split * tiles_total + nsplits - 1) / nsplits, t1 = ((split + 1) * tiles_total + nsplits - 1) / nsplits;
  const int ntiles = t1 - t0;                       // tile t0 + i goes to warpgroup i & 1 as its (i >> 1)-th
  const unsigned long long wait_ns = a.wait_ns ? a.wait_ns : kDefaultWaitNs;
  bool dead = false;
  constexpr int NH = NQ / 2;                        // columns per warpgroup
  float o_acc[NH];                                  // softmax threads: O^T[dh index][own columns] of the tiles so far
#pragma unroll
  for (int j = 0; j < NH; ++j) o_acc[j] = 0.f;

  if (warp >= 17) {
    // ---- producers (one lane each): warp 17 feeds the K buffers, warp 18 the V buffers.  A buffer is free again
    // when the MMAs that read it have completed, which is what s_ready / o_ready of its warpgroup report.
    if (lane == 0) {
      const bool is_v = warp == 18;
      const CUtensorMap *tm = is_v ? &tmV : &tmK;
      const uint32_t full = is_v ? full_v : full_k, freed = is_v ? o_ready : s_ready;
      const uint32_t dst0 = sb + (is_v ? LY::V_OFF : LY::K_OFF);
      uint64_t pol;
      asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(pol));
      for (int i = 0; i < ntiles; ++i) {
        const int w = i & 1, q = i >> 1, t = t0 + i;
        if (q > 0) mbar_wait(freed + 8 * w, (q - 1) & 1, a.err, dead, wait_ns);
        mbar_expect_tx(full + 8 * w, kTcStage);
#pragma unroll
        for (int ph = 0; ph < 2; ++ph) {            // 64-position x 64-element boxes; a half lies inside one page
          const int p0 = t * kTcTile + ph * 64;
          const int row = (int)kv_row(a.pages, slot, p0 < kv_len ? p0 : 0, a.max_ctx);   // a half beyond the context: any rows
#pragma unroll
          for (int h = 0; h < 2; ++h)
            tma_load_2d(dst0 + (uint32_t)(w * kTcStage + h * kTcSlab + ph * 8192), tm, kvh * kTcDh + h * 64, row,
                        full + 8 * w, pol);
        }
      }
    }
  } else if (warp == 16) {
    // ---- MMA issuer (one lane): S^T of tile i, then O^T of tile i - 1
    if (lane == 0) {
      const uint32_t idesc_k = instr_desc_m128(NQ), idesc_mn = idesc_k | (1u << 15);
      // operand descriptors of warpgroup 0; another buffer, dh half or k step only moves the start address
      const uint64_t kdesc0 = smem_desc(sb + LY::K_OFF), qdesc0 = smem_desc(sb + LY::Q_OFF);
      const uint64_t vdesc0 = smem_desc_mn(sb + LY::V_OFF, kTcSlab), pdesc0 = smem_desc(sb + LY::P_OFF);
      mbar_wait(q_ready, 0, a.err, dead, wait_ns);
      for (int i = 0; i <= ntiles; ++i) {
        if (i < ntiles) {
          const int w = i & 1, q = i >> 1;
          mbar_wait(full_k + 8 * w, q & 1, a.err, dead, wait_ns);
          if (q > 0) mbar_wait(p_ready + 8 * w, (q - 1) & 1, a.err, dead, wait_ns);   // S^T of its previous tile has been read
          tc_fence_after();
          uint32_t acc = 0;
          for (int pl = 0; pl < a.q_planes; ++pl)
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
              tc_mma(tmem + w * 2 * NQ, kdesc0 + (uint64_t)((w * kTcStage + (kk >> 2) * kTcSlab + (kk & 3) * 32) >> 4),
                     qdesc0 + (uint64_t)((pl * 2 * LY::Q_SLAB + (kk >> 2) * LY::Q_SLAB + (kk & 3) * 32) >> 4), idesc_k, acc);
              acc = 1;
            }
          tc_commit(s_ready + 8 * w);
        }
        if (i >= 1) {
          const int w = (i - 1) & 1, q = (i - 1) >> 1;
          mbar_wait(p_ready + 8 * w, q & 1, a.err, dead, wait_ns);
          mbar_wait(full_v + 8 * w, q & 1, a.err, dead, wait_ns);
          tc_fence_after();
          uint32_t acc = 0;
          for (int pl = 0; pl < a.p_planes; ++pl)
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              const uint64_t bdesc = pdesc0 + (uint64_t)((w * 4 * LY::Q_SLAB + pl * 2 * LY::Q_SLAB + (ks >> 2) * LY::Q_SLAB + (ks & 3) * 32) >> 4);
              tc_mma(tmem + w * 2 * NQ + NQ, vdesc0 + (uint64_t)((w * kTcStage + ks * 2048) >> 4), bdesc, idesc_mn, acc);
              acc = 1;
            }
          tc_commit(o_ready + 8 * w);
        }
      }
    }
  } else {
    // ---- the four softmax warpgroups: tile group g takes tiles g, g + 2, ...; half h of it owns the query columns
    // [h NH, (h + 1) NH) of those tiles
    const int wgi = warp >> 2, g = wgi >> 1, h = wgi & 1, wt = tid & (kTcWg - 1);
    const int c_lo = h * NH;
    const uint32_t tlane = tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(g * 2 * NQ + c_lo);
    {
#pragma unroll
      for (int it = 0; it < QIT; ++it) {
        const int idx = it * kTcSoft + tid, j = idx >> 4, c = idx & 15;
        if (j < NQ) {
          const int off = (c >> 3) * LY::Q_SLAB + j * 128 + (((c & 7) ^ (j & 7)) << 4);
          *reinterpret_cast<uint4 *>(base + LY::Q_OFF + off) = qh[it];
          *reinterpret_cast<uint4 *>(base + LY::Q_OFF + 2 * LY::Q_SLAB + off) = ql[it];
        }
      }
      TC_STAMP(15);
      fence_async_smem();
      mbar_arrive(q_ready);
      if (tid < ncols) {
        const int qr = q0 + tid;
        s_oidx[tid] = (uint32_t)(((s * a.rw.Ms + qr / G) * a.H + kvh * G + qr % G) * kTcDh);
      }
    }
    TC_STAMP(2);
    const float scale_log2 = rsqrtf((float)kTcDh) * 1.4426950408889634f;
    // where this thread's position pair goes in a P row: 64-position half, 16-byte chunk, element
    const int p_half = wt >> 6, p_chunk = (wt & 63) >> 3, p_el2 = wt & 6, odd = wt & 1;
    uint8_t *pbase = base + LY::P_OFF + g * 4 * LY::Q_SLAB;

    for (int i = g; i < ntiles; i += 2) {
      const int q = i >> 1, t = t0 + i;
      const int p = t * kTcTile + wt;
      const bool pvalid = p < kv_len;
      // visibility of position p for this half's query columns (bit jj = column c_lo + jj): the committed prefix
      // is visible to all, new row u = p - n to the rows whose mask has bit u
      uint32_t vis = pvalid ? ~0u : 0u;
      if (pvalid && p >= n) {
        const int u = p - n, mw = u >> 5, b = u & 31;
        vis = 0u;
#pragma unroll
        for (int jj = 0; jj < NH; ++jj) {
          const int qr = min(q0 + c_lo + jj, qrows_total - 1);
          const uint32_t word = a.mask[(size_t)(s * a.rw.Ms + qr / G) * kMaskWords + mw];
          vis |= ((word >> b) & 1u) << jj;
        }
      }
      __syncwarp();
      mbar_wait(s_ready + 8 * g, q & 1, a.err, dead, wait_ns);
      tc_fence_after();
      if (i == 0) TC_STAMP(3);
      // pass 1: the tile's scores of this position (one wait for all TMEM loads), scaled and masked, and the
      // column maxima over the tile's positions
      float sv[NH];
      tc_ld_cols<NH>(tlane, sv);
      tc_ld_wait();
#pragma unroll
      for (int j = 0; j < NH; ++j) sv[j] = ((vis >> j) & 1u) ? sv[j] * scale_log2 : -INFINITY;
      warp_cols_to_smem<NH, false>(sv, &s_red[g][c_lo], warp & 3, lane);
      wg_sync(wgi);
      if (i == 0) TC_STAMP(4);
      if (wt < NH) {
        const int j = c_lo + wt;
        const float4 v = *reinterpret_cast<const float4 *>(s_red[g][j]);
        const float4 ps = *reinterpret_cast<const float4 *>(s_lred[g][j]);      // the previous tile's sums of P
        const float mt = fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w));
        const float m_old = s_m[g][j], m_new = fmaxf(m_old, mt);
        const float cr = exp2f(m_old - (m_new == -INFINITY ? 0.f : m_new));
        s_corr[g][j] = cr;
        s_m[g][j] = m_new;
        s_l[g][j] = (s_l[g][j] + ((ps.x + ps.y) + (ps.z + ps.w))) * cr;
      }
      wg_sync(wgi);
      if (i == 0) TC_STAMP(5);
      // pass 2: P = 2^(s - m) as bf16 (hi, lo) into the B operand of the second contraction.  Lanes 2i and 2i + 1
      // hold neighbouring positions: they swap one column of each column pair, so that every lane converts and
      // stores two neighbouring positions of one column as one 32-bit word.
#pragma unroll
      for (int c0 = 0; c0 < NH; c0 += 8) {
        float ms[8];
#pragma unroll
        for (int q4 = 0; q4 < 2; ++q4) {
          const float4 m4 = *reinterpret_cast<const float4 *>(&s_m[g][c_lo + c0 + 4 * q4]);
          ms[4 * q4] = m4.x; ms[4 * q4 + 1] = m4.y; ms[4 * q4 + 2] = m4.z; ms[4 * q4 + 3] = m4.w;
        }
        float *r = sv + c0;
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) {
          const float msafe = (ms[jj] == -INFINITY) ? 0.f : ms[jj];
          r[jj] = exp2f(r[jj] - msafe);                                       // masked: 2^-inf = 0
        }
#pragma unroll
        for (int jj = 0; jj < 8; jj += 2) {
          const float got = __shfl_xor_sync(0xffffffffu, odd ? r[jj] : r[jj + 1], 1);
          const float x = odd ? got : r[jj], y = odd ? r[jj + 1] : got;      // positions 2i, 2i + 1 of column jj + odd
          const __nv_bfloat162 hh = __floats2bfloat162_rn(x, y);
          const float2 hf = __bfloat1622float2(hh);
          const __nv_bfloat162 ll = __floats2bfloat162_rn(x - hf.x, y - hf.y);
          const int j = c_lo + c0 + jj + odd;
          const int off = p_half * LY::Q_SLAB + j * 128 + ((p_chunk ^ (j & 7)) << 4) + p_el2 * 2;
          *reinterpret_cast<__nv_bfloat162 *>(pbase + off) = hh;
          *reinterpret_cast<__nv_bfloat162 *>(pbase + 2 * LY::Q_SLAB + off) = ll;
        }
      }
      warp_cols_to_smem<NH, true>(sv, &s_lred[g][c_lo], warp & 3, lane);      // this warp's sums of P per column
      if (!pvalid && h == 0) {   // a position beyond the context: its V row may hold anything, and 0 x NaN is NaN
        mbar_wait(full_v + 8 * g, q & 1, a.err, dead, wait_ns);
        uint4 *v0 = reinterpret_cast<uint4 *>(base + LY::V_OFF + g * kTcStage + wt * 128);
        uint4 *v1 = reinterpret_cast<uint4 *>(base + LY::V_OFF + g * kTcStage + kTcSlab + wt * 128);
#pragma unroll
        for (int c = 0; c < 8; ++c) { v0[c] = make_uint4(0u, 0u, 0u, 0u); v1[c] = make_uint4(0u, 0u, 0u, 0u); }
      }
      fence_async_smem();
      tc_fence_before();
      mbar_arrive(p_ready + 8 * g);
      if (i == 0) TC_STAMP(6);
      mbar_wait(o_ready + 8 * g, q & 1, a.err, dead, wait_ns);
      tc_fence_after();
      if (i == 0) TC_STAMP(7);
      // O^T of the tile joins the running one
      float *ov = sv;                                  // the scores are dead
      tc_ld_cols<NH>(tlane + NQ, ov);
      tc_ld_wait();
#pragma unroll
      for (int q4 = 0; q4 < NH / 4; ++q4) {
        const float4 c4 = *reinterpret_cast<const float4 *>(&s_corr[g][c_lo + 4 * q4]);
        o_acc[4 * q4] = o_acc[4 * q4] * c4.x + ov[4 * q4];
        o_acc[4 * q4 + 1] = o_acc[4 * q4 + 1] * c4.y + ov[4 * q4 + 1];
        o_acc[4 * q4 + 2] = o_acc[4 * q4 + 2] * c4.z + ov[4 * q4 + 2];
        o_acc[4 * q4 + 3] = o_acc[4 * q4 + 3] * c4.w + ov[4 * q4 + 3];
      }
      tc_fence_before();
      if (i == 0) TC_STAMP(8);
    }
  }
  TC_STAMP(9);
  // ---- merge: o = sum_p 2^(m_p - M) O_p / sum_p 2^(m_p - M) l_p over the partials p = (kv split, tile group).
  // Columns go in groups of four; group c is finalised by CTA c % splits.  Once every CTA of the cluster has left
  // its tile loop (its buffers are free), every softmax thread pushes its columns of its tile group's partial into
  // the owners' shared memory (16-byte remote stores: O^T[dh][4 columns]), the columns' (m, l) likewise; after a
  // second cluster barrier the owners merge what they received, in partial order, from their own shared memory.
  // A lone CTA takes the same route through its own shared memory.
  const int nsp = nsplits;
  const int my_g = warp >> 3, my_lo = ((warp >> 2) & 1) * NH, my_t = tid & (kTcWg - 1);   // of a softmax thread
  if (warp < 16) {
    wg_sync(warp >> 2);                              // the last tile's sums of P are in shared memory
    if (my_t < NH) {
      const int j = my_lo + my_t;
      const float4 ps = *reinterpret_cast<const float4 *>(s_lred[my_g][j]);
      s_l[my_g][j] += (ps.x + ps.y) + (ps.z + ps.w);
    }
  }
  tc_fence_before();
  cg::cluster_group cluster = cg::this_cluster();
  if (nsp > 1) cluster.sync(); else __syncthreads();
  TC_STAMP(11);
  if (warp == 16) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTcTmemCols) : "memory");
  }
  const int rank = (nsp > 1) ? (int)cluster.block_rank() : 0;
  constexpr int NG = NQ / 4;                                    // column groups
  const int slots = (NG + nsp - 1) / nsp;                       // groups an owner may receive from one partial
  const int nparts = 2 * nsp, part = 2 * rank + my_g;
  float4 *sM = reinterpret_cast<float4 *>(base + LY::K_OFF);    // [partials][slots][128 dh] x 4 columns, over the K and V buffers
  if (warp < 16) {
    int owner = (my_lo / 4) % nsp, slot_c = (my_lo / 4) / nsp;
#pragma unroll
    for (int c = 0; c < NH / 4; ++c) {
      if (my_lo + 4 * c < ncols) {
        float4 *dst = (nsp > 1) ? cluster.map_shared_rank(sM, owner) : sM;
        dst[(size_t)(part * slots + slot_c) * kTcDh + my_t] = make_float4(o_acc[4 * c], o_acc[4 * c + 1], o_acc[4 * c + 2], o_acc[4 * c + 3]);
      }
      if (++owner == nsp) { owner = 0; ++slot_c; }
    }
    if (my_t < NH && my_lo + my_t < ncols) {
      const int j = my_lo + my_t, ow = (j >> 2) % nsp, sl = (j >> 2) / nsp;
      float *dm = (nsp > 1) ? cluster.map_shared_rank(s_pm, ow) : s_pm;
      float *dl = (nsp > 1) ? cluster.map_shared_rank(s_pl, ow) : s_pl;
      dm[(part * slots + sl) * 4 + (j & 3)] = s_m[my_g][j];
      dl[(part * slots + sl) * 4 + (j & 3)] = s_l[my_g][j];
    }
  }
  TC_STAMP(12);
  if (nsp > 1) cluster.sync(); else __syncthreads();
  TC_STAMP(13);
  // owners: warpgroup w takes the received groups w, w + 4, ...; thread t of it dh index t of the group's four columns
  if (warp < 16) {
    for (int sl = warp >> 2; rank + sl * nsp < NG && 4 * (rank + sl * nsp) < ncols; sl += 4) {
      const int j0 = 4 * (rank + sl * nsp);
      float4 M = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
      for (int sp = 0; sp < nparts; ++sp) {
        const float4 pm = *reinterpret_cast<const float4 *>(&s_pm[(sp * slots + sl) * 4]);
        M.x = fmaxf(M.x, pm.x); M.y = fmaxf(M.y, pm.y); M.z = fmaxf(M.z, pm.z); M.w = fmaxf(M.w, pm.w);
      }
      float4 L = make_float4(0.f, 0.f, 0.f, 0.f), acc = L;
      for (int sp = 0; sp < nparts; ++sp) {
        const float4 pm = *reinterpret_cast<const float4 *>(&s_pm[(sp * slots + sl) * 4]);
        const float4 pl = *reinterpret_cast<const float4 *>(&s_pl[(sp * slots + sl) * 4]);
        const float4 ov = sM[(size_t)(sp * slots + sl) * kTcDh + my_t];
        // a partial without tiles, or a column all of whose positions were masked in it: weight 0
        const float wx = (pm.x == -INFINITY) ? 0.f : exp2f(pm.x - M.x), wy = (pm.y == -INFINITY) ? 0.f : exp2f(pm.y - M.y);
        const float wz = (pm.z == -INFINITY) ? 0.f : exp2f(pm.z - M.z), ww = (pm.w == -INFINITY) ? 0.f : exp2f(pm.w - M.w);
        L.x += wx * pl.x; L.y += wy * pl.y; L.z += wz * pl.z; L.w += ww * pl.w;
        acc.x += wx * ov.x; acc.y += wy * ov.y; acc.z += wz * ov.z; acc.w += ww * ov.w;
      }
      const float val[4] = {acc.x * ((L.x > 0.f) ? 1.f / L.x : 0.f), acc.y * ((L.y > 0.f) ? 1.f / L.y : 0.f),
                            acc.z * ((L.z > 0.f) ? 1.f / L.z : 0.f), acc.w * ((L.w > 0.f) ? 1.f / L.w : 0.f)};
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        if (j0 + c < ncols) {
          const bf16 hv = __float2bfloat16_rn(val[c]);
          const size_t idx = (size_t)s_oidx[j0 + c] + my_t;
          a.o[idx] = hv;
          a.o[a.o_lo_off + idx] = __float2bfloat16_rn(val[c] - __bfloat162float(hv));
        }
      }
    }
  }
  TC_STAMP(14);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn kv_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// A K or V plane of one layer as [rows][Hkv * 128] bf16, boxes of 64 rows x 64 elements, 128-byte swizzle, zero
// fill beyond the last row.  Cached: the same planes recur every step.
bool kv_map(CUtensorMap *m, const void *plane, uint64_t rows, uint64_t width) {
  typedef std::tuple<const void *, uint64_t, uint64_t> Key;
  static std::map<Key, CUtensorMap> cache;
  const Key key(plane, rows, width);
  auto it = cache.find(key);
  if (it != cache.end()) { *m = it->second; return true; }
  if (!kv_encode_fn()) return false;
  const cuuint64_t dims[2] = {width, rows};
  const cuuint64_t strides[1] = {width * 2};
  const cuuint32_t box[2] = {64, 64};
  const cuuint32_t estr[2] = {1, 1};
  if (kv_encode_fn()(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(plane), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  if (cache.size() > 4096) cache.clear();
  cache[key] = *m;
  return true;
}

template <int NQ>
cudaError_t launch_nq(const CUtensorMap &tmK, const CUtensorMap &tmV, const AttnArgs &a, int qblocks, int qper, bool pdl,
                      cudaStream_t st) {
  constexpr int SMEM = TcLayout<NQ>::BYTES + 1024;      // + what aligning the base to 1024 bytes may take
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(tree_attn_tc_kernel<NQ>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(a.splits, a.Hkv, a.rw.n_seq * qblocks);
  cfg.blockDim = dim3(kTcThreads);
  cfg.dynamicSmemBytes = SMEM;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = a.splits; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, tree_attn_tc_kernel<NQ>, tmK, tmV, a, qper, pdl ? 1 : 0);
}

}  // namespace

#ifdef FIRP_ATTN_TRACE
extern "C" int firp_debug_attn_trace(unsigned long long *out) {
  return (int)cudaMemcpyFromSymbol(out, g_attn_trace, sizeof(unsigned long long) * 16);
}
#endif

void attention_tc_blocks(int qrows, int *qblocks, int *qper) {
  *qblocks = (qrows + kAttnTcMaxCols - 1) / kAttnTcMaxCols;
  *qper = (qrows + *qblocks - 1) / *qblocks;
}

int attention_tc_splits(int groups, int kv_tiles, int sm_count) {
  // one CTA per SM, two tiles in flight per CTA (one per tile group): rounds x (the longest split's tiles per tile
  // group at ~2.8 us each + the fixed cost of a CTA, + the cluster barriers when there is more than one split)
  int best = 1;
  float best_cost = 1e30f;
  for (int s = 1; s <= kAttnMaxSplits && s <= (kv_tiles > 0 ? kv_tiles : 1); ++s) {
    const int rounds = (s * groups + sm_count - 1) / sm_count;
    const int per = (kv_tiles + s - 1) / s;
    const float cost = (float)rounds * (2.8f * (float)((per + 1) / 2) + 8.f + (s > 1 ? 1.5f : 0.f));
    if (cost < best_cost - 1e-6f) { best_cost = cost; best = s; }
  }
  return best;
}

cudaError_t launch_attention_tc(const AttnArgs &a, bool pdl, cudaStream_t st) {
  if (a.dh != kTcDh) return cudaErrorInvalidValue;
  const int G = a.H / a.Hkv;
  int qblocks, qper;
  attention_tc_blocks(a.rows_active * G, &qblocks, &qper);
  const uint64_t width = (uint64_t)a.Hkv * kTcDh, rows = a.kv_stride / width;
  CUtensorMap tmK, tmV;
  if (!kv_map(&tmK, a.kcache, rows, width) || !kv_map(&tmV, a.kcache + a.kv_stride, rows, width)) return cudaErrorInvalidValue;
  if (qper <= 16) return launch_nq<16>(tmK, tmV, a, qblocks, qper, pdl, st);
  if (qper <= 32) return launch_nq<32>(tmK, tmV, a, qblocks, qper, pdl, st);
  return launch_nq<48>(tmK, tmV, a, qblocks, qper, pdl, st);
}

}  // namespace firp
