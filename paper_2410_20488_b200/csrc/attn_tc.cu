// Tree-masked split-KV decode attention on the tcgen05 tensor cores (Section 3.4 "Tree attention"; Section 3.3
// for the pseudo rows), head dimension 128.
//
// Roles are swapped as in the GEMMs: a tile of 128 cached positions is the MMA's M dimension, the query rows of
// the block (tree rows x heads of the group, <= 80) its N dimension.
//   S^T = K Q^T      K tile [128 pos][128 dh] K-major (TMA, 128-byte swizzle), Q [NQ][128] K-major (hi and lo
//                    bf16 planes, both accumulated into the same fp32 columns)           -> TMEM columns [0, NQ)
//   softmax          thread i owns position i of the tile (= TMEM lane i): scale, visibility, column maxima over
//                    the 128 positions (warp reduction + shared memory), P = 2^(s - m) as bf16 (hi, lo) planes
//                    written to shared memory as [NQ][128 pos] K-major
//   O^T = V^T P^T    V tile [128 pos][128 dh] as the MN-major A operand (M = dh)         -> TMEM columns [NQ, 2NQ)
//   l^T = 1 P^T      an all-ones A tile: every lane receives the column sums of P        -> TMEM columns [2NQ, 3NQ)
// The running (max, sum, O) of the online softmax live in shared memory / registers: thread i keeps O^T[i][*]
// (dh index i, all query columns), rescaled per column when the maximum moves.  K and V tiles are double
// buffered.  Grid = (kv split, kv head, sequence x query block), the splits of one (kv head, query block) form a
// cluster and merge their partial results through distributed shared memory exactly like the mma.sync kernel.
// One CTA per SM (shared memory), so the 256 TMEM columns it allocates are never contended.  Every mbarrier wait
// is bounded; a wait that runs out sets the status word and the kernel runs to its end.
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
constexpr int kTcThreads = 128;
constexpr int kTcSlab = kTcTile * 128;      // bytes of one [128 rows][64 elements] slab
constexpr int kTcStage = 2 * kTcSlab;       // a K or V tile: two slabs (dh halves)
constexpr int kTcTmemCols = 256;

template <int NQ> struct TcLayout {
  static constexpr int Q_SLAB = NQ * 128;                 // [NQ rows][64 elements]
  static constexpr int K_OFF = 0;                         // [2 stages][2 dh halves][128 pos][128 B]
  static constexpr int V_OFF = K_OFF + 2 * kTcStage;      // [2 stages][2 dh halves][128 pos][128 B]
  static constexpr int ONES_OFF = V_OFF + 2 * kTcStage;   // [128 rows][16 elements], unswizzled
  static constexpr int Q_OFF = ONES_OFF + 4096;           // [2 planes][2 dh halves][NQ][128 B]
  static constexpr int P_OFF = Q_OFF + 4 * Q_SLAB;        // [2 planes][2 pos halves][NQ][128 B]
  static constexpr int BYTES = P_OFF + 4 * Q_SLAB;
  static_assert(NQ % 16 == 0 && NQ >= 16 && 3 * NQ <= kTcTmemCols, "query columns per block");
  static_assert((NQ + 8) * kTcDh * 4 <= 2 * kTcStage, "a partial O^T must fit the key stages");
  static_assert(BYTES + 1024 + 4096 <= 227 * 1024, "shared memory budget (dynamic + alignment + static)");
};

// MN-major operand, 128-byte swizzle: 64 elements of M contiguous (128 bytes), the 8 rows of a K group 128 bytes
// apart, K groups `1024` bytes apart (stride offset), 64-element M blocks lbo_bytes apart (leading offset).
__device__ __forceinline__ uint64_t smem_desc_mn(uint32_t addr, uint32_t lbo_bytes) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// order-preserving map float <-> int (its own inverse)
__device__ __forceinline__ int f2ord(float f) { int b = __float_as_int(f); return b ^ ((b >> 31) & 0x7fffffff); }
__device__ __forceinline__ float ord2f(int b) { return __int_as_float(b ^ ((b >> 31) & 0x7fffffff)); }

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
  __shared__ __align__(16) int s_red[NQ][4];        // per column: the four warps' maxima of the tile (order-mapped)
  __shared__ __align__(16) float s_m[NQ];           // running max (log2 units)
  __shared__ __align__(16) float s_corr[NQ];        // 2^(old max - new max) of the current tile
  __shared__ __align__(16) float s_l[NQ];           // running sum
  __shared__ float s_pm[NQ + kAttnMaxSplits], s_pl[NQ + kAttnMaxSplits];   // (max, sum) received for the merge: [split][slot]
  __shared__ __align__(8) uint64_t s_bar[6];        // K landed [2], V landed [2], S^T complete, O^T and l^T complete
  __shared__ uint32_t s_tmem;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  TC_STAMP(0);
  uint8_t *base = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t sb = smem_u32(base);
  const uint32_t bar0 = smem_u32(s_bar), bar_s = bar0 + 32, bar_o = bar0 + 40;

  if (tid == 0) {
    for (int i = 0; i < 6; ++i) mbar_init(bar0 + 8 * i, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  {  // the all-ones A tile: [128 rows][16 elements], unswizzled 8 x 16-byte core matrices (4 KB)
    const uint4 ones = make_uint4(0x3F803F80u, 0x3F803F80u, 0x3F803F80u, 0x3F803F80u);
    uint4 *o = reinterpret_cast<uint4 *>(base + LY::ONES_OFF);
    o[tid] = ones; o[tid + kTcThreads] = ones;
  }
  for (int j = tid; j < NQ; j += kTcThreads) { s_m[j] = -INFINITY; s_l[j] = 0.f; }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(kTcTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
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
  const int kv_len = min(n + a.rows_active, a.max_ctx);
  const int tiles_total = (kv_len + kTcTile - 1) / kTcTile;
  const int t0 = (split * tiles_total + nsplits - 1) / nsplits, t1 = ((split + 1) * tiles_total + nsplits - 1) / nsplits;
  const unsigned long long wait_ns = a.wait_ns ? a.wait_ns : kDefaultWaitNs;
  bool dead = false;

  uint64_t pol = 0;
  auto load_tile = [&](int st, int t) {             // thread 0: K and V of tile t as 64-position x 64-element boxes
    mbar_expect_tx(bar0 + 8 * st, kTcStage);
    mbar_expect_tx(bar0 + 16 + 8 * st, kTcStage);
#pragma unroll
    for (int ph = 0; ph < 2; ++ph) {
      const int p0 = t * kTcTile + ph * 64;
      const int row = (int)kv_row(a.pages, slot, p0 < kv_len ? p0 : 0, a.max_ctx);   // a half beyond the context: any rows
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const uint32_t off = (uint32_t)(st * kTcStage + h * kTcSlab + ph * 8192);
        tma_load_2d(sb + LY::K_OFF + off, &tmK, kvh * kTcDh + h * 64, row, bar0 + 8 * st, pol);
        tma_load_2d(sb + LY::V_OFF + off, &tmV, kvh * kTcDh + h * 64, row, bar0 + 16 + 8 * st, pol);
      }
    }
  };
  if (tid == 0) {
    asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(pol));
    if (t0 < t1) load_tile(0, t0);
    if (t0 + 1 < t1) load_tile(1, t0 + 1);
  }
  // queries of this block: column j = query row q0 + j -> (tree row (q0 + j) / G, head kvh G + (q0 + j) % G)
  {
    constexpr int IT = NQ * 16 / kTcThreads;          // 16-byte chunks per thread and plane
    uint4 qh[IT], ql[IT];
#pragma unroll
    for (int it = 0; it < IT; ++it) {                 // all loads in flight before the first store
      const int idx = it * kTcThreads + tid, j = idx >> 4, c = idx & 15, qr = q0 + j;
      qh[it] = make_uint4(0u, 0u, 0u, 0u); ql[it] = qh[it];
      if (j < ncols) {
        const bf16 *src = a.q + ((size_t)(s * a.rw.Ms + qr / G) * a.H + kvh * G + qr % G) * kTcDh + c * 8;
        qh[it] = *reinterpret_cast<const uint4 *>(src);
        ql[it] = *reinterpret_cast<const uint4 *>(src + a.q_lo_off);
      }
    }
#pragma unroll
    for (int it = 0; it < IT; ++it) {
      const int idx = it * kTcThreads + tid, j = idx >> 4, c = idx & 15;
      const int off = (c >> 3) * LY::Q_SLAB + j * 128 + (((c & 7) ^ (j & 7)) << 4);
      *reinterpret_cast<uint4 *>(base + LY::Q_OFF + off) = qh[it];
      *reinterpret_cast<uint4 *>(base + LY::Q_OFF + 2 * LY::Q_SLAB + off) = ql[it];
    }
  }
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  TC_STAMP(2);
  const uint32_t tmem = s_tmem;
  const uint32_t tlane = tmem + ((uint32_t)(warp * 32) << 16);

  const uint32_t idesc_k = instr_desc_m128(NQ), idesc_mn = idesc_k | (1u << 15);
  const uint64_t ones_desc = (uint64_t)(((sb + LY::ONES_OFF) & 0x3FFFFu) >> 4) | ((uint64_t)(128 >> 4) << 16) |
                             ((uint64_t)(256 >> 4) << 32) | ((uint64_t)1 << 46);
  // operand descriptors of stage 0; another stage, dh half or k step only moves the start address (16-byte units)
  const uint64_t kdesc0 = smem_desc(sb + LY::K_OFF), qdesc0 = smem_desc(sb + LY::Q_OFF);
  const uint64_t vdesc0 = smem_desc_mn(sb + LY::V_OFF, kTcSlab), pdesc0 = smem_desc(sb + LY::P_OFF);
  auto issue_s = [&](int st) {                      // thread 0: S^T = K Q^T
    uint32_t acc = 0;
    for (int pl = 0; pl < a.q_planes; ++pl)
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) {
        tc_mma(tmem, kdesc0 + (uint64_t)((st * kTcStage + (kk >> 2) * kTcSlab + (kk & 3) * 32) >> 4),
               qdesc0 + (uint64_t)((pl * 2 * LY::Q_SLAB + (kk >> 2) * LY::Q_SLAB + (kk & 3) * 32) >> 4), idesc_k, acc);
        acc = 1;
      }
    tc_commit(bar_s);
  };
  auto issue_o = [&](int st) {                      // thread 0: O^T = V^T P^T and l^T = 1 P^T
    uint32_t acc = 0;
    for (int pl = 0; pl < a.p_planes; ++pl)
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const uint64_t bdesc = pdesc0 + (uint64_t)((pl * 2 * LY::Q_SLAB + (ks >> 2) * LY::Q_SLAB + (ks & 3) * 32) >> 4);
        tc_mma(tmem + NQ, vdesc0 + (uint64_t)((st * kTcStage + ks * 2048) >> 4), bdesc, idesc_mn, acc);
        tc_mma(tmem + 2 * NQ, ones_desc, bdesc, idesc_k, acc);
        acc = 1;
      }
    tc_commit(bar_o);
  };

  float o_acc[NQ];
#pragma unroll
  for (int j = 0; j < NQ; ++j) o_acc[j] = 0.f;
  const float scale_log2 = rsqrtf((float)kTcDh) * 1.4426950408889634f;
  // where this thread's position goes in a P row: 64-position half, 16-byte chunk, element
  const int p_half = tid >> 6, p_chunk = (tid & 63) >> 3, p_el2 = tid & 6, odd = tid & 1;

  if (tid == 0 && t0 < t1) {
    mbar_wait(bar0, 0, a.err, dead, wait_ns);
    tc_fence_after();
    issue_s(0);
  }
  for (int t = t0; t < t1; ++t) {
    const int i = t - t0, st = i & 1;
    const int p = t * kTcTile + tid;
    const bool pvalid = p < kv_len;
    // visibility of position p for every query column: the committed prefix is visible to all, new row u = p - n
    // to the rows whose mask has bit u
    uint32_t vis[(NQ + 31) / 32];
#pragma unroll
    for (int w = 0; w < (NQ + 31) / 32; ++w) vis[w] = pvalid ? ~0u : 0u;
    if (pvalid && p >= n) {
      const int u = p - n, w = u >> 5, b = u & 31;
#pragma unroll
      for (int w2 = 0; w2 < (NQ + 31) / 32; ++w2) vis[w2] = 0u;
#pragma unroll
      for (int j = 0; j < NQ; ++j) {
        const int qr = min(q0 + j, qrows_total - 1);
        const uint32_t word = a.mask[(size_t)(s * a.rw.Ms + qr / G) * kMaskWords + w];
        vis[j >> 5] |= ((word >> b) & 1u) << (j & 31);
      }
    }
    __syncwarp();
    mbar_wait(bar_s, i & 1, a.err, dead, wait_ns);
    tc_fence_after();
    if (i == 0) TC_STAMP(3);
    // pass 1: column maxima over the tile's positions
#pragma unroll
    for (int c0 = 0; c0 < NQ; c0 += 16) {
      float r[16];
      tc_ld16(tlane + c0, r);
      tc_ld_wait();
      int mine = 0;
#pragma unroll
      for (int jj = 0; jj < 16; ++jj) {
        const int j = c0 + jj;
        const float v = ((vis[j >> 5] >> (j & 31)) & 1u) ? r[jj] * scale_log2 : -INFINITY;
        const int o = __reduce_max_sync(0xffffffffu, f2ord(v));
        if (lane == jj) mine = o;
      }
      if (lane < 16) s_red[c0 + lane][warp] = mine;
    }
    __syncthreads();
    if (i == 0) TC_STAMP(4);
    if (tid < NQ) {
      const int4 v = *reinterpret_cast<const int4 *>(s_red[tid]);
      const float mt = ord2f(max(max(v.x, v.y), max(v.z, v.w)));
      const float m_old = s_m[tid], m_new = fmaxf(m_old, mt);
      s_corr[tid] = exp2f(m_old - (m_new == -INFINITY ? 0.f : m_new));
      s_m[tid] = m_new;
    }
    __syncthreads();
    if (i == 0) TC_STAMP(5);
    // pass 2: P = 2^(s - m) as bf16 (hi, lo) into the B operand of the second contraction.  Lanes 2i and 2i + 1
    // hold neighbouring positions: they swap one column of each column pair, so that every lane converts and
    // stores two neighbouring positions of one column as one 32-bit word.
#pragma unroll
    for (int c0 = 0; c0 < NQ; c0 += 16) {
      float r[16], ms[16];
      tc_ld16(tlane + c0, r);
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        const float4 m4 = *reinterpret_cast<const float4 *>(&s_m[c0 + 4 * q4]);
        ms[4 * q4] = m4.x; ms[4 * q4 + 1] = m4.y; ms[4 * q4 + 2] = m4.z; ms[4 * q4 + 3] = m4.w;
      }
      tc_ld_wait();
#pragma unroll
      for (int jj = 0; jj < 16; ++jj) {
        const int j = c0 + jj;
        const float msafe = (ms[jj] == -INFINITY) ? 0.f : ms[jj];
        r[jj] = ((vis[j >> 5] >> (j & 31)) & 1u) ? exp2f(r[jj] * scale_log2 - msafe) : 0.f;
      }
#pragma unroll
      for (int jj = 0; jj < 16; jj += 2) {
        const float got = __shfl_xor_sync(0xffffffffu, odd ? r[jj] : r[jj + 1], 1);
        const float x = odd ? got : r[jj], y = odd ? r[jj + 1] : got;      // positions 2i, 2i + 1 of column jj + odd
        const __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
        const float2 hf = __bfloat1622float2(h);
        const __nv_bfloat162 l = __floats2bfloat162_rn(x - hf.x, y - hf.y);
        const int j = c0 + jj + odd;
        const int off = p_half * LY::Q_SLAB + j * 128 + ((p_chunk ^ (j & 7)) << 4) + p_el2 * 2;
        *reinterpret_cast<__nv_bfloat162 *>(base + LY::P_OFF + off) = h;
        *reinterpret_cast<__nv_bfloat162 *>(base + LY::P_OFF + 2 * LY::Q_SLAB + off) = l;
      }
    }
    if (!pvalid) {       // a position beyond the context: its V row may hold anything, and 0 x NaN is NaN
      mbar_wait(bar0 + 16 + 8 * st, (i >> 1) & 1, a.err, dead, wait_ns);
      uint4 *v0 = reinterpret_cast<uint4 *>(base + LY::V_OFF + st * kTcStage + tid * 128);
      uint4 *v1 = reinterpret_cast<uint4 *>(base + LY::V_OFF + st * kTcStage + kTcSlab + tid * 128);
#pragma unroll
      for (int c = 0; c < 8; ++c) { v0[c] = make_uint4(0u, 0u, 0u, 0u); v1[c] = make_uint4(0u, 0u, 0u, 0u); }
    }
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    if (i == 0) TC_STAMP(6);
    if (tid == 0) {
      tc_fence_after();
      mbar_wait(bar0 + 16 + 8 * st, (i >> 1) & 1, a.err, dead, wait_ns);
      issue_o(st);
      if (t + 1 < t1) {
        mbar_wait(bar0 + 8 * (st ^ 1), ((i + 1) >> 1) & 1, a.err, dead, wait_ns);
        issue_s(st ^ 1);
      }
    }
    __syncwarp();
    mbar_wait(bar_o, i & 1, a.err, dead, wait_ns);
    tc_fence_after();
    if (i == 0) TC_STAMP(7);
    if (tid == 0 && t + 2 < t1) load_tile(st, t + 2);       // both tiles of this stage have been consumed
    __syncwarp();
    // O^T of the tile joins the running one; the column sums go to the columns' owners
#pragma unroll
    for (int c0 = 0; c0 < NQ; c0 += 16) {
      float r[16];
      tc_ld16(tlane + NQ + c0, r);
      tc_ld_wait();
#pragma unroll
      for (int jj = 0; jj < 16; ++jj) o_acc[c0 + jj] = o_acc[c0 + jj] * s_corr[c0 + jj] + r[jj];
      if (warp == ((c0 >> 4) & 3)) {
        float ls[16];
        tc_ld16(tlane + 2 * NQ + c0, ls);
        tc_ld_wait();
        float pick = 0.f;
#pragma unroll
        for (int jj = 0; jj < 16; ++jj) if (lane == jj) pick = ls[jj];
        if (lane < 16) s_l[c0 + lane] = s_l[c0 + lane] * s_corr[c0 + lane] + pick;
      }
    }
    if (i == 0) TC_STAMP(8);
  }
  TC_STAMP(9);
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTcTmemCols) : "memory");
  }
  // merge: o = sum_s 2^(m_s - M) O_s / sum_s 2^(m_s - M) l_s.  Column j is finalised by CTA j % splits: once every
  // CTA of the cluster has left its tile loop (its stages are free), each pushes its partial (m, l, O^T column)
  // into the owner's shared memory with plain remote stores; after a second cluster barrier the owners merge
  // what they received, in split order, from their own shared memory.
  cg::cluster_group cluster = cg::this_cluster();
  TC_STAMP(10);
  cluster.sync();
  TC_STAMP(11);
  const int rank = (int)cluster.block_rank(), nsp = (int)cluster.num_blocks();
  const int slots = (NQ + nsp - 1) / nsp;                       // columns an owner may receive from one split
  float *sM = reinterpret_cast<float *>(base + LY::K_OFF);      // [splits][slots][128] floats (<= (NQ + 8) x 512 B)
  {
    int owner = 0, slot = 0;
#pragma unroll
    for (int j = 0; j < NQ; ++j) {
      if (j < ncols) cluster.map_shared_rank(sM, owner)[(size_t)(rank * slots + slot) * kTcDh + tid] = o_acc[j];
      if (++owner == nsp) { owner = 0; ++slot; }
    }
    if (tid < ncols) {
      const int ow = tid % nsp, sl = tid / nsp;
      cluster.map_shared_rank(s_pm, ow)[rank * slots + sl] = s_m[tid];
      cluster.map_shared_rank(s_pl, ow)[rank * slots + sl] = s_l[tid];
    }
  }
  TC_STAMP(12);
  cluster.sync();
  TC_STAMP(13);
  constexpr int TPR = kTcDh / 4, RP = kTcThreads / TPR;      // threads per column, columns per pass
  const int c4 = (tid % TPR) * 4, sub = tid / TPR;
  for (int slot = sub; rank + slot * nsp < ncols; slot += RP) {
    const int j = rank + slot * nsp;
    float M = -INFINITY;
    for (int sp = 0; sp < nsp; ++sp) M = fmaxf(M, s_pm[sp * slots + slot]);
    float L = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int sp = 0; sp < nsp; ++sp) {
      const float pm = s_pm[sp * slots + slot];
      if (pm != -INFINITY) {
        const float w = exp2f(pm - M);
        const float4 ov = *reinterpret_cast<const float4 *>(sM + (size_t)(sp * slots + slot) * kTcDh + c4);
        L += w * s_pl[sp * slots + slot];
        acc.x += w * ov.x; acc.y += w * ov.y; acc.z += w * ov.z; acc.w += w * ov.w;
      }
    }
    const float inv = (L > 0.f) ? 1.f / L : 0.f;
    const float val[4] = {acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv};
    const int qr = q0 + j;
    const int r = s * a.rw.Ms + qr / G, head = kvh * G + qr % G;
    const __nv_bfloat162 h01 = __floats2bfloat162_rn(val[0], val[1]), h23 = __floats2bfloat162_rn(val[2], val[3]);
    const float2 f01 = __bfloat1622float2(h01), f23 = __bfloat1622float2(h23);
    const __nv_bfloat162 l01 = __floats2bfloat162_rn(val[0] - f01.x, val[1] - f01.y);
    const __nv_bfloat162 l23 = __floats2bfloat162_rn(val[2] - f23.x, val[3] - f23.y);
    const size_t idx = ((size_t)r * a.H + head) * kTcDh + c4;
    *reinterpret_cast<uint2 *>(a.o + idx) =
        make_uint2(*reinterpret_cast<const uint32_t *>(&h01), *reinterpret_cast<const uint32_t *>(&h23));
    *reinterpret_cast<uint2 *>(a.o + a.o_lo_off + idx) =
        make_uint2(*reinterpret_cast<const uint32_t *>(&l01), *reinterpret_cast<const uint32_t *>(&l23));
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
  // one CTA per SM: the fewest rounds of the longest split's tiles (+ ~2 tiles' worth of fixed cost per round)
  int best = 1;
  float best_cost = 1e30f;
  for (int s = 1; s <= kAttnMaxSplits && s <= (kv_tiles > 0 ? kv_tiles : 1); ++s) {
    const int rounds = (s * groups + sm_count - 1) / sm_count;
    const float cost = (float)rounds * ((float)((kv_tiles + s - 1) / s) + 2.f);
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
  if (qper <= 48) return launch_nq<48>(tmK, tmV, a, qblocks, qper, pdl, st);
  return launch_nq<80>(tmK, tmV, a, qblocks, qper, pdl, st);
}

}  // namespace firp
