// The decoder layers of one FIRP step (Section 3.2-3.4) as ONE persistent kernel: every GEMM, the residual /
// RMSNorm passes, the rotary / SwiGLU / logits finishers, Eq. 3 and the tree attention run as phases of a
// single cooperative launch with one CTA per SM.
//
// Why: the step is a weight stream (13.3 GB per step at the 7B shape against ~0.3 GB of everything else).
// With one kernel per operation every boundary drains the shared-memory pipeline of the GEMM before it and
// refills the one after it, and HBM idles meanwhile.  Here the weight producer of a CTA never stops: it walks
// the GEMMs of the whole step in order and keeps the shared-memory ring full across phase boundaries, so while
// the CTAs synchronise, normalise, rotate or attend, the first tiles of the next matrix are already on chip.
// (Measured on B200: reading through L2 is not faster than reading HBM for this access pattern, so prefetching
// into L2 buys nothing; the ring is the only buffer that hides a dependency.)
//
// Per CTA, 11 warps:
//   warp 0     weight producer: TMA (128-byte swizzle) into a ring of 32 KB stages; depends on nothing
//   warp 6     activation producer: the (hi, lo) bf16 planes of the k block, after the phase's inputs are complete
//              (signalled by the workers through a shared-memory barrier)
//   warp 1     MMA issuer: tcgen05.mma kind::f16, accumulators in TMEM; roles swapped as in the stand-alone GEMM
//              (weight rows = MMA M, token rows = MMA N, the planes side by side as one N)
//   warps 2-5, 7-10  workers: TMEM -> partial tiles (stream-K; one group of four warps per weight tile of the
//              supertile), then every non-GEMM phase: the elementwise passes are spread over all CTAs, the attention
//              runs one (kv head, query block, kv split) item per CTA at a time on warps 2-5, in the shared memory
//              the activation ring does not need meanwhile
// Phases are separated by a grid-wide barrier (an arrival counter in global memory; every wait is bounded and
// reports through the status word).  Partial tiles are summed in ascending CTA order, the attention splits in
// ascending split order: results are identical from run to run.
#include <cuda.h>

#include <cstring>
#include <map>
#include <vector>

#include "attn_device.cuh"
#include "finish_device.cuh"
#include "firp_kernels.cuh"
#include "launch_util.cuh"
#include "norm_device.cuh"
#include "tc_device.cuh"

namespace firp {

namespace {

constexpr int BM = 128, TM = 2, BK = kGemmBK;
constexpr int W_TILE = BM * 128, W_STAGE = TM * W_TILE;   // one unit: 2 x 128 weight rows x 64 k = 32 KB
constexpr int kFThreads = 352;                            // 11 warps: 3 single-thread roles + 8 worker warps
constexpr int kWorkers = 256;
constexpr int SW = 4;                                     // weight stages (128 KB in flight per SM; a fifth changed nothing)
constexpr int SX = 4;                                     // activation stages
constexpr int kRegion = 96 * 1024;                        // activation ring, reused by the attention phases
constexpr int kSmallBytes = kAttnQRows * kMaskWords * 4 + kAttnQRows * 4;   // s_mask, s_row
constexpr int kBarBytes = 256;
constexpr int kFusedSmem = SW * W_STAGE + kRegion + kSmallBytes + kBarBytes;
static_assert(kFusedSmem <= 227 * 1024, "shared memory budget");
static_assert(attn_smem_bytes<128>() <= kRegion, "attention tiles must fit the activation ring's region");
constexpr int kMaxClasses = 16;
constexpr int kMaxFusedGemms = 512;
constexpr int kMaxFusedOps = 1000;
constexpr int kMaxSplitsFused = 16;

enum FusedOpType : uint8_t { OP_NORM = 0, OP_ROOT_SPLIT, OP_GEMM, OP_FINISH, OP_ATTN, OP_MERGE };
enum RowMode { ROWS_LINEAR = 0, ROWS_GATE_UP = 1, ROWS_ROTARY = 2 };

struct GemmClass {
  int mode, F, half;   // how a supertile maps to weight rows
  int U, KB, G;        // stream-K schedule: CTAs 0..G-1 share the units (G = min(grid, U)), the others have none
  int P;               // activation planes
  int xmap;            // tensor map of the activations
  int N, K;
  int epi;             // GemmEpilogue of its finisher
};

struct FusedOp {
  uint8_t type, cls, planes, pad;   // cls: GEMM class (OP_GEMM / OP_FINISH); planes: OP_NORM output planes, OP_FINISH(pseudo): 1 = pre-norm variant
  int16_t layer;                    // decoder layer (cache plane of the finisher / attention), -1: none
  int16_t v0, nv;                   // OP_NORM: rows [v0, v0 + nv) of every sequence
  int16_t act;                      // rows alive in this layer
  int16_t aux;                      // OP_NORM: class whose partial tiles are pending (-1 none); OP_FINISH(pseudo): first prediction step
  const void *ptr;                  // OP_NORM: gain vector; OP_FINISH(pseudo): bias or NULL
};

struct FusedParams {
  Rows rw;
  int d, H, Hkv, dh, F, V, Rp, max_ctx, splits;
  float eps;
  float *h, *ws, *ss, *logits, *attn_ws;
  bf16 *x, *xp, *q, *o, *y, *kv;
  size_t kv_seq, kv_layer, kv_plane;
  KvPages pages;
  const float2 *rope; const int32_t *pos, *seq_ids, *ctx_len; const uint32_t *mask;
  int *err; unsigned *bar; unsigned long long wait_ns;
  const CUtensorMap *maps;
  int n_gemm, n_ops, n_cls;
  GemmClass cls[kMaxClasses];
  uint16_t gemm_cls[kMaxFusedGemms], gemm_map[kMaxFusedGemms];
  FusedOp ops[kMaxFusedOps];
};
static_assert(sizeof(FusedParams) <= 32000, "kernel parameter space");

#ifdef FIRP_TRACE     // development aid, not part of the product build: per-CTA time stamps of every phase
__device__ unsigned long long *g_trace = nullptr;
#define FIRP_STAMP(slot) do { if (wtid == 0 && g_trace) g_trace[((size_t)cta * kMaxFusedOps + oi) * 2 + (slot)] = globaltimer(); } while (0)
#else
#define FIRP_STAMP(slot) do { } while (0)
#endif

struct WorkerSync { static __device__ __forceinline__ void sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); } };      // all 8 worker warps
struct AttnGroupSync { static __device__ __forceinline__ void sync() { asm volatile("bar.sync 3, 128;" ::: "memory"); } };   // warps 2..5

__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }

// Grid-wide barrier of the worker warps (256 threads per CTA).  Monotonic arrival counter; `epoch` counts the
// barriers passed.  The wait is bounded: on expiry the status word is set and this thread stops waiting for good.
__device__ __forceinline__ void grid_sync(unsigned *ctr, unsigned &epoch, int wtid, int *err, bool &dead,
                                          unsigned long long wait_ns, bool tma_reads_follow) {
  if (tma_reads_follow) fence_proxy_async();   // what this thread wrote will be read by TMA loads of other CTAs
  WorkerSync::sync();
  ++epoch;
  if (wtid == 0 && !dead) {
    const unsigned target = epoch * gridDim.x;
    // release at gpu scope, cumulative: it also orders what the other workers wrote before the block barrier
    asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(ctr) : "memory");
    const unsigned long long t0 = globaltimer();
    uint32_t spins = 0;
    for (;;) {
      unsigned v;
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ctr) : "memory");
      if (v >= target) break;
      if ((++spins & 63u) == 0 && globaltimer() - t0 > wait_ns) {
        dead = true;
        atomicExch(err, kErrGridTimeout);
        break;
      }
    }
  }
  WorkerSync::sync();             // the acquire of thread 0 reaches the other workers through this barrier
}

template <int NPAD>
__global__ void __launch_bounds__(kFThreads, 1) fused_layers_kernel(const __grid_constant__ FusedParams P) {
  constexpr int X_PLANE = NPAD * 128;          // bytes of one activation plane of a stage
  constexpr int X_STAGE = 3 * X_PLANE;         // room for three planes, whatever the phase uses
  static_assert(SX * X_STAGE <= kRegion, "activation ring must fit its region");
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  const uint32_t w_ring = base, x_ring = base + SW * W_STAGE;
  uint8_t *region = smem_raw + SW * W_STAGE;
  uint32_t (*s_mask)[kMaskWords] = reinterpret_cast<uint32_t (*)[kMaskWords]>(region + kRegion);
  int *s_row = reinterpret_cast<int *>(region + kRegion + kAttnQRows * kMaskWords * 4);
  const uint32_t bars = x_ring + kRegion + kSmallBytes;
  const uint32_t full_w = bars, empty_w = full_w + 8 * SW, full_x = empty_w + 8 * SW, empty_x = full_x + 8 * SX,
                 acc_full = empty_x + 8 * SX, acc_empty = acc_full + 16, xgo = acc_empty + 16, tmem_slot = xgo + 8;
  volatile uint32_t *tmem_slot_ptr = reinterpret_cast<volatile uint32_t *>(smem_raw + (tmem_slot - base));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x, G = gridDim.x;
  const unsigned long long wait_ns = P.wait_ns ? P.wait_ns : kDefaultWaitNs;

  if ((base & 1023u) != 0) {       // swizzled tiles need 1024-byte alignment: refuse rather than compute garbage
    if (threadIdx.x == 0) atomicExch(P.err, kErrTimeout + 2);
    return;
  }
  if (threadIdx.x == 0) {
    for (int i = 0; i < SW; ++i) { mbar_init(full_w + 8 * i, 1); mbar_init(empty_w + 8 * i, 1); }
    for (int i = 0; i < SX; ++i) { mbar_init(full_x + 8 * i, 1); mbar_init(empty_x + 8 * i, 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(acc_full + 8 * i, 1); mbar_init(acc_empty + 8 * i, 8); }
    mbar_init(xgo, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  griddep_launch();
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_ptr;

  bool dead = false;
  if (warp == 0) {
    if (lane == 0) {             // ---- weight producer: all GEMMs of the step, back to back
      uint64_t pol;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
      int k = 0;
      for (int g = 0; g < P.n_gemm; ++g) {
        const GemmClass &c = P.cls[P.gemm_cls[g]];
        const CUtensorMap *tm = P.maps + P.gemm_map[g];
        const StreamK sk{c.U, c.KB, c.G};
        const int u0 = cta < c.G ? sk_begin(sk, cta) : 0, n_units = cta < c.G ? sk_begin(sk, cta + 1) - u0 : 0;
        for (int it = 0; it < n_units; ++it, ++k) {
          const int u = u0 + it;
          const int st = u / c.KB, kb = u - st * c.KB;
          const int sl = k % SW;
          mbar_wait(empty_w + 8 * sl, ((k / SW) & 1) ^ 1, P.err, dead, wait_ns);
          mbar_expect_tx(full_w + 8 * sl, W_STAGE);
          const uint32_t dst = w_ring + sl * W_STAGE, bar = full_w + 8 * sl;
          if (c.mode == ROWS_ROTARY) {
            const int hp = BM / c.half;               // heads per supertile
            tma_load_4d(dst, tm, kb * BK, 0, 0, st * hp, bar, pol);
            tma_load_4d(dst + W_TILE, tm, kb * BK, 0, 1, st * hp, bar, pol);
          } else if (c.mode == ROWS_GATE_UP) {
            tma_load_2d(dst, tm, kb * BK, st * BM, bar, pol);
            tma_load_2d(dst + W_TILE, tm, kb * BK, c.F + st * BM, bar, pol);
          } else {
            tma_load_2d(dst, tm, kb * BK, st * (TM * BM), bar, pol);
            tma_load_2d(dst + W_TILE, tm, kb * BK, st * (TM * BM) + BM, bar, pol);
          }
        }
      }
    }
  } else if (warp == 6) {
    if (lane == 0) {             // ---- activation producer
      uint64_t pol;
      asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
      const int xrows = min((P.rw.R + 7) & ~7, NPAD);
      int k = 0;
      for (int g = 0; g < P.n_gemm; ++g) {
        const GemmClass &c = P.cls[P.gemm_cls[g]];
        const CUtensorMap *tm = P.maps + c.xmap;
        const StreamK sk{c.U, c.KB, c.G};
        const int u0 = cta < c.G ? sk_begin(sk, cta) : 0, n_units = cta < c.G ? sk_begin(sk, cta + 1) - u0 : 0;
        mbar_wait(xgo, g & 1, P.err, dead, wait_ns);     // the workers have passed the barrier before this GEMM
        fence_proxy_async();
        for (int it = 0; it < n_units; ++it, ++k) {
          const int kb = (u0 + it) % c.KB;
          const int sl = k % SX;
          mbar_wait(empty_x + 8 * sl, ((k / SX) & 1) ^ 1, P.err, dead, wait_ns);
          mbar_expect_tx(full_x + 8 * sl, c.P * xrows * 128);
          const uint32_t dst = x_ring + sl * X_STAGE;
          for (int pl = 0; pl < c.P; ++pl)
            tma_load_2d(dst + pl * X_PLANE, tm, kb * BK, pl * P.Rp, full_x + 8 * sl, pol);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {             // ---- MMA issuer
      int kw = 0;
      unsigned use[2] = {0u, 0u};
      for (int g = 0; g < P.n_gemm; ++g) {
        const GemmClass &c = P.cls[P.gemm_cls[g]];
        const StreamK sk{c.U, c.KB, c.G};
        const int u0 = cta < c.G ? sk_begin(sk, cta) : 0, u1 = cta < c.G ? sk_begin(sk, cta + 1) : 0;
        const int ACC = c.P * NPAD;                       // accumulator columns per weight tile
        const int nbuf = (2 * TM * ACC <= 512) ? 2 : 1;
        const uint32_t idesc = instr_desc_m128(ACC);
        int seg = 0;
        int u = u0;
        while (u < u1) {
          const int st = u / c.KB, kb0 = u - st * c.KB;
          const int kb1 = min(c.KB, kb0 + (u1 - u));
          const int buf = seg % nbuf;
          mbar_wait(acc_empty + 8 * buf, (use[buf] & 1u) ^ 1u, P.err, dead, wait_ns);   // the workers have drained it
          tc_fence_after();
          const uint32_t acc = tmem_base + (uint32_t)(buf * TM * ACC);
          for (int kb = kb0; kb < kb1; ++kb, ++kw) {
            const int sw = kw % SW, sx = kw % SX;
            mbar_wait(full_w + 8 * sw, (kw / SW) & 1, P.err, dead, wait_ns);
            mbar_wait(full_x + 8 * sx, (kw / SX) & 1, P.err, dead, wait_ns);
            tc_fence_after();
            const uint32_t wst = w_ring + sw * W_STAGE, xst = x_ring + sx * X_STAGE;
            const uint64_t dx = smem_desc(xst);
#pragma unroll
            for (int kk = 0; kk < BK / 16; ++kk) {
#pragma unroll
              for (int t = 0; t < TM; ++t) {
                const uint64_t da = smem_desc(wst + t * W_TILE) + 2 * kk;
                tc_mma(acc + t * ACC, da, dx + 2 * kk, idesc, (kb > kb0 || kk > 0) ? 1u : 0u);
              }
            }
            tc_commit(empty_w + 8 * sw);
            tc_commit(empty_x + 8 * sx);
          }
          tc_commit(acc_full + 8 * buf);
          ++use[buf];
          u += kb1 - kb0;
          ++seg;
        }
      }
    }
  } else {                       // ---- workers: warps 2..5 (group A) and 7..10 (group B)
    const int wgroup = warp >= 7 ? 1 : 0;
    const int wtid = wgroup ? threadIdx.x - 224 + 128 : threadIdx.x - 64;   // 0..255
    const int quarter = warp & 3;                   // TMEM lane quarter this warp may read
    const int li = quarter * 32 + lane;             // row within each 128-row tile = TMEM lane
    const unsigned tbase = (unsigned)cta * (unsigned)kWorkers + (unsigned)wtid, tstride = (unsigned)G * (unsigned)kWorkers;
    unsigned epoch = 0;
    unsigned use[2] = {0u, 0u};
    const int nq = P.H * P.dh;
    const size_t plane_elems = (size_t)P.Rp * BM, slot_elems = TM * plane_elems;
    griddep_wait();                                  // tree bookkeeping and embeddings are complete
    if (P.n_ops > 0 && P.ops[0].type == OP_GEMM && wtid == 0) mbar_arrive(xgo);
    for (int oi = 0; oi < P.n_ops; ++oi) {
      const FusedOp &op = P.ops[oi];
      FIRP_STAMP(0);
      switch (op.type) {
        case OP_GEMM: {          // TMEM -> partial tiles of this CTA's segments
          const GemmClass &c = P.cls[op.cls];
          const StreamK sk{c.U, c.KB, c.G};
          const int u0 = cta < c.G ? sk_begin(sk, cta) : 0, u1 = cta < c.G ? sk_begin(sk, cta + 1) : 0;
          const int ACC = c.P * NPAD;
          const int nbuf = (2 * TM * ACC <= 512) ? 2 : 1;
          int seg = 0;
          int u = u0;
          while (u < u1) {
            const int st = u / c.KB, kb0 = u - st * c.KB;
            const int kb1 = min(c.KB, kb0 + (u1 - u));
            const int buf = seg % nbuf;
            mbar_wait(acc_full + 8 * buf, use[buf] & 1u, P.err, dead, wait_ns);
            tc_fence_after();
            // group A drains the first weight tile of the supertile, group B the second
            const uint32_t tacc = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * TM * ACC + wgroup * ACC);
            float *my_ws = P.ws + (size_t)(cta * kGemmSlots + seg) * slot_elems + (size_t)wgroup * plane_elems + li;
            for (int c0 = 0; c0 < P.rw.R && seg < kGemmSlots; c0 += 16) {
              float r0[16];
              tc_ld16(tacc + c0, r0);
              tc_ld_wait();
              for (int pl = 1; pl < c.P; ++pl) {      // columns pl * NPAD .. hold the sums over plane pl
                float l0[16];
                tc_ld16(tacc + pl * NPAD + c0, l0);
                tc_ld_wait();
#pragma unroll
                for (int j = 0; j < 16; ++j) r0[j] += l0[j];
              }
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                const int m = c0 + j;
                if (m < P.rw.R) __stcg(my_ws + (size_t)m * BM, r0[j]);
              }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty + 8 * buf);
            ++use[buf];
            u += kb1 - kb0;
            ++seg;
          }
          break;
        }
        case OP_NORM: {
          Partials pend{};
          pend.ws = P.ws; pend.ws_rows = P.Rp;
          if (op.aux >= 0) { const GemmClass &c = P.cls[op.aux]; pend.sk = StreamK{c.U, c.KB, c.G}; }
          const unsigned total = (unsigned)(P.rw.n_seq * op.nv * (P.d >> 2));
          for (unsigned t = tbase; t < total; t += tstride)
            rmsnorm_item(P.rw, op.v0, op.nv, P.h, pend, (const bf16 *)op.ptr, P.d, P.x, (size_t)P.Rp * P.d, op.planes, P.ss, t);
          break;
        }
        case OP_ROOT_SPLIT: {
          const unsigned total = (unsigned)(P.rw.n_seq * (P.rw.chains ? P.rw.T : 1) * (P.d >> 2));
          for (unsigned t = tbase; t < total; t += tstride) root_split_item(P.rw, P.h, (const bf16 *)op.ptr, P.d, P.xp, (size_t)P.Rp * P.d, t);
          break;
        }
        case OP_FINISH: {
          const GemmClass &c = P.cls[op.cls];
          Partials p{};
          p.sk = StreamK{c.U, c.KB, c.G}; p.ws = P.ws; p.ws_rows = P.Rp;
          GemmArgs a{};
          a.R = P.rw.R; a.rw = P.rw; a.rows_active = op.act; a.N = c.N; a.K = c.K; a.eps = P.eps;
          const int n_st = c.U / c.KB;
          if (c.epi == EPI_QKV_ROPE) {
            a.ss = P.ss; a.H = P.H; a.Hkv = P.Hkv; a.dh = P.dh; a.rope = P.rope; a.seq_ids = P.seq_ids; a.pos = P.pos;
            a.q = P.q; a.q_lo_off = (size_t)P.Rp * nq; a.kcache = P.kv + (size_t)op.layer * P.kv_layer;
            a.seq_stride = P.kv_seq; a.kv_stride = P.kv_plane; a.max_ctx = P.max_ctx; a.pages = P.pages;
          } else if (c.epi == EPI_SWIGLU) {
            a.ss = P.ss; a.y = P.y; a.y_lo_off = (size_t)P.Rp * P.F; a.F = P.F;
          } else if (c.epi == EPI_LOGITS) {
            a.ss = P.ss; a.logits = P.logits;
          } else {               // EPI_PSEUDO: one token row per source row of Eq. 3
            a.R = P.rw.n_seq * (P.rw.chains ? P.rw.T : 1);
            a.h_rows = P.h; a.pred_b = (const bf16 *)op.ptr; a.pseudo0 = op.aux;
            if (op.planes) a.ss = P.ss;      // pre-norm variant: divide by the source row's RMS
          }
          const unsigned total = (unsigned)(n_st * a.R * 32);
          for (unsigned t = tbase; t < total; t += tstride) {
            if (c.epi == EPI_QKV_ROPE) qkv_finish_item(p, a, n_st, t);
            else if (c.epi == EPI_SWIGLU) swiglu_finish_item(p, a, n_st, t);
            else if (c.epi == EPI_LOGITS) logits_finish_item(p, a, n_st, t);
            else pseudo_finish_item(p, a, n_st, t);
          }
          break;
        }
        case OP_ATTN: {          // one (sequence x query block, kv head, kv split) item at a time
          AttnArgs a{};
          a.rw = P.rw; a.rows_active = op.act; a.H = P.H; a.Hkv = P.Hkv; a.dh = P.dh;
          a.q = P.q; a.q_lo_off = (size_t)P.Rp * nq; a.kcache = P.kv + (size_t)op.layer * P.kv_layer;
          a.seq_stride = P.kv_seq; a.kv_stride = P.kv_plane; a.max_ctx = P.max_ctx; a.pages = P.pages;
          a.seq_ids = P.seq_ids; a.ctx_len = P.ctx_len; a.pos = P.pos; a.mask = P.mask; a.splits = P.splits;
          a.q_planes = 2; a.p_planes = 2;
          const int Gq = P.H / P.Hkv;
          const int qblocks = (op.act * Gq + kAttnQRows - 1) / kAttnQRows;
          const int n_items = P.rw.n_seq * qblocks * P.Hkv * P.splits;
          const size_t item_floats = (size_t)kAttnQRows * (P.dh + 2);
          for (int item = cta; item < n_items && wgroup == 0; item += G) {      // group A's four warps; group B waits at the barrier
            const int split = item % P.splits, rest = item / P.splits;
            const int kvh = rest % P.Hkv, z = rest / P.Hkv;
            float *out = P.attn_ws + (size_t)item * item_floats;
            if (P.dh == 128)
              attn_split_item<128, AttnGroupSync>(a, region, s_mask, s_row, wtid, z / qblocks, kvh, z % qblocks, split, P.splits,
                                               out, out + kAttnQRows, out + 2 * kAttnQRows);
            else
              attn_split_item<64, AttnGroupSync>(a, region, s_mask, s_row, wtid, z / qblocks, kvh, z % qblocks, split, P.splits,
                                              out, out + kAttnQRows, out + 2 * kAttnQRows);
          }
          break;
        }
        case OP_MERGE: {         // o = sum_s 2^(m_s - M) O_s / sum_s 2^(m_s - M) l_s, splits in ascending order
          const int Gq = P.H / P.Hkv, dh = P.dh, tpr = dh >> 2;
          const int qrows_total = op.act * Gq;
          const int qblocks = (qrows_total + kAttnQRows - 1) / kAttnQRows;
          const size_t item_floats = (size_t)kAttnQRows * (dh + 2);
          const unsigned total = (unsigned)(P.rw.n_seq * P.Hkv * qrows_total * tpr);
          for (unsigned t = tbase; t < total; t += tstride) {
            const int c4 = (int)(t % (unsigned)tpr) * 4;
            unsigned rest = t / (unsigned)tpr;
            const int qr = (int)(rest % (unsigned)qrows_total); rest /= (unsigned)qrows_total;
            const int kvh = (int)(rest % (unsigned)P.Hkv), s = (int)(rest / (unsigned)P.Hkv);
            const int qb = qr / kAttnQRows, i = qr % kAttnQRows;
            const float *it0 = P.attn_ws + (size_t)(((s * qblocks + qb) * P.Hkv + kvh) * P.splits) * item_floats;
            float M = -INFINITY;
            for (int sp = 0; sp < P.splits; ++sp) M = fmaxf(M, __ldcg(it0 + (size_t)sp * item_floats + i));
            float L = 0.f;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int sp = 0; sp < P.splits; ++sp) {
              const float *it = it0 + (size_t)sp * item_floats;
              const float pm = __ldcg(it + i);
              if (pm != -INFINITY) {
                const float w = exp2f(pm - M);
                const float4 ov = __ldcg(reinterpret_cast<const float4 *>(it + 2 * kAttnQRows + (size_t)i * dh + c4));
                L += w * __ldcg(it + kAttnQRows + i);
                acc.x += w * ov.x; acc.y += w * ov.y; acc.z += w * ov.z; acc.w += w * ov.w;
              }
            }
            const float inv = (L > 0.f) ? 1.f / L : 0.f;
            const float val[4] = {acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv};
            uint2 hi, lo;
            split4(val, hi, lo);
            const int r = s * P.rw.Ms + qr / Gq, head = kvh * Gq + qr % Gq;
            const size_t idx = ((size_t)r * P.H + head) * dh + c4;
            *reinterpret_cast<uint2 *>(P.o + idx) = hi;
            *reinterpret_cast<uint2 *>(P.o + (size_t)P.Rp * nq + idx) = lo;
          }
          break;
        }
        default: break;
      }
      FIRP_STAMP(1);
      if (oi + 1 == P.n_ops) break;      // nothing in this kernel reads what the last phase wrote
      const bool gemm_next = P.ops[oi + 1].type == OP_GEMM;
      grid_sync(P.bar, epoch, wtid, P.err, dead, wait_ns, gemm_next);
      if (gemm_next && wtid == 0) mbar_arrive(xgo);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}

// A wait that nothing will ever satisfy, with the same bounded-wait routine the product kernels use: one CTA
// initialises a shared-memory barrier nobody arrives on and waits for it.  The wait runs out after wait_ns, the
// status word is set and the kernel returns normally.
__global__ void wait_selftest_kernel(int *err, unsigned long long wait_ns) {
  __shared__ __align__(8) unsigned long long bar;
  const uint32_t b = smem_u32(&bar);
  if (threadIdx.x == 0) {
    mbar_init(b, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    bool dead = false;
    mbar_wait(b, 0, err, dead, wait_ns);
  }
}

// ---- host side ---------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn fused_encode_fn() {
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

// bf16 maps with 64-element inner boxes and 128-byte swizzle: 2-D [rows][K] (half == 0) or the 4-D view
// [rows / (2 half)][2][half][K] of a QKV weight whose box is the same rotary half of 128 / half heads
bool encode_map(CUtensorMap *m, const void *ptr, uint64_t rows, uint64_t K, uint32_t box_rows, uint32_t half) {
  CUresult rc;
  if (half == 0) {
    const cuuint64_t dims[2] = {K, rows};
    const cuuint64_t strides[1] = {K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)BK, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    rc = fused_encode_fn()(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else {
    const cuuint64_t dims[4] = {K, half, 2, rows / (2 * half)};
    const cuuint64_t strides[3] = {K * 2, (cuuint64_t)half * K * 2, (cuuint64_t)2 * half * K * 2};
    const cuuint32_t box[4] = {(cuuint32_t)BK, half, 1, (cuuint32_t)BM / half};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    rc = fused_encode_fn()(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(ptr), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }
  return rc == CUDA_SUCCESS;
}

int fused_sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 1;
  }
  return n;
}

GemmClass make_class(int epi, int N, int K, int P, int xmap, int F, int H, int Hkv, int dh, int grid = 0) {
  if (grid == 0) grid = fused_sm_count();
  GemmClass c{};
  c.epi = epi; c.N = N; c.K = K; c.P = P; c.xmap = xmap;
  c.mode = ROWS_LINEAR;
  int n_st = (N + TM * BM - 1) / (TM * BM);
  if (epi == EPI_SWIGLU) { c.mode = ROWS_GATE_UP; c.F = F; n_st = (F + BM - 1) / BM; }
  else if (epi == EPI_QKV_ROPE) { c.mode = ROWS_ROTARY; c.half = dh / 2; const int hp = BM / c.half; n_st = (H + 2 * Hkv + hp - 1) / hp; }
  c.KB = (K + BK - 1) / BK;
  c.U = n_st * c.KB;
  c.G = c.U < grid ? c.U : grid;
  return c;
}

// a CTA's range must touch at most kGemmSlots supertiles (one scratch slot each)
bool class_fits(const GemmClass &c, int) {
  const int per = (c.U + c.G - 1) / c.G;
  return (per + c.KB - 2) / c.KB + 1 <= kGemmSlots && (long long)(c.U + 1) * (c.G + 1) < (1ll << 31);
}

}  // namespace

struct FusedPlan {
  FusedParams prm{};
  std::vector<CUtensorMap> maps;
  // what the plan was built for
  Rows rw{}; int tl[8]{}; bool want_head = false; uint64_t weights_gen = 0; const void *bufs_key = nullptr;
  bool valid = false;
};

FusedPlan *fused_plan_create() { return new FusedPlan(); }
void fused_plan_destroy(FusedPlan *p) { delete p; }
size_t fused_map_bytes(int n_layers) { return sizeof(CUtensorMap) * (size_t)(4 * n_layers + 1 + 8 + 4 + 1); }   // rounded up to 256 bytes
size_t fused_attn_ws_floats(int max_batch, int H, int Hkv, int dh) {
  const int Gq = H / Hkv;
  const int groups = max_batch * Hkv * ((48 * Gq + kAttnQRows - 1) / kAttnQRows);
  const int items = groups > 320 ? groups : 320;
  return (size_t)items * kAttnQRows * (dh + 2);
}

cudaError_t launch_wait_selftest(int *err, unsigned long long wait_ns, cudaStream_t st) {
  wait_selftest_kernel<<<1, 32, 0, st>>>(err, wait_ns ? wait_ns : kDefaultWaitNs);
  return cudaGetLastError();
}

#ifdef FIRP_TRACE
extern "C" int firp_debug_set_trace(unsigned long long *buf) {
  return (int)cudaMemcpyToSymbol(g_trace, &buf, sizeof(buf));
}
extern "C" int firp_debug_max_ops() { return kMaxFusedOps; }
#endif

bool fused_eligible(const FusedShape &sh, const Rows &rw) {
  if (!fused_encode_fn()) return false;
  if (rw.R > 48 || rw.R < 1) return false;
  if (sh.dh != 64 && sh.dh != 128) return false;
  const int G = fused_sm_count();
  if (G > kGemmMaxCtas) return false;
  const int nq = sh.H * sh.dh;
  const GemmClass c[5] = {make_class(EPI_QKV_ROPE, (sh.H + 2 * sh.Hkv) * sh.dh, sh.d, 2, 0, sh.F, sh.H, sh.Hkv, sh.dh),
                          make_class(EPI_RESIDUAL, sh.d, nq, 2, 0, sh.F, sh.H, sh.Hkv, sh.dh),
                          make_class(EPI_SWIGLU, 2 * sh.F, sh.d, 2, 0, sh.F, sh.H, sh.Hkv, sh.dh),
                          make_class(EPI_RESIDUAL, sh.d, sh.F, 2, 0, sh.F, sh.H, sh.Hkv, sh.dh),
                          make_class(EPI_LOGITS, sh.V, sh.d, 2, 0, sh.F, sh.H, sh.Hkv, sh.dh)};
  for (const GemmClass &k : c) if (!class_fits(k, G)) return false;
  if (rw.kc > 0 && !class_fits(make_class(EPI_PSEUDO, sh.d, sh.d, 2, 0, sh.F, sh.H, sh.Hkv, sh.dh), G)) return false;
  const int ops = sh.L * 10 + rw.kc * 4 + 8;
  return ops <= kMaxFusedOps && sh.L * 4 + rw.kc + 1 <= kMaxFusedGemms;
}

cudaError_t launch_fused_layers(FusedPlan *plan, const FusedStep &fs, bool pdl, cudaStream_t st, int *launches) {
  const FusedShape &sh = fs.shape;
  const Rows &rw = fs.rw;
  const int G = fused_sm_count();
  const int L = sh.L, d = sh.d, H = sh.H, Hkv = sh.Hkv, dh = sh.dh, F = sh.F, nq = H * dh;
  const int NPAD = rw.R <= 16 ? 16 : 48;
  const bool same = plan->valid && memcmp(&plan->rw, &rw, sizeof(Rows)) == 0 && memcmp(plan->tl, fs.tl, sizeof(plan->tl)) == 0 &&
                    plan->want_head == fs.want_head && plan->weights_gen == fs.weights_gen && plan->bufs_key == (const void *)fs.d_maps;
  FusedParams &P = plan->prm;
  if (!same) {
    plan->valid = false;
    P = FusedParams{};
    P.rw = rw; P.d = d; P.H = H; P.Hkv = Hkv; P.dh = dh; P.F = F; P.V = sh.V; P.Rp = fs.Rp; P.max_ctx = sh.max_ctx; P.eps = sh.eps;
    P.h = fs.h; P.ws = fs.ws; P.ss = fs.ss; P.attn_ws = fs.attn_ws; P.x = fs.x; P.xp = fs.xp; P.q = fs.q; P.o = fs.o; P.y = fs.y;
    P.kv = fs.kv; P.kv_seq = fs.kv_seq; P.kv_layer = fs.kv_layer; P.kv_plane = fs.kv_plane; P.pages = fs.pages;
    P.rope = fs.rope; P.pos = fs.pos; P.seq_ids = fs.seq_ids; P.ctx_len = fs.ctx_len; P.mask = fs.mask;
    P.err = fs.err; P.bar = fs.bar; P.maps = reinterpret_cast<const CUtensorMap *>(fs.d_maps);
    // tensor maps: 4 per layer, lm-head, one per Eq. 3 GEMM, then the activations x, xp, o, y
    const int m_lm = 4 * L, m_pred0 = 4 * L + 1, m_x = 4 * L + 9;
    std::vector<CUtensorMap> &maps = plan->maps;
    maps.assign(4 * L + 13, CUtensorMap{});
    bool ok = true;
    for (int j = 0; j < L && ok; ++j) {
      ok = ok && encode_map(&maps[4 * j + 0], fs.wqkv[j], (uint64_t)(H + 2 * Hkv) * dh, d, BM, dh / 2);
      ok = ok && encode_map(&maps[4 * j + 1], fs.wo[j], d, nq, BM, 0);
      ok = ok && encode_map(&maps[4 * j + 2], fs.wgu[j], 2 * (uint64_t)F, d, BM, 0);
      ok = ok && encode_map(&maps[4 * j + 3], fs.wd[j], d, F, BM, 0);
    }
    if (fs.want_head) ok = ok && encode_map(&maps[m_lm], fs.lm_head, sh.V, d, BM, 0);
    const int xrows = std::min((rw.R + 7) & ~7, NPAD);
    ok = ok && encode_map(&maps[m_x + 0], fs.x, (uint64_t)2 * fs.Rp + rw.R, d, xrows, 0);
    ok = ok && encode_map(&maps[m_x + 1], fs.xp, (uint64_t)fs.Rp + rw.R, d, xrows, 0);
    ok = ok && encode_map(&maps[m_x + 2], fs.o, (uint64_t)fs.Rp + rw.R, nq, xrows, 0);
    ok = ok && encode_map(&maps[m_x + 3], fs.y, (uint64_t)fs.Rp + rw.R, F, xrows, 0);
    if (!ok) return cudaErrorInvalidValue;
    // GEMM classes
    enum { C_QKV = 0, C_O, C_GU, C_DOWN, C_LM, C_PSEUDO0 };
    P.cls[C_QKV] = make_class(EPI_QKV_ROPE, (H + 2 * Hkv) * dh, d, 2, m_x + 0, F, H, Hkv, dh);
    P.cls[C_O] = make_class(EPI_RESIDUAL, d, nq, 2, m_x + 2, F, H, Hkv, dh);
    P.cls[C_GU] = make_class(EPI_SWIGLU, 2 * F, d, 2, m_x + 0, F, H, Hkv, dh);
    P.cls[C_DOWN] = make_class(EPI_RESIDUAL, d, F, 2, m_x + 3, F, H, Hkv, dh);
    P.cls[C_LM] = make_class(EPI_LOGITS, sh.V, d, 2, m_x + 0, F, H, Hkv, dh);
    P.n_cls = C_PSEUDO0;
    int n_ops = 0, n_gemm = 0;
    auto add_op = [&](uint8_t type, int cls, int planes, int layer, int v0, int nv, int act, int aux, const void *ptr) {
      FusedOp &o = P.ops[n_ops++];
      o.type = type; o.cls = (uint8_t)cls; o.planes = (uint8_t)planes; o.pad = 0; o.layer = (int16_t)layer;
      o.v0 = (int16_t)v0; o.nv = (int16_t)nv; o.act = (int16_t)act; o.aux = (int16_t)aux; o.ptr = ptr;
    };
    auto add_gemm = [&](int cls, int map, int layer, int act) {
      P.gemm_cls[n_gemm] = (uint16_t)cls; P.gemm_map[n_gemm] = (uint16_t)map; ++n_gemm;
      add_op(OP_GEMM, cls, 0, layer, 0, 0, act, 0, nullptr);
    };
    int alive = 0, pending = -1, n_pred = 0;
    const int per_step = rw.chains ? rw.T : 1;
    for (int j = 0; j < L; ++j) {
      int ins = 0;
      while (alive + ins < rw.kc && fs.tl[alive + ins] == j) ++ins;
      const int carried = rw.T + alive * per_step, act = carried + ins * per_step;
      add_op(OP_NORM, 0, 2, j, 0, carried, carried, pending, fs.g_attn[j]);
      pending = -1;
      if (ins > 0) {       // Eq. 3 on the raw (now complete) residual rows, then the norm of the new rows
        if (n_pred >= 8 || P.n_cls >= kMaxClasses) return cudaErrorInvalidConfiguration;
        const int cls = P.n_cls++;
        P.cls[cls] = make_class(EPI_PSEUDO, ins * d, d, 2, m_x + 1, F, H, Hkv, dh);
        if (!class_fits(P.cls[cls], G)) return cudaErrorInvalidConfiguration;
        if (!encode_map(&maps[m_pred0 + n_pred], (const bf16 *)fs.pred_w + (size_t)alive * d * d, (uint64_t)ins * d, d, BM, 0))
          return cudaErrorInvalidValue;
        add_op(OP_ROOT_SPLIT, 0, 0, j, 0, 0, act, 0, fs.prenorm ? fs.g_attn[j] : nullptr);
        add_gemm(cls, m_pred0 + n_pred, j, act);
        add_op(OP_FINISH, cls, fs.prenorm ? 1 : 0, j, 0, 0, act, alive, fs.pred_b ? (const bf16 *)fs.pred_b + (size_t)alive * d : nullptr);
        add_op(OP_NORM, 0, 2, j, carried, act - carried, act, -1, fs.g_attn[j]);
        ++n_pred;
        alive += ins;
      }
      add_gemm(C_QKV, 4 * j + 0, j, act);
      add_op(OP_FINISH, C_QKV, 0, j, 0, 0, act, 0, nullptr);
      add_op(OP_ATTN, 0, 0, j, 0, 0, act, 0, nullptr);
      add_op(OP_MERGE, 0, 0, j, 0, 0, act, 0, nullptr);
      add_gemm(C_O, 4 * j + 1, j, act);
      add_op(OP_NORM, 0, 2, j, 0, act, act, C_O, fs.g_mlp[j]);
      add_gemm(C_GU, 4 * j + 2, j, act);
      add_op(OP_FINISH, C_GU, 0, j, 0, 0, act, 0, nullptr);
      add_gemm(C_DOWN, 4 * j + 3, j, act);
      pending = C_DOWN;
    }
    if (fs.want_head) {
      add_op(OP_NORM, 0, 2, -1, 0, rw.Ms, rw.Ms, pending, fs.g_final);
      pending = -1;
      add_gemm(C_LM, m_lm, -1, rw.Ms);
      add_op(OP_FINISH, C_LM, 0, -1, 0, 0, rw.Ms, 0, nullptr);
    }
    P.n_ops = n_ops; P.n_gemm = n_gemm;
    cudaError_t e = cudaMemcpyAsync(fs.d_maps, maps.data(), sizeof(CUtensorMap) * maps.size(), cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return e;
    plan->rw = rw; memcpy(plan->tl, fs.tl, sizeof(plan->tl)); plan->want_head = fs.want_head;
    plan->weights_gen = fs.weights_gen; plan->bufs_key = (const void *)fs.d_maps;
    plan->valid = true;
  }
  // per-call values
  P.logits = fs.logits;
  P.wait_ns = fs.wait_ns;
  {
    // kv splits: every (sequence x query block, kv head, split) is one work item, a CTA takes items cta, cta + G, ...
    // Pick the split count that minimises the 64-position tiles the busiest CTA walks through (rounds x tiles per
    // split), with a charge per round for the latency of an item's first loads (measured: about 2.5 tiles' worth).
    const int Gq = H / Hkv;
    const int tiles = (fs.n_hi_max + rw.Ms + kAttnTile - 1) / kAttnTile;
    const int groups = rw.n_seq * Hkv * ((rw.Ms * Gq + kAttnQRows - 1) / kAttnQRows);
    const size_t cap_items = fused_attn_ws_floats(fs.max_batch, H, Hkv, dh) / ((size_t)kAttnQRows * (dh + 2));
    int best = 1;
    float best_cost = 1e30f;
    for (int s = 1; s <= kMaxSplitsFused && s <= tiles; ++s) {
      if ((size_t)groups * s > cap_items) break;
      const int rounds = (groups * s + G - 1) / G, per = (tiles + s - 1) / s;
      const float cost = (float)rounds * ((float)per + 2.5f);   // an item costs about 2.5 tiles' worth before its first tile
      if (cost < best_cost - 1e-6f) { best_cost = cost; best = s; }
    }
    P.splits = best;
  }
  static bool configured[2] = {false, false};
  auto kernel = NPAD == 16 ? fused_layers_kernel<16> : fused_layers_kernel<48>;
  if (!configured[NPAD == 16]) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kFusedSmem);
    if (e != cudaSuccess) return e;
    configured[NPAD == 16] = true;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)G);
  cfg.blockDim = dim3(kFThreads);
  cfg.dynamicSmemBytes = kFusedSmem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 2 : 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, P);
  if (e == cudaSuccess && launches) ++*launches;
  return e;
}

}  // namespace firp
