// Skinny weight-streaming GEMM on the 5th-generation tensor cores (tcgen05 + TMEM), operands
// staged by TMA.  out[m][n] = sum_k X[m][k] * W[n][k], M = T + k token rows, W read once.
//
// Roles are swapped: weight rows are the MMA M dimension (one TMEM lane each), token rows the
// MMA N dimension (one TMEM column each).  A "supertile" is 2 x 128 weight rows that share one
// activation tile per k block, chosen so that both operands of a fused epilogue meet in one
// thread: lane i of the first 128 rows and lane i of the second are a rotary pair (c, c + dh/2),
// a gate row and its up row, or simply rows n and n + 128.
//
// Persistent stream-K schedule: the (supertile, k block) units of the whole matrix, 32 KB of
// weights each, are cut into one contiguous range per SM, so every SM streams the same number of
// bytes whatever the matrix shape.  A range crosses supertile boundaries; each piece ("segment")
// accumulates in TMEM and its fp32 partial tile is stored to the CTA's scratch slot.  The kernel
// that consumes the GEMM (RMSNorm for the residual GEMMs, the rotary / SwiGLU / logits finishers
// otherwise) sums the slots of a supertile in CTA order, so every sum has a fixed order and results
// are identical from run to run; no CTA ever waits for another.  The finishers are small-footprint
// kernels that stay resident beside the next GEMM's CTAs: under programmatic dependent launch the
// next weight stream starts while they run.
//
// Per CTA (one per SM):
//   warp 0   : weight producer (one thread, TMA, 128-byte swizzle, deep ring).  Weights never
//              depend on the previous kernel, so under programmatic dependent launch this stream
//              starts while the predecessor drains.
//   warp 6   : activation producer: the (hi, lo) bf16 planes of the matching k block (L2
//              resident, own shorter ring), after waiting for the previous kernel.
//   warp 1   : MMA issuer: tcgen05.mma kind::f16, M = 128, K = 16; the bf16 planes of the
//              activations (hi, lo, or hi, mid, lo) sit one after the other in shared memory and are
//              multiplied as ONE operand of N = planes x NPAD token columns (the sums over each
//              plane land in neighbouring TMEM columns and are added in the epilogue);
//              tcgen05.commit releases ring slots.
//   warps 2-5: epilogue: tcgen05.ld (lane = weight row, column = token), hi + lo, store of the
//              partial tile; overlapped with the next segment's main loop through a second
//              accumulator buffer.
// Every mbarrier wait is bounded (~2 s): on expiry the status word is set and the kernel runs to
// its end; TMEM is always released.
#include <cuda.h>

#include <cstdlib>
#include <map>
#include <tuple>

#include "firp_kernels.cuh"
#include "launch_util.cuh"
#include "tc_device.cuh"

namespace firp {

namespace {

constexpr int BM = 128;            // weight rows per MMA tile
constexpr int TM = 2;              // MMA tiles per supertile
constexpr int BK = kGemmBK;        // 64 bf16 = 128 bytes = one swizzle row
constexpr int kThreads = 224;      // 7 warps
constexpr int W_TILE = BM * 128;   // bytes of one 128-row weight tile of a k block
constexpr int W_STAGE = TM * W_TILE;

constexpr int pow2_cols(int c) { return c <= 32 ? 32 : c <= 64 ? 64 : c <= 128 ? 128 : c <= 256 ? 256 : 512; }

// NPAD = token rows padded to a multiple of 8; P = bf16 planes of the activations (2: hi + lo,
// 3: hi + mid + lo).  The planes of a stage sit one after the other in shared memory; when P * NPAD is
// a legal MMA N (a multiple of 16, <= 256) they are multiplied as one operand, otherwise plane by plane.
template <int NPAD, int P> struct TcCfg {
  static constexpr int X_PLANE = NPAD * 128;                   // bytes of one activation plane per stage
  static constexpr int X_STAGE = P * X_PLANE;
  // two planes are merged only while two accumulator buffers still fit the 512 TMEM columns (measured: the
  // second buffer -- epilogue of one segment under the main loop of the next -- is worth more than one MMA
  // instead of two); three planes are always merged when legal (measured the other way round)
  static constexpr bool MERGE = (P * NPAD <= 256) && ((P * NPAD) % 16 == 0) && (2 * TM * P * NPAD <= 512 || NPAD % 16 != 0 || P > 2);
  static constexpr int ACC_COLS = MERGE ? P * NPAD : NPAD;     // accumulator columns per weight tile
  static constexpr int NBUF = (2 * TM * ACC_COLS <= 512) ? 2 : 1;   // accumulator buffers
  static constexpr int TMEM_COLS = pow2_cols(NBUF * TM * ACC_COLS);
  // ring depths: as many 32 KB weight stages as fit beside two to four activation stages
  // (an activation stage of the 144-row variant is 36 KB and comes from L2 in ~2 us: with two stages that
  // latency, not the weight stream or the MMAs, set the pace of a unit; three stages beside three weight stages)
  static constexpr int SX = X_STAGE <= 8 * 1024 ? 4 : (X_STAGE <= 40 * 1024 ? 3 : 2);
  static constexpr int SW = (227 * 1024 - 1280 - SX * X_STAGE) / W_STAGE > 6 ? 6 : (227 * 1024 - 1280 - SX * X_STAGE) / W_STAGE;
  static constexpr int RING_BYTES = SW * W_STAGE + SX * X_STAGE;
  static constexpr int SMEM = RING_BYTES + 1024 /* alignment slack */ + 256 /* barriers */;
  static_assert(!MERGE || NPAD % 8 == 0, "planes must start on a swizzle atom");
  static_assert(MERGE || NPAD % 16 == 0, "MMA N must be a multiple of 16");
  static_assert(SW >= 3 && SMEM <= 227 * 1024, "shared memory budget");
  static_assert((2 * SW + 2 * SX + 2 * NBUF) * 8 + 8 <= 256, "barrier area");
};

// How the 2 x 128 rows of supertile `st` map to weight rows.
//   ROWS_LINEAR   rows st*256 .. +255 (two boxes of 128 rows)
//   ROWS_GATE_UP  gate rows st*128 .. +127, then the matching up rows F + st*128 ..
//   ROWS_ROTARY   first halves (c < dh/2) of 128/(dh/2) heads, then their second halves, fetched
//                 through a 4-D view [head][half][c][k] of the weight so that each is one box
enum RowMode { ROWS_LINEAR = 0, ROWS_GATE_UP = 1, ROWS_ROTARY = 2 };
struct Sched {
  StreamK sk;      // units, k blocks per supertile, CTAs
  int mode;        // RowMode
  int F;           // ROWS_GATE_UP: rows of the gate matrix
  int half;        // ROWS_ROTARY: dh / 2
  int n_st;        // supertiles
  int pdl;         // launched with programmatic stream serialization
  int ws_rows;     // token rows per scratch tile
  int l2_ahead;    // units each CTA prefetches into L2 beyond its shared-memory ring
};

// L2 prefetch of the two weight tiles of unit (supertile st, k block kb) under schedule sc
__device__ __forceinline__ void prefetch_unit(const CUtensorMap *tm, const Sched &sc, int st, int kb, uint64_t pol) {
  if (sc.mode == ROWS_ROTARY) {
    const int hp = BM / sc.half;
    tma_prefetch_4d(tm, kb * BK, 0, 0, st * hp, pol);
    tma_prefetch_4d(tm, kb * BK, 0, 1, st * hp, pol);
  } else if (sc.mode == ROWS_GATE_UP) {
    tma_prefetch_2d(tm, kb * BK, st * BM, pol);
    tma_prefetch_2d(tm, kb * BK, sc.F + st * BM, pol);
  } else {
    tma_prefetch_2d(tm, kb * BK, st * (TM * BM), pol);
    tma_prefetch_2d(tm, kb * BK, st * (TM * BM) + BM, pol);
  }
}

template <int NPAD, int P>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
               const __grid_constant__ CUtensorMap tmNext, GemmArgs a, Sched sc, Sched nx) {
  using Cfg = TcCfg<NPAD, P>;
  constexpr int SW = Cfg::SW, SX = Cfg::SX, X_STAGE = Cfg::X_STAGE, X_PLANE = Cfg::X_PLANE, NBUF = Cfg::NBUF;
  constexpr int ACC = Cfg::ACC_COLS;
  constexpr bool MERGE = Cfg::MERGE;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;      // swizzled tiles need 1024-byte alignment
  uint8_t *data = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t w_ring = base, x_ring = base + SW * W_STAGE;
  const uint32_t bars = base + Cfg::RING_BYTES;                     // 8-byte barriers
  const uint32_t full_w = bars, empty_w = full_w + 8 * SW, full_x = empty_w + 8 * SW, empty_x = full_x + 8 * SX,
                 acc_full = empty_x + 8 * SX, acc_empty = acc_full + 8 * NBUF, tmem_slot = acc_empty + 8 * NBUF;
  volatile uint32_t *tmem_slot_ptr =
      reinterpret_cast<volatile uint32_t *>(data + Cfg::RING_BYTES + 16 * SW + 16 * SX + 16 * NBUF);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x;
  const StreamK sk = sc.sk;
  const int KB = sk.KB;
  const int u0 = sk_begin(sk, cta), u1 = sk_begin(sk, cta + 1);
  const int n_units = u1 - u0;

  if (threadIdx.x == 0) {
    for (int i = 0; i < SW; ++i) { mbar_init(full_w + 8 * i, 1); mbar_init(empty_w + 8 * i, 1); }
    for (int i = 0; i < SX; ++i) { mbar_init(full_x + 8 * i, 1); mbar_init(empty_x + 8 * i, 1); }
    for (int i = 0; i < NBUF; ++i) { mbar_init(acc_full + 8 * i, 1); mbar_init(acc_empty + 8 * i, 4); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();                 // barriers are initialised
  if (sc.pdl) griddep_launch();    // the next kernel may start its own weight stream as SMs free up
  // The two producers start at once; the warps that touch TMEM (MMA issuer and epilogue) meet on their own
  // barrier once warp 1 has allocated (and later frees) the accumulator columns.
  uint32_t tmem_base = 0;
  if (warp >= 1 && warp <= 5) {
    if (warp == 1) {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(Cfg::TMEM_COLS) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    asm volatile("bar.sync 2, 160;" ::: "memory");
    tc_fence_after();
    tmem_base = *tmem_slot_ptr;
  }

  bool dead = false;
  const unsigned long long wait_ns = a.wait_ns ? a.wait_ns : kDefaultWaitNs;
  if (warp == 0) {
    if (lane == 0) {             // ---- weight producer: does not wait for the previous kernel
      uint64_t pol;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmW) : "memory");
      // While the ring is full (typically: the activations are not there yet because the previous kernel is
      // still running) the stream goes on into L2: units up to l2_ahead beyond the ring are prefetched, so
      // HBM stays busy during the small kernels between two GEMMs and the ring later refills from L2.
      int pf = SW;
      for (int it = 0; it < n_units; ++it) {
        for (const int upto = min(n_units, it + SW + sc.l2_ahead); pf < upto; ++pf) {
          const int up = u0 + pf;
          prefetch_unit(&tmW, sc, up / KB, up % KB, pol);
        }
        const int u = u0 + it;
        const int st = u / KB, kb = u - st * KB;
        const int sl = it % SW;
        mbar_wait(empty_w + 8 * sl, ((it / SW) & 1) ^ 1, a.err, dead, wait_ns);
        mbar_expect_tx(full_w + 8 * sl, W_STAGE);
        const uint32_t dst = w_ring + sl * W_STAGE, bar = full_w + 8 * sl;
        if (sc.mode == ROWS_ROTARY) {
          const int hp = BM / sc.half;               // heads per supertile
          tma_load_4d(dst, &tmW, kb * BK, 0, 0, st * hp, bar, pol);
          tma_load_4d(dst + W_TILE, &tmW, kb * BK, 0, 1, st * hp, bar, pol);
        } else if (sc.mode == ROWS_GATE_UP) {
          tma_load_2d(dst, &tmW, kb * BK, st * BM, bar, pol);
          tma_load_2d(dst + W_TILE, &tmW, kb * BK, sc.F + st * BM, bar, pol);
        } else {
          tma_load_2d(dst, &tmW, kb * BK, st * (TM * BM), bar, pol);
          tma_load_2d(dst + W_TILE, &tmW, kb * BK, st * (TM * BM) + BM, bar, pol);
        }
      }
      // all own loads are out: bring the head of the next GEMM's range of this CTA into L2
      if (nx.l2_ahead > 0 && cta < nx.sk.G) {
        const int v0 = sk_begin(nx.sk, cta), v1 = min(sk_begin(nx.sk, cta + 1), v0 + nx.l2_ahead);
        for (int v = v0; v < v1; ++v) prefetch_unit(&tmNext, nx, v / nx.sk.KB, v % nx.sk.KB, pol);
      }
    }
  } else if (warp == 6) {
    if (lane == 0) {             // ---- activation producer
      uint64_t pol;
      asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
      if (sc.pdl) griddep_wait();
      const int xrows = min((a.R + 7) & ~7, NPAD);
      for (int it = 0; it < n_units; ++it) {
        const int kb = (int)((u0 + it) % KB);
        const int sl = it % SX;
        mbar_wait(empty_x + 8 * sl, ((it / SX) & 1) ^ 1, a.err, dead, wait_ns);
        mbar_expect_tx(full_x + 8 * sl, P * xrows * 128);
        const uint32_t dst = x_ring + sl * X_STAGE;
#pragma unroll
        for (int pl = 0; pl < P; ++pl)
          tma_load_2d(dst + pl * X_PLANE, &tmX, kb * BK, pl * a.plane_rows, full_x + 8 * sl, pol);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {             // ---- MMA issuer
      constexpr uint32_t idesc = instr_desc_m128(MERGE ? P * NPAD : NPAD);
      int it = 0, seg = 0;
      int u = u0;
      while (u < u1) {
        const int st = u / KB, kb0 = u - st * KB;
        const int kb1 = min(KB, kb0 + (u1 - u));
        const int buf = seg % NBUF;
        mbar_wait(acc_empty + 8 * buf, ((seg / NBUF) & 1) ^ 1, a.err, dead, wait_ns);   // epilogue has drained this buffer
        tc_fence_after();
        const uint32_t acc = tmem_base + (uint32_t)(buf * TM * ACC);
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const int sw = it % SW, sx = it % SX;
          mbar_wait(full_w + 8 * sw, (it / SW) & 1, a.err, dead, wait_ns);
          mbar_wait(full_x + 8 * sx, (it / SX) & 1, a.err, dead, wait_ns);
          tc_fence_after();
          const uint32_t wst = w_ring + sw * W_STAGE, xst = x_ring + sx * X_STAGE;
          const uint64_t dx = smem_desc(xst);
#pragma unroll
          for (int kk = 0; kk < BK / 16; ++kk) {
#pragma unroll
            for (int t = 0; t < TM; ++t) {
              const uint64_t da = smem_desc(wst + t * W_TILE) + 2 * kk;
              tc_mma(acc + t * ACC, da, dx + 2 * kk, idesc, (kb > kb0 || kk > 0) ? 1u : 0u);
              if (!MERGE) {
#pragma unroll
                for (int pl = 1; pl < P; ++pl) tc_mma(acc + t * ACC, da, dx + (pl * X_PLANE >> 4) + 2 * kk, idesc, 1u);
              }
            }
          }
          tc_commit(empty_w + 8 * sw);   // the slots are free once these MMAs have read them
          tc_commit(empty_x + 8 * sx);
        }
        tc_commit(acc_full + 8 * buf);
        u += kb1 - kb0;
        ++seg;
      }
    }
  } else {                       // ---- epilogue warps 2..5: TMEM lane quarter = warp % 4
    if (sc.pdl) griddep_wait();
    const int quarter = warp & 3;
    const int i = quarter * 32 + lane;            // row within each 128-row tile = TMEM lane
    const size_t plane_elems = (size_t)sc.ws_rows * BM, slot_elems = TM * plane_elems;
    int seg = 0;
    int u = u0;
    while (u < u1) {
      const int st = u / KB, kb0 = u - st * KB;
      const int kb1 = min(KB, kb0 + (u1 - u));
      const int buf = seg % NBUF;
      mbar_wait(acc_full + 8 * buf, (seg / NBUF) & 1, a.err, dead, wait_ns);
      tc_fence_after();
      const uint32_t tacc = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * TM * ACC);
      float *my_ws = a.ws + (size_t)(cta * kGemmSlots + seg) * slot_elems + i;
      for (int c0 = 0; c0 < a.R && seg < kGemmSlots; c0 += 16) {
        float r0[16], r1[16];
        tc_ld16(tacc + c0, r0);
        tc_ld16(tacc + ACC + c0, r1);
        tc_ld_wait();
        if (MERGE) {             // columns pl * NPAD .. hold the sums over plane pl
#pragma unroll
          for (int pl = 1; pl < P; ++pl) {
            float l0[16], l1[16];
            tc_ld16(tacc + pl * NPAD + c0, l0);
            tc_ld16(tacc + ACC + pl * NPAD + c0, l1);
            tc_ld_wait();
#pragma unroll
            for (int j = 0; j < 16; ++j) { r0[j] += l0[j]; r1[j] += l1[j]; }
          }
        }
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int m = c0 + j;
          if (m < a.R) {
            __stcg(my_ws + (size_t)m * BM, r0[j]);
            __stcg(my_ws + plane_elems + (size_t)m * BM, r1[j]);
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty + 8 * buf);   // the MMA warp may reuse this accumulator
      u += kb1 - kb0;
      ++seg;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(Cfg::TMEM_COLS) : "memory");
  }
}

// ---- host side ---------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
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

// bf16 tensor maps with 64-element (128-byte) inner boxes, 128-byte swizzle, zero fill out of bounds.
//   half == 0: 2-D [rows][K], box [box_rows][64]
//   half  > 0: 4-D view [rows / (2 half)][2][half][K] of a QKV weight, box [128 / half][1][half][64]:
//              the same half of 128 / half neighbouring heads
// Encoded maps are cached: the same few (pointer, shape) pairs recur every step.
bool make_map(CUtensorMap *m, const void *ptr, uint64_t rows, uint64_t K, uint32_t box_rows, uint32_t half) {
  typedef std::tuple<const void *, uint64_t, uint64_t, uint32_t, uint32_t> Key;
  static std::map<Key, CUtensorMap> cache;
  const Key key(ptr, rows, K, box_rows, half);
  auto it = cache.find(key);
  if (it != cache.end()) { *m = it->second; return true; }
  CUresult rc;
  if (half == 0) {
    const cuuint64_t dims[2] = {K, rows};
    const cuuint64_t strides[1] = {K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)BK, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    rc = encode_fn()(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else {
    const cuuint64_t dims[4] = {K, half, 2, rows / (2 * half)};
    const cuuint64_t strides[3] = {K * 2, (cuuint64_t)half * K * 2, (cuuint64_t)2 * half * K * 2};
    const cuuint32_t box[4] = {(cuuint32_t)BK, half, 1, (cuuint32_t)BM / half};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    rc = encode_fn()(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(ptr), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }
  if (rc != CUDA_SUCCESS) return false;
  if (cache.size() > 4096) cache.clear();
  cache[key] = *m;
  return true;
}

int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 1;
  }
  return n;
}

Sched make_sched(GemmEpilogue epi, const GemmArgs &a, bool pdl);

template <int NPAD, int P>
cudaError_t launch_np(const GemmArgs &a, const Sched &sc, cudaStream_t st) {
  using Cfg = TcCfg<NPAD, P>;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<NPAD, P>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  const int xrows = std::min((a.R + 7) & ~7, NPAD);
  CUtensorMap tmW, tmX;
  if (!make_map(&tmW, a.W, (uint64_t)a.N, (uint64_t)a.K, BM, sc.mode == ROWS_ROTARY ? (uint32_t)sc.half : 0u))
    return cudaErrorInvalidValue;
  if (!make_map(&tmX, a.X, (uint64_t)(P - 1) * a.plane_rows + a.R, (uint64_t)a.K, (uint32_t)xrows, 0)) return cudaErrorInvalidValue;
  // the GEMM that follows (if any): its weight map and schedule, for the tail prefetch
  CUtensorMap tmNext = tmW;
  Sched nx{};
  if (a.next_W && a.next_units > 0) {
    GemmArgs b{};
    b.W = a.next_W; b.N = a.next_N; b.K = a.next_K; b.F = a.next_F; b.dh = a.next_dh; b.plane_rows = a.plane_rows;
    b.H = a.next_heads; b.Hkv = 0;
    nx = make_sched((GemmEpilogue)a.next_epi, b, false);
    nx.l2_ahead = a.next_units;
    if (!make_map(&tmNext, b.W, (uint64_t)b.N, (uint64_t)b.K, BM, nx.mode == ROWS_ROTARY ? (uint32_t)nx.half : 0u))
      return cudaErrorInvalidValue;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)sc.sk.G);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = Cfg::SMEM;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = sc.pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, gemm_tc_kernel<NPAD, P>, tmW, tmX, tmNext, a, sc, nx);
}

cudaError_t launch_rows(const GemmArgs &a, const Sched &sc, cudaStream_t st) {
  if (a.planes == 3) {   // N = 3 NPAD must be a multiple of 16
    if (a.R <= 16) return launch_np<16, 3>(a, sc, st);
    if (a.R <= 48) return launch_np<48, 3>(a, sc, st);
    if (a.R <= 80) return launch_np<80, 3>(a, sc, st);
    return launch_np<144, 3>(a, sc, st);
  }
  if (a.planes == 1) {   // plain bf16 activations (the hi plane alone)
    if (a.R <= 16) return launch_np<16, 1>(a, sc, st);
    if (a.R <= 48) return launch_np<48, 1>(a, sc, st);
    if (a.R <= 80) return launch_np<80, 1>(a, sc, st);
    return launch_np<144, 1>(a, sc, st);
  }
  if (a.R <= 16) return launch_np<16, 2>(a, sc, st);
  if (a.R <= 40) return launch_np<40, 2>(a, sc, st);
  if (a.R <= 48) return launch_np<48, 2>(a, sc, st);
  if (a.R <= 80) return launch_np<80, 2>(a, sc, st);
  return launch_np<144, 2>(a, sc, st);
}

Sched make_sched(GemmEpilogue epi, const GemmArgs &a, bool pdl) {
  Sched sc{};
  sc.pdl = pdl ? 1 : 0;
  sc.ws_rows = a.plane_rows;
  sc.l2_ahead = a.l2_ahead < 0 ? 0 : a.l2_ahead;
  sc.mode = ROWS_LINEAR; sc.n_st = (a.N + TM * BM - 1) / (TM * BM);
  if (epi == EPI_SWIGLU) {
    sc.mode = ROWS_GATE_UP; sc.F = a.F; sc.n_st = (a.F + BM - 1) / BM;
  } else if (epi == EPI_QKV_ROPE) {
    sc.mode = ROWS_ROTARY; sc.half = a.dh / 2;
    const int hp = BM / sc.half;
    sc.n_st = (a.H + 2 * a.Hkv + hp - 1) / hp;
  }
  sc.sk.KB = (a.K + BK - 1) / BK;
  sc.sk.U = sc.n_st * sc.sk.KB;
  sc.sk.G = std::min(sm_count(), sc.sk.U);
  // With more than 80 rows the MMAs fall behind the weight stream, and a lookahead beyond the ring only fills L2
  // with tiles that are evicted before they are read and then fetched twice (measured at 140 rows: 1.8x the weight
  // bytes from DRAM, step 10 % slower).  With few rows the stream is the bound and the deep lookahead pays.
  if (a.R > 80) sc.l2_ahead = 0;
  return sc;
}

}  // namespace

bool gemm_tc_available() { return encode_fn() != nullptr; }

cudaError_t launch_gemm_tc(GemmEpilogue epi, const GemmArgs &a, bool pdl, cudaStream_t st, StreamK *sk_out) {
  if (!encode_fn()) return cudaErrorNotSupported;
  const Sched sc = make_sched(epi, a, pdl);
  // a CTA's range of U / G units touches at most this many supertiles, each needing a scratch slot
  const int per = (sc.sk.U + sc.sk.G - 1) / sc.sk.G;
  if (sc.sk.G > kGemmMaxCtas || (per + sc.sk.KB - 2) / sc.sk.KB + 1 > kGemmSlots ||
      (long long)(sc.sk.U + 1) * (sc.sk.G + 1) >= (1ll << 31))   // the schedule arithmetic is 32-bit
    return cudaErrorInvalidConfiguration;
  if (sk_out) *sk_out = sc.sk;
  return launch_rows(a, sc, st);
}

}  // namespace firp
