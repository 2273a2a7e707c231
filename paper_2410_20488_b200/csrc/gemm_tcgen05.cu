// Skinny weight-streaming GEMM on the 5th-generation tensor cores (tcgen05 + TMEM), operands
// staged by TMA.  out[m][n] = sum_k X[m][k] * W[n][k], M = T + k token rows, W read once.
//
// Roles are swapped: a tile is 128 weight rows (the MMA M dimension, one TMEM lane each) by all
// token rows (the MMA N dimension, one TMEM column each).  Per CTA:
//   warp 0   : weight producer.  One thread streams [128 rows x 64 k] bf16 tiles (two 64-row TMA
//              boxes, 128-byte swizzle) through a deep ring.  Weights never depend on the previous
//              kernel, so this warp does not wait for it: under programmatic dependent launch the
//              weight stream of this GEMM starts while its predecessor drains.
//   warp 6   : activation producer.  Streams the matching [NPAD x 64] hi and lo activation tiles
//              (L2-resident) through a short ring, after waiting for the previous kernel.
//   warp 1   : MMA issuer.  One thread issues tcgen05.mma (M=128, N=NPAD, K=16, bf16 x bf16 -> fp32
//              in TMEM): per 64-wide k block 4 steps x {hi, lo} activations into one accumulator;
//              tcgen05.commit hands ring slots back to the producers.
//   warps 2-5: epilogue.  tcgen05.ld the accumulator (lane = weight row, column = token), stage it
//              as C[token][row] in shared memory and run the fused epilogue.
// Every mbarrier wait is bounded: after ~2 s it sets the status word and falls through, so a
// broken pipeline ends with an error code instead of a hang; TMEM is always released.
#include <cuda.h>

#include <map>
#include <tuple>

#include "firp_kernels.cuh"
#include "gemm_epilogue.cuh"

namespace firp {

namespace {

constexpr int BM = 128;           // weight rows per tile
constexpr int BK = kGemmBK;       // 64 bf16 = 128 bytes = one swizzle row
constexpr int kThreads = 224;     // 7 warps
constexpr int W_TILE = BM * 128;  // bytes per weight stage
constexpr int kErrTimeout = 100;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned long long globaltimer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  `dead` is sticky per thread: after one timeout later waits return at once.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, int *err, bool &dead) {
  if (dead || mbar_try_wait(bar, parity)) return;
  const unsigned long long t0 = globaltimer();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 255u) == 0 && globaltimer() - t0 > 2000000000ull) {
      dead = true;
      atomicExch(err, kErrTimeout);
      return;
    }
  }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *tm, int x, int y, uint32_t bar,
                                            uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(bar), "l"(policy) : "memory");
}
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
               ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t *r) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                 "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
               : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory operand descriptor: K-major tile of 128-byte rows, 128-byte swizzle, 8-row groups
// 1024 bytes apart (start address >> 4 in bits 0-13, leading offset 1 in bits 16-29 (unused for
// swizzled K-major), stride offset 1024 >> 4 in bits 32-45, version 1 in bits 46-47, layout 2 =
// SWIZZLE_128B in bits 61-63).  Advancing K by 16 elements adds 32 bytes to the start address.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) |
         ((uint64_t)2 << 61);
}
// Instruction descriptor, kind::f16: fp32 accumulator (bits 4-5 = 1), A and B bf16 (bits 7-9, 10-12 = 1),
// both K-major (bits 15, 16 = 0), N >> 3 in bits 17-22, M >> 4 in bits 24-28.
__host__ __device__ constexpr uint32_t instr_desc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

template <int NPAD> struct TcCfg {
  static constexpr int X_TILE = NPAD * 128;                      // bytes of one activation plane per stage
  static constexpr int WS = (NPAD <= 48) ? 5 : (NPAD <= 80 ? 4 : 8);  // weight ring depth (two CTAs per SM up to NPAD = 80)
  static constexpr int XS = 2;                                   // activation ring depth
  static constexpr int TMEM_COLS = NPAD <= 32 ? 32 : (NPAD <= 64 ? 64 : (NPAD <= 128 ? 128 : 256));
  static constexpr int RING_BYTES = WS * W_TILE + XS * 2 * X_TILE;
  static constexpr int C_BYTES = NPAD * BM * 4;
  static constexpr int DATA_BYTES = RING_BYTES > C_BYTES ? RING_BYTES : C_BYTES;
  static constexpr int SMEM = DATA_BYTES + 1024 /* alignment slack */ + 256 /* barriers */;
};

struct TcArgs {
  int box1_off;   // rows from the first 64-row box of a tile to the second (64, or pair_off)
  int tile_rows;  // rows a tile advances the first box by (128 contiguous, 64 paired)
  int pdl;        // launched with programmatic stream serialization
};

template <int NPAD, int EPI>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX, GemmArgs a,
               TileMap tm, TcArgs t) {
  using Cfg = TcCfg<NPAD>;
  constexpr int WS = Cfg::WS, XS = Cfg::XS, X_TILE = Cfg::X_TILE;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;      // swizzled tiles need 1024-byte alignment
  uint8_t *data = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t w_ring = base, x_ring = base + WS * W_TILE;
  const uint32_t bars = base + Cfg::DATA_BYTES;                     // 8-byte barriers
  const uint32_t full_w = bars, empty_w = bars + 8 * WS, full_x = bars + 16 * WS, empty_x = full_x + 8 * XS,
                 accum_bar = empty_x + 8 * XS, tmem_slot = accum_bar + 8;
  volatile uint32_t *tmem_slot_ptr = reinterpret_cast<volatile uint32_t *>(data + Cfg::DATA_BYTES + 16 * WS + 16 * XS + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = blockIdx.x, split = blockIdx.y;
  const int kb_total = (a.K + BK - 1) / BK;
  const int kb_per = (kb_total + a.splits - 1) / a.splits;
  const int kb0 = split * kb_per;
  const int nkb = max(min(kb_total, kb0 + kb_per) - kb0, 0);

  if (threadIdx.x == 0) {
    for (int i = 0; i < WS; ++i) { mbar_init(full_w + 8 * i, 1); mbar_init(empty_w + 8 * i, 1); }
    for (int i = 0; i < XS; ++i) { mbar_init(full_x + 8 * i, 1); mbar_init(empty_x + 8 * i, 1); }
    mbar_init(accum_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {   // TMEM: one warp allocates (and later frees) the accumulator columns
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(Cfg::TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_acc = *tmem_slot_ptr;
  if (t.pdl) griddep_launch();   // the next kernel may start its own weight stream

  bool dead = false;
  if (warp == 0) {
    if (lane == 0) {             // ---- weight producer: does not wait for the previous kernel
      uint64_t pol;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
      const int r0 = tile * t.tile_rows, r1 = r0 + t.box1_off;
      for (int it = 0; it < nkb; ++it) {
        const int st = it % WS;
        mbar_wait(empty_w + 8 * st, ((it / WS) & 1) ^ 1, a.err, dead);
        mbar_expect_tx(full_w + 8 * st, W_TILE);
        const int k0 = (kb0 + it) * BK;
        tma_load_2d(w_ring + st * W_TILE, &tmW, k0, r0, full_w + 8 * st, pol);
        tma_load_2d(w_ring + st * W_TILE + W_TILE / 2, &tmW, k0, r1, full_w + 8 * st, pol);
      }
    }
  } else if (warp == 6) {
    if (lane == 0) {             // ---- activation producer
      uint64_t pol;
      asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
      if (t.pdl) griddep_wait();
      for (int it = 0; it < nkb; ++it) {
        const int st = it % XS;
        mbar_wait(empty_x + 8 * st, ((it / XS) & 1) ^ 1, a.err, dead);
        mbar_expect_tx(full_x + 8 * st, 2 * X_TILE);
        const int k0 = (kb0 + it) * BK;
        tma_load_2d(x_ring + st * 2 * X_TILE, &tmX, k0, 0, full_x + 8 * st, pol);
        tma_load_2d(x_ring + st * 2 * X_TILE + X_TILE, &tmX, k0, a.plane_rows, full_x + 8 * st, pol);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {             // ---- MMA issuer
      constexpr uint32_t idesc = instr_desc(NPAD);
      for (int it = 0; it < nkb; ++it) {
        const int sw = it % WS, sx = it % XS;
        mbar_wait(full_w + 8 * sw, (it / WS) & 1, a.err, dead);
        mbar_wait(full_x + 8 * sx, (it / XS) & 1, a.err, dead);
        tc_fence_after();
        const uint64_t da = smem_desc(w_ring + sw * W_TILE);
        const uint64_t dhi = smem_desc(x_ring + sx * 2 * X_TILE), dlo = smem_desc(x_ring + sx * 2 * X_TILE + X_TILE);
#pragma unroll
        for (int kk = 0; kk < BK / 16; ++kk) {
          tc_mma(tmem_acc, da + 2 * kk, dhi + 2 * kk, idesc, (it | kk) != 0);
          tc_mma(tmem_acc, da + 2 * kk, dlo + 2 * kk, idesc, 1u);
        }
        tc_commit(empty_w + 8 * sw);   // slots are free once these MMAs have read them
        tc_commit(empty_x + 8 * sx);
      }
      tc_commit(accum_bar);
    }
  } else {                       // ---- epilogue warps 2..5: TMEM lane quarter = warp % 4
    if (t.pdl) griddep_wait();
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;          // tile-local weight row = TMEM lane
    float *C = reinterpret_cast<float *>(data);   // C[token][BM], reuses the rings
    if (nkb > 0) {
      mbar_wait(accum_bar, 0, a.err, dead);
      tc_fence_after();
#pragma unroll
      for (int c0 = 0; c0 < NPAD; c0 += 16) {
        uint32_t r[16];
        tc_ld16(tmem_acc + ((uint32_t)(quarter * 32) << 16) + c0, r);
        tc_ld_wait();
#pragma unroll
        for (int j = 0; j < 16; ++j) C[(c0 + j) * BM + row] = __uint_as_float(r[j]);
      }
    } else {
      for (int m = 0; m < NPAD; ++m) C[m * BM + row] = 0.f;
    }
    tc_fence_before();
    asm volatile("bar.sync 1, 128;" ::: "memory");
    gemm_epilogue<EPI, BM>(C, BM, tile, split, a, tm, threadIdx.x - 64, 128);
  }
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(Cfg::TMEM_COLS) : "memory");
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

// 2-D bf16 tensor [rows][K] (K contiguous), box [box_rows][64], 128-byte swizzle, zero fill out of bounds.
// Encoded maps are cached: the same few (pointer, shape) pairs recur every step.
bool make_map(CUtensorMap *m, const void *ptr, uint64_t rows, uint64_t K, uint32_t box_rows) {
  typedef std::tuple<const void *, uint64_t, uint64_t, uint32_t> Key;
  static std::map<Key, CUtensorMap> cache;
  const Key key(ptr, rows, K, box_rows);
  auto it = cache.find(key);
  if (it != cache.end()) { *m = it->second; return true; }
  const cuuint64_t dims[2] = {K, rows};
  const cuuint64_t strides[1] = {K * 2};
  const cuuint32_t box[2] = {(cuuint32_t)BK, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  if (encode_fn()(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  if (cache.size() > 4096) cache.clear();
  cache[key] = *m;
  return true;
}

template <int NPAD, int EPI>
cudaError_t launch_np(const GemmArgs &a, const TileMap &tm, const TcArgs &t, int tiles, cudaStream_t st) {
  using Cfg = TcCfg<NPAD>;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<NPAD, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  CUtensorMap tmW, tmX;
  if (!make_map(&tmW, a.W, (uint64_t)a.N, (uint64_t)a.K, 64)) return cudaErrorInvalidValue;
  if (!make_map(&tmX, a.X, (uint64_t)a.plane_rows + a.R, (uint64_t)a.K, NPAD)) return cudaErrorInvalidValue;
  GemmArgs b = a;
  b.splits = (EPI == EPI_PARTIAL) ? a.splits : 1;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(tiles, b.splits);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = Cfg::SMEM;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = t.pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, gemm_tc_kernel<NPAD, EPI>, tmW, tmX, b, tm, t);
}

template <int EPI>
cudaError_t launch_epi(const GemmArgs &a, const TileMap &tm, const TcArgs &t, int tiles, cudaStream_t st) {
  if (a.R <= 16) return launch_np<16, EPI>(a, tm, t, tiles, st);
  if (a.R <= 48) return launch_np<48, EPI>(a, tm, t, tiles, st);
  if (a.R <= 80) return launch_np<80, EPI>(a, tm, t, tiles, st);
  return launch_np<144, EPI>(a, tm, t, tiles, st);
}

}  // namespace

bool gemm_tc_available() { return encode_fn() != nullptr; }

cudaError_t launch_gemm_tc(GemmEpilogue epi, const GemmArgs &a, bool pdl, cudaStream_t st) {
  if (!encode_fn()) return cudaErrorNotSupported;
  TileMap tm{};
  TcArgs t{64, BM, pdl ? 1 : 0};
  switch (epi) {
    case EPI_QKV_ROPE:   // contiguous tiles of 128 / dh whole heads
      return launch_epi<EPI_QKV_ROPE>(a, tm, t, (a.N + BM - 1) / BM, st);
    case EPI_SWIGLU:     // 64 gate rows + the matching 64 up rows
      tm.paired = 1; tm.tiles_per_unit = (a.F + 63) / 64; tm.unit_stride = 0; tm.pair_off = a.F; tm.group_rows = a.F;
      t.box1_off = a.F; t.tile_rows = 64;
      return launch_epi<EPI_SWIGLU>(a, tm, t, tm.tiles_per_unit, st);
    case EPI_LOGITS:
      return launch_epi<EPI_LOGITS>(a, tm, t, (a.N + BM - 1) / BM, st);
    default:
      return launch_epi<EPI_PARTIAL>(a, tm, t, (a.N + BM - 1) / BM, st);
  }
}

}  // namespace firp
