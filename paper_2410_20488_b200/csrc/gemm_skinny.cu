// Skinny weight-streaming GEMM: out[m][n] = sum_k X[m][k] * W[n][k] with M = T + k token rows
// (<= 144) against a large bf16 weight matrix that is read exactly once.
//
// Operand roles are swapped relative to a usual GEMM: the 64 weight rows of a tile are the
// MMA "M" dimension and the token rows are the MMA "N" dimension, so the weight stream
// determines the tile and the few token rows ride along.  Each CTA owns one 64-row weight
// tile (optionally one split of K), streams it through a multi-stage cp.async pipeline with
// 128-byte rows (XOR-swizzled 16-byte chunks), accumulates in fp32 on the tensor cores and
// hands the tile to a fused epilogue through shared memory.
//
// A tile may be "paired": rows [base, base+32) and [base+pair_off, base+pair_off+32).  This puts
// both members of a rotary pair (c, c + dh/2), or a gate row and its up row, in one CTA, so RoPE
// and SwiGLU are applied in the epilogue without touching the weight layout.
#include "firp_kernels.cuh"
#include "gemm_epilogue.cuh"

namespace firp {

namespace {

constexpr int BN = kGemmBN;   // weight rows per tile
constexpr int BK = kGemmBK;   // k per stage (128 bytes of bf16)
constexpr int kThreads = 128; // 4 warps, each owns 16 weight rows

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async_16(uint32_t dst, const void *src, bool valid) {
  const int sz = valid ? 16 : 0;   // src-size 0 => the 16 bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(sz));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float *c, const uint32_t *a, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// MT = number of 8-token MMA n-tiles (token rows padded to MT*8)
template <int MT, int EPI, int STAGES>
__global__ void __launch_bounds__(kThreads)
gemm_skinny_mma_kernel(GemmArgs a, TileMap tm, int splits) {
  constexpr int MT2 = (MT + 1) / 2;                 // ldmatrix.x4 covers two n-tiles
  constexpr int XROWS = MT2 * 16;
  constexpr int W_BYTES = BN * 128, X_BYTES = XROWS * 128, STAGE_BYTES = W_BYTES + 2 * X_BYTES;   // W, X hi, X lo
  extern __shared__ __align__(128) uint8_t smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tile = blockIdx.x, split = blockIdx.y;
  const int kb_total = (a.K + BK - 1) / BK;
  const int kb_per = (kb_total + splits - 1) / splits;
  const int kb0 = split * kb_per, kb1 = min(kb_total, kb0 + kb_per);
  const int nkb = max(kb1 - kb0, 0);

  // per-thread load assignment: 16-byte chunks; a 128-byte row has 8 chunks
  auto load_stage = [&](int stage, int kb) {
    uint8_t *ws = smem + stage * STAGE_BYTES, *xs = ws + W_BYTES;
    const int k0 = kb * BK;
    for (int ch = tid; ch < BN * 8; ch += kThreads) {
      const int r = ch >> 3, c = ch & 7;
      bool valid;
      const int n = tile_row<BN>(tm, tile, r, a.N, valid);
      valid = valid && (k0 + c * 8 < a.K);
      const bf16 *src = valid ? a.W + (size_t)n * a.K + k0 + c * 8 : a.W;
      cp_async_16(smem_u32(ws + r * 128 + ((c ^ (r & 7)) << 4)), src, valid);
    }
    for (int ch = tid; ch < MT * 8 * 8; ch += kThreads) {
      const int r = ch >> 3, c = ch & 7;
      const bool valid = (r < a.R) && (k0 + c * 8 < a.K);
      const bf16 *src = valid ? a.X + (size_t)r * a.K + k0 + c * 8 : a.X;
      cp_async_16(smem_u32(xs + r * 128 + ((c ^ (r & 7)) << 4)), src, valid);
      cp_async_16(smem_u32(xs + X_BYTES + r * 128 + ((c ^ (r & 7)) << 4)), valid ? src + a.x_lo_off : a.X, valid);
    }
  };

  float acc[MT][4];
#pragma unroll
  for (int i = 0; i < MT; ++i) { acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f; }

#pragma unroll
  for (int s = 0; s < STAGES - 1; ++s) {
    if (s < nkb) load_stage(s, kb0 + s);
    cp_async_commit();
  }
  for (int it = 0; it < nkb; ++it) {
    cp_async_wait<STAGES - 2>();
    __syncthreads();
    if (it + STAGES - 1 < nkb) load_stage((it + STAGES - 1) % STAGES, kb0 + it + STAGES - 1);
    cp_async_commit();
    const uint8_t *ws = smem + (it % STAGES) * STAGE_BYTES, *xs = ws + W_BYTES;
    const int mi = lane >> 3, r8 = lane & 7;
#pragma unroll
    for (int kk = 0; kk < BK / 16; ++kk) {
      uint32_t af[4];
      {
        const int row = warp * 16 + (mi & 1) * 8 + r8, chunk = kk * 2 + (mi >> 1);
        ldmatrix_x4(af[0], af[1], af[2], af[3], smem_u32(ws + row * 128 + ((chunk ^ (row & 7)) << 4)));
      }
#pragma unroll
      for (int p = 0; p < MT2; ++p) {
        uint32_t b0, b1, b2, b3;
        const int row = p * 16 + (mi >> 1) * 8 + r8, chunk = kk * 2 + (mi & 1);
        const int off = row * 128 + ((chunk ^ (row & 7)) << 4);
        ldmatrix_x4(b0, b1, b2, b3, smem_u32(xs + off));             // hi halves
        mma_bf16(acc[2 * p], af, b0, b1);
        if (2 * p + 1 < MT) mma_bf16(acc[2 * p + 1], af, b2, b3);
        ldmatrix_x4(b0, b1, b2, b3, smem_u32(xs + X_BYTES + off));   // lo halves, same accumulators
        mma_bf16(acc[2 * p], af, b0, b1);
        if (2 * p + 1 < MT) mma_bf16(acc[2 * p + 1], af, b2, b3);
      }
    }
  }
  cp_async_wait<0>();
  __syncthreads();

  // stage the fp32 tile: C[token][weight row]
  constexpr int LDC = BN + 1;
  float *C = reinterpret_cast<float *>(smem);
  {
    const int g = lane >> 2, t4 = lane & 3;
#pragma unroll
    for (int nt = 0; nt < MT; ++nt) {
      const int m0 = nt * 8 + t4 * 2, col = warp * 16 + g;
      C[m0 * LDC + col] = acc[nt][0];
      C[(m0 + 1) * LDC + col] = acc[nt][1];
      C[m0 * LDC + col + 8] = acc[nt][2];
      C[(m0 + 1) * LDC + col + 8] = acc[nt][3];
    }
  }
  __syncthreads();
  gemm_epilogue<EPI, BN>(C, LDC, tile, split, a, tm, tid, kThreads);
}

// split-K factor of the residual GEMMs: enough CTAs to cover the SMs about twice, at least
// 8 k-blocks per split, and no empty split
int split_k(int N, int K) {
  const int tiles = (N + BN - 1) / BN, kb = (K + BK - 1) / BK;
  int s = (2 * 148 + tiles - 1) / tiles;
  s = s < 1 ? 1 : (s > 8 ? 8 : s);
  while (s > 1 && kb / s < 8) --s;
  const int per = (kb + s - 1) / s;
  return (kb + per - 1) / per;
}

template <int MT, int EPI>
cudaError_t launch_mt(const GemmArgs &a, const TileMap &tm, int tiles, cudaStream_t st) {
  constexpr int MT2 = (MT + 1) / 2;
  constexpr int STAGE_BYTES = BN * 128 + 2 * MT2 * 16 * 128;
  constexpr int STAGES = (MT <= 5) ? 5 : (MT <= 9 ? 4 : 3);
  constexpr int C_BYTES = MT * 8 * (BN + 1) * 4;
  constexpr int SMEM = (STAGES * STAGE_BYTES > C_BYTES) ? STAGES * STAGE_BYTES : C_BYTES;
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(gemm_skinny_mma_kernel<MT, EPI, STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
    configured = true;
  }
  const int splits = (EPI == EPI_RESIDUAL) ? split_k(a.N, a.K) : 1;
  gemm_skinny_mma_kernel<MT, EPI, STAGES><<<dim3(tiles, splits), kThreads, SMEM, st>>>(a, tm, splits);
  return cudaGetLastError();
}

template <int EPI>
cudaError_t launch_epi(const GemmArgs &a, const TileMap &tm, int tiles, cudaStream_t st) {
  const int mt = (a.R + 7) / 8;
  if (mt <= 2) return launch_mt<2, EPI>(a, tm, tiles, st);
  if (mt <= 5) return launch_mt<5, EPI>(a, tm, tiles, st);
  if (mt <= 9) return launch_mt<9, EPI>(a, tm, tiles, st);
  return launch_mt<18, EPI>(a, tm, tiles, st);
}

}  // namespace

cudaError_t launch_gemm_mma(GemmEpilogue epi, const GemmArgs &a, cudaStream_t st) {
  TileMap tm{};
  switch (epi) {
    case EPI_QKV_ROPE: {
      const int half = a.dh / 2;
      tm.paired = 1; tm.tiles_per_unit = (half + 31) / 32; tm.unit_stride = a.dh; tm.pair_off = half; tm.group_rows = half;
      return launch_epi<EPI_QKV_ROPE>(a, tm, (a.H + 2 * a.Hkv) * tm.tiles_per_unit, st);
    }
    case EPI_SWIGLU:
      tm.paired = 1; tm.tiles_per_unit = (a.F + 31) / 32; tm.unit_stride = 0; tm.pair_off = a.F; tm.group_rows = a.F;
      return launch_epi<EPI_SWIGLU>(a, tm, tm.tiles_per_unit, st);
    case EPI_LOGITS:
      return launch_epi<EPI_LOGITS>(a, tm, (a.N + BN - 1) / BN, st);
    default:
      return launch_epi<EPI_RESIDUAL>(a, tm, (a.N + BN - 1) / BN, st);
  }
}

cudaError_t launch_gemm(GemmEpilogue epi, const GemmArgs &a, bool use_tc, bool pdl, cudaStream_t st, StreamK *sk_out) {
  if (use_tc) return launch_gemm_tc(epi, a, pdl, st, sk_out);
  if (sk_out) *sk_out = StreamK{0, 1, 1};   // the mma.sync kernel adds into the residual stream itself
  return launch_gemm_mma(epi, a, st);
}

}  // namespace firp
