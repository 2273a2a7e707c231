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

// Tile geometry: which global weight row a tile-local row maps to.
struct TileMap {
  int paired;          // 0: rows tile*64 + i;  1: two 32-row groups pair_off apart
  int tiles_per_unit;  // paired: 32-row tiles per unit (a head, or the whole gate matrix)
  int unit_stride;     // paired: rows between units
  int pair_off;        // paired: distance between the two groups
  int group_rows;      // paired: valid rows per group within a unit (dh/2, or F)
};

__device__ __forceinline__ int tile_row(const TileMap &tm, int tile, int i, int N, bool &valid) {
  if (!tm.paired) {
    const int r = tile * BN + i;
    valid = r < N;
    return r;
  }
  const int unit = tile / tm.tiles_per_unit, sub = tile % tm.tiles_per_unit;
  const int grp = i >> 5, w = sub * 32 + (i & 31);
  valid = w < tm.group_rows;
  return unit * tm.unit_stride + grp * tm.pair_off + w;
}

// ---- epilogues: C is the fp32 tile in shared memory, C[m * ldc + col], col = tile-local weight row
template <int EPI>
__device__ __forceinline__ void epilogue(const float *C, int ldc, int tile, int split, const GemmArgs &a,
                                         const TileMap &tm) {
  const int tid = threadIdx.x;
  if (EPI == EPI_PARTIAL) {
    float *out = a.partial + (size_t)split * a.partial_stride;
    for (int idx = tid; idx < a.R * BN; idx += kThreads) {
      const int m = idx / BN, col = idx % BN, n = tile * BN + col;
      if (n < a.N) out[(size_t)m * a.N + n] = C[m * ldc + col];
    }
  } else if (EPI == EPI_LOGITS) {
    for (int idx = tid; idx < a.R * BN; idx += kThreads) {
      const int m = idx / BN, col = idx % BN, n = tile * BN + col;
      if (n < a.N) a.logits[(size_t)m * a.N + n] = C[m * ldc + col];
    }
  } else if (EPI == EPI_SWIGLU) {
    for (int idx = tid; idx < a.R * 32; idx += kThreads) {
      const int m = idx >> 5, i = idx & 31, j = tile * 32 + i;
      if (j < a.F) {
        const float g = C[m * ldc + i], u = C[m * ldc + 32 + i];
        a.y[(size_t)m * a.F + j] = __float2bfloat16(g / (1.f + __expf(-g)) * u);
      }
    }
  } else {  // EPI_QKV_ROPE
    const int half = a.dh >> 1;
    const int unit = tile / tm.tiles_per_unit, c0 = (tile % tm.tiles_per_unit) * 32;
    for (int idx = tid; idx < a.R * 32; idx += kThreads) {
      const int m = idx >> 5, i = idx & 31, c = c0 + i;
      const int s = m / a.rw.Ms, v = m % a.rw.Ms;
      if (c >= half || v >= a.rows_active) continue;
      float x1 = C[m * ldc + i], x2 = C[m * ldc + 32 + i];
      if (unit < a.H + a.Hkv) {   // queries and keys are rotated at the row's tree position
        const float2 cs = a.rope[(size_t)m * half + c];
        const float y1 = x1 * cs.x - x2 * cs.y, y2 = x2 * cs.x + x1 * cs.y;
        x1 = y1; x2 = y2;
      }
      if (unit < a.H) {
        bf16 *dst = a.q + (size_t)m * a.H * a.dh + unit * a.dh + c;
        dst[0] = __float2bfloat16(x1); dst[half] = __float2bfloat16(x2);
      } else {
        const int is_v = unit >= a.H + a.Hkv;
        const int kvh = unit - a.H - (is_v ? a.Hkv : 0);
        const int slot = a.seq_ids[s];
        const int p = a.ctx_len[slot] + v;
        if (p < a.max_ctx) {
          bf16 *dst = a.kcache + (size_t)slot * a.seq_stride + (is_v ? a.kv_stride : 0) +
                      ((size_t)p * a.Hkv + kvh) * a.dh + c;
          dst[0] = __float2bfloat16(x1); dst[half] = __float2bfloat16(x2);
        }
      }
    }
  }
}

// MT = number of 8-token MMA n-tiles (token rows padded to MT*8)
template <int MT, int EPI, int STAGES>
__global__ void __launch_bounds__(kThreads)
gemm_skinny_mma_kernel(GemmArgs a, TileMap tm) {
  constexpr int MT2 = (MT + 1) / 2;                 // ldmatrix.x4 covers two n-tiles
  constexpr int XROWS = MT2 * 16;
  constexpr int W_BYTES = BN * 128, X_BYTES = XROWS * 128, STAGE_BYTES = W_BYTES + X_BYTES;
  extern __shared__ __align__(128) uint8_t smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tile = blockIdx.x, split = blockIdx.y;
  const int kb_total = (a.K + BK - 1) / BK;
  const int kb_per = (kb_total + a.splits - 1) / a.splits;
  const int kb0 = split * kb_per, kb1 = min(kb_total, kb0 + kb_per);
  const int nkb = max(kb1 - kb0, 0);

  // per-thread load assignment: 16-byte chunks; a 128-byte row has 8 chunks
  auto load_stage = [&](int stage, int kb) {
    uint8_t *ws = smem + stage * STAGE_BYTES, *xs = ws + W_BYTES;
    const int k0 = kb * BK;
    for (int ch = tid; ch < BN * 8; ch += kThreads) {
      const int r = ch >> 3, c = ch & 7;
      bool valid;
      const int n = tile_row(tm, tile, r, a.N, valid);
      valid = valid && (k0 + c * 8 < a.K);
      const bf16 *src = valid ? a.W + (size_t)n * a.K + k0 + c * 8 : a.W;
      cp_async_16(smem_u32(ws + r * 128 + ((c ^ (r & 7)) << 4)), src, valid);
    }
    for (int ch = tid; ch < MT * 8 * 8; ch += kThreads) {
      const int r = ch >> 3, c = ch & 7;
      const bool valid = (r < a.R) && (k0 + c * 8 < a.K);
      const bf16 *src = valid ? a.X + (size_t)r * a.K + k0 + c * 8 : a.X;
      cp_async_16(smem_u32(xs + r * 128 + ((c ^ (r & 7)) << 4)), src, valid);
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
        ldmatrix_x4(b0, b1, b2, b3, smem_u32(xs + row * 128 + ((chunk ^ (row & 7)) << 4)));
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
  epilogue<EPI>(C, LDC, tile, split, a, tm);
}

template <int MT, int EPI>
void launch_mt(const GemmArgs &a, const TileMap &tm, int tiles, cudaStream_t st) {
  constexpr int MT2 = (MT + 1) / 2;
  constexpr int STAGE_BYTES = BN * 128 + MT2 * 16 * 128;
  constexpr int STAGES = (MT <= 5) ? 6 : (MT <= 9 ? 5 : 4);
  constexpr int C_BYTES = MT * 8 * (BN + 1) * 4;
  constexpr int SMEM = (STAGES * STAGE_BYTES > C_BYTES) ? STAGES * STAGE_BYTES : C_BYTES;
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(gemm_skinny_mma_kernel<MT, EPI, STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
    configured = true;
  }
  const int splits = (EPI == EPI_PARTIAL) ? a.splits : 1;
  GemmArgs b = a;
  b.splits = splits;
  gemm_skinny_mma_kernel<MT, EPI, STAGES><<<dim3(tiles, splits), kThreads, SMEM, st>>>(b, tm);
}

template <int EPI>
void launch_epi(const GemmArgs &a, const TileMap &tm, int tiles, cudaStream_t st) {
  const int mt = (a.R + 7) / 8;
  if (mt <= 2) launch_mt<2, EPI>(a, tm, tiles, st);
  else if (mt <= 5) launch_mt<5, EPI>(a, tm, tiles, st);
  else if (mt <= 9) launch_mt<9, EPI>(a, tm, tiles, st);
  else launch_mt<18, EPI>(a, tm, tiles, st);
}

}  // namespace

int gemm_split_k(int N, int K) {
  // enough CTAs to cover the SMs about twice, but at least 8 k-blocks per split
  const int tiles = (N + BN - 1) / BN, kb = (K + BK - 1) / BK;
  int s = (2 * 148 + tiles - 1) / tiles;
  s = s < 1 ? 1 : s;
  while (s > 1 && kb / s < 8) --s;
  return s > 8 ? 8 : s;
}

void launch_gemm(GemmEpilogue epi, const GemmArgs &a, cudaStream_t st) {
  TileMap tm{};
  int tiles;
  switch (epi) {
    case EPI_QKV_ROPE: {
      const int half = a.dh / 2;
      tm.paired = 1; tm.tiles_per_unit = (half + 31) / 32; tm.unit_stride = a.dh; tm.pair_off = half; tm.group_rows = half;
      tiles = (a.H + 2 * a.Hkv) * tm.tiles_per_unit;
      launch_epi<EPI_QKV_ROPE>(a, tm, tiles, st);
      break;
    }
    case EPI_SWIGLU:
      tm.paired = 1; tm.tiles_per_unit = (a.F + 31) / 32; tm.unit_stride = 0; tm.pair_off = a.F; tm.group_rows = a.F;
      tiles = tm.tiles_per_unit;
      launch_epi<EPI_SWIGLU>(a, tm, tiles, st);
      break;
    case EPI_LOGITS:
      tiles = (a.N + BN - 1) / BN;
      launch_epi<EPI_LOGITS>(a, tm, tiles, st);
      break;
    default:
      tiles = (a.N + BN - 1) / BN;
      launch_epi<EPI_PARTIAL>(a, tm, tiles, st);
      break;
  }
}

}  // namespace firp
