// Tree-masked split-KV decode attention as a kernel of its own (the tile loop lives in attn_device.cuh).
// Grid = (kv split, kv head, sequence x query block); the CTAs of one (kv head, query block) form a
// thread-block cluster.  Each split leaves its unnormalised (running max, sum, O) in its own shared memory;
// after a cluster barrier every CTA merges a share of the query rows by reading its peers' partials through
// distributed shared memory and writes the final rows, so there is no second kernel and the merge order is
// fixed.
#include <cooperative_groups.h>

#include <cstdlib>

#include "attn_device.cuh"
#include "firp_kernels.cuh"
#include "launch_util.cuh"

namespace cg = cooperative_groups;

namespace firp {

namespace {


template <int DH>
__global__ void __launch_bounds__(kAttnThreads) tree_attn_kernel(AttnArgs a, int pdl) {
  extern __shared__ __align__(128) uint8_t smem[];
  constexpr int Q_BYTES = kAttnQRows * DH * 2;
  __shared__ uint32_t s_mask[kAttnQRows][kMaskWords];
  __shared__ int s_row[kAttnQRows];                     // global row index of each query row, -1 = padding
  __shared__ float s_m[kAttnQRows], s_l[kAttnQRows];        // this split's running max (log2 units) and sum per query row
  if (pdl) { griddep_launch(); griddep_wait(); }

  const int tid = threadIdx.x;
  const int kvh = blockIdx.y;
  const int G = a.H / a.Hkv;
  const int qrows_total = a.rows_active * G;
  const int qblocks = (qrows_total + kAttnQRows - 1) / kAttnQRows;
  const int s = blockIdx.z / qblocks, qb = blockIdx.z % qblocks;
  float *sO = reinterpret_cast<float *>(smem + 2 * Q_BYTES);        // [kAttnQRows][DH], over the key tiles
  attn_split_item<DH, AttnCtaSync>(a, smem, s_mask, s_row, tid, s, kvh, qb, blockIdx.x, a.splits, s_m, s_l, sO);
  // merge: o = sum_s 2^(m_s - M) O_s / sum_s 2^(m_s - M) l_s; CTA `rank` finalises rows rank, rank + splits, ...
  cg::cluster_group cluster = cg::this_cluster();
  cluster.sync();
  const int rank = (int)cluster.block_rank(), nsp = (int)cluster.num_blocks();
  // a thread finalises 4 neighbouring dims of a row; rows rank, rank + nsp, ... belong to this CTA
  constexpr int TPR = DH / 4, RP = kAttnThreads / TPR;  // threads per row, rows per pass
  const int c4 = (tid % TPR) * 4, sub = tid / TPR;
  for (int q0 = 0; rank + q0 * nsp < kAttnQRows; q0 += 2 * RP) {     // two passes at a time: 16 remote float4 loads in flight
    float4 ov[2][kAttnMaxSplits];
    float pm[2][kAttnMaxSplits], pl[2][kAttnMaxSplits];   // every split's (max, sum) of the row, fetched with its O
    int row[2];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int i = rank + (q0 + u * RP + sub) * nsp;
      row[u] = (i < kAttnQRows && qb * kAttnQRows + i < qrows_total) ? i : -1;
#pragma unroll
      for (int sp = 0; sp < kAttnMaxSplits; ++sp) {
        const bool on = row[u] >= 0 && sp < nsp;
        ov[u][sp] = on ? *reinterpret_cast<const float4 *>(cluster.map_shared_rank(sO + row[u] * DH + c4, sp))
                       : make_float4(0.f, 0.f, 0.f, 0.f);
        pm[u][sp] = on ? *cluster.map_shared_rank(&s_m[row[u]], sp) : -INFINITY;
        pl[u][sp] = on ? *cluster.map_shared_rank(&s_l[row[u]], sp) : 0.f;
      }
    }
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int i = row[u];
      if (i < 0) continue;
      float M = -INFINITY;
#pragma unroll
      for (int sp = 0; sp < kAttnMaxSplits; ++sp) M = fmaxf(M, pm[u][sp]);
      float L = 0.f;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int sp = 0; sp < kAttnMaxSplits; ++sp) {
        if (pm[u][sp] != -INFINITY) {
          const float w = exp2f(pm[u][sp] - M);
          L += w * pl[u][sp];
          acc.x += w * ov[u][sp].x; acc.y += w * ov[u][sp].y; acc.z += w * ov[u][sp].z; acc.w += w * ov[u][sp].w;
        }
      }
      const float inv = (L > 0.f) ? 1.f / L : 0.f;
      const float val[4] = {acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv};
      const int qr = qb * kAttnQRows + i;
      const int r = s * a.rw.Ms + qr / G, head = kvh * G + qr % G;
      const __nv_bfloat162 h01 = __floats2bfloat162_rn(val[0], val[1]), h23 = __floats2bfloat162_rn(val[2], val[3]);
      const float2 f01 = __bfloat1622float2(h01), f23 = __bfloat1622float2(h23);
      const __nv_bfloat162 l01 = __floats2bfloat162_rn(val[0] - f01.x, val[1] - f01.y);
      const __nv_bfloat162 l23 = __floats2bfloat162_rn(val[2] - f23.x, val[3] - f23.y);
      const size_t idx = ((size_t)r * a.H + head) * DH + c4;
      *reinterpret_cast<uint2 *>(a.o + idx) =
          make_uint2(*reinterpret_cast<const uint32_t *>(&h01), *reinterpret_cast<const uint32_t *>(&h23));
      *reinterpret_cast<uint2 *>(a.o + a.o_lo_off + idx) =
          make_uint2(*reinterpret_cast<const uint32_t *>(&l01), *reinterpret_cast<const uint32_t *>(&l23));
    }
  }
  cluster.sync();                                   // peers may still be reading this CTA's partials
}

template <int DH> cudaError_t launch_dh(const AttnArgs &a, bool pdl, cudaStream_t st) {
  constexpr int SMEM = attn_smem_bytes<DH>();
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(tree_attn_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  const int G = a.H / a.Hkv;
  const int qblocks = (a.rows_active * G + kAttnQRows - 1) / kAttnQRows;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(a.splits, a.Hkv, a.rw.n_seq * qblocks);
  cfg.blockDim = dim3(kAttnThreads);
  cfg.dynamicSmemBytes = SMEM;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = a.splits; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, tree_attn_kernel<DH>, a, pdl ? 1 : 0);
}

}  // namespace

int attention_splits(int groups, int kv_tiles) {
  // CTAs of one (kv head, query block) = one cluster (<= 8): about two CTAs per SM over the whole grid,
  // never more splits than 64-position tiles
  const int budget = 296;
  int s = 1;
  while (s < kAttnMaxSplits && 2 * s * groups <= budget && 2 * s <= kv_tiles) s *= 2;
  return s;
}

cudaError_t launch_attention(const AttnArgs &a, bool pdl, cudaStream_t st) {
  return a.dh == 128 ? launch_dh<128>(a, pdl, st) : launch_dh<64>(a, pdl, st);
}

}  // namespace firp
