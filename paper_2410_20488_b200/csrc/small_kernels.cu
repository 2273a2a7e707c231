// Small kernels of the FIRP step: tree bookkeeping, embedding, residual-add + RMSNorm,
// the pseudo-hidden projection (Eq. 3), top-B, the acceptance walk / next tree, KV compaction.
#include "firp_kernels.cuh"
#include "launch_util.cuh"
#include "norm_device.cuh"


namespace firp {

// ---------------------------------------------------------------------------
// Tree prep (Section 3.4 "Tree attention"; Section 3.3 for the pseudo rows):
// depth, absolute position, ancestor-or-self bitmask, rotary table.
// One CTA per sequence; the extended parent array lives in shared memory.
// ---------------------------------------------------------------------------
__global__ void tree_prep_kernel(Rows rw, const int32_t *parents, int parents_stride, const int32_t *seq_ids,
                                 const int32_t *ctx_len, int dh, float theta, TreeMeta meta,
                                 int32_t *out_depth, uint32_t *out_mask, int out_mask_words, unsigned *zero_word, int pdl) {
  __shared__ int32_t ext[kMaxTreeRows];
  __shared__ int32_t sdepth[kMaxTreeRows];
  if (pdl) { griddep_launch(); griddep_wait(); }
  const int s = blockIdx.x, tid = threadIdx.x;
  if (zero_word && s == 0 && tid == 0) *zero_word = 0u;
  const int n = ctx_len[seq_ids[s]];
  for (int v = tid; v < rw.Ms; v += blockDim.x) {
    int p;
    if (v < rw.T) p = parents[s * parents_stride + v];     // stride 0: one template for every sequence
    else if (rw.chains) p = v - rw.T;   // step 1 of node u (row T + u) hangs off u, step i off step i-1 of the same node
    else p = (v == rw.T) ? rw.anchor : v - 1;
    ext[v] = p;
  }
  __syncthreads();
  for (int v = tid; v < rw.Ms; v += blockDim.x) {
    uint32_t bits[kMaskWords];
#pragma unroll
    for (int w = 0; w < kMaskWords; ++w) bits[w] = 0u;
    int dep = -1;
    int u = v;
    for (int it = 0; it < rw.Ms && u >= 0; ++it) {   // parents[u] < u, so at most Ms hops
      if (!(rw.masked && u >= rw.T && u != v)) {     // "Masked": other pseudo rows stay invisible, depth still counts them
#pragma unroll
        for (int w = 0; w < kMaskWords; ++w) if ((u >> 5) == w) bits[w] |= 1u << (u & 31);
      }
      ++dep;
      u = ext[u];
    }
    sdepth[v] = dep;
    const int r = s * rw.Ms + v;
    meta.depth[r] = dep;
    meta.pos[r] = n + dep;
#pragma unroll
    for (int w = 0; w < kMaskWords; ++w) meta.mask[(size_t)r * kMaskWords + w] = bits[w];
    if (out_depth) out_depth[r] = dep;
    if (out_mask)
      for (int w = 0; w < out_mask_words; ++w) out_mask[(size_t)r * out_mask_words + w] = bits[w];
  }
  __syncthreads();
  const int half = dh / 2;
  const double l2t = log2((double)theta);
  for (int i = tid; i < rw.Ms * half; i += blockDim.x) {
    const int v = i / half, c = i % half;
    const double inv_freq = exp2(-2.0 * (double)c / (double)dh * l2t);
    const double ang = (double)(n + sdepth[v]) * inv_freq;
    double sn, cs;
    sincos(ang, &sn, &cs);
    meta.rope[(size_t)(s * rw.Ms + v) * half + c] = make_float2((float)cs, (float)sn);
  }
}

void launch_tree_prep(const Rows &rw, const int32_t *d_parents, int parents_stride, const int32_t *d_seq_ids, const int32_t *d_ctx_len,
                      int dh, float theta, TreeMeta meta, int32_t *out_depth, uint32_t *out_mask, int out_mask_words,
                      unsigned *zero_word, bool pdl, cudaStream_t st) {
  launch_k(tree_prep_kernel, dim3(rw.n_seq), dim3(256), 0, st, pdl, rw, d_parents, parents_stride, d_seq_ids, d_ctx_len, dh, theta, meta,
           out_depth, out_mask, out_mask_words, zero_word, pdl ? 1 : 0);
}

// ---------------------------------------------------------------------------
// Embedding gather: fp32 residual rows from bf16 table rows; pseudo rows start at zero.
// ---------------------------------------------------------------------------
__global__ void embed_kernel(Rows rw, const int32_t *tokens, const bf16 *__restrict__ embed, int d,
                             int vocab, float *h, int pdl) {
  if (pdl) { griddep_launch(); griddep_wait(); }
  const int r = blockIdx.x, s = r / rw.Ms, v = r % rw.Ms;
  float *dst = h + (size_t)r * d;
  if (v >= rw.T) {
    for (int c = threadIdx.x; c < d; c += blockDim.x) dst[c] = 0.f;
    return;
  }
  int tok = tokens[s * rw.T + v];
  tok = min(max(tok, 0), vocab - 1);
  const bf16 *src = embed + (size_t)tok * d;
  for (int c = threadIdx.x * 2; c < d; c += blockDim.x * 2) {
    const __nv_bfloat162 p = *reinterpret_cast<const __nv_bfloat162 *>(src + c);
    *reinterpret_cast<float2 *>(dst + c) = __bfloat1622float2(p);
  }
}

void launch_embed(const Rows &rw, const int32_t *d_tokens, const bf16 *embed, int d, int vocab, float *h, bool pdl,
                  cudaStream_t st) {
  launch_k(embed_kernel, dim3(rw.R), dim3(128), 0, st, pdl, rw, d_tokens, embed, d, vocab, h, pdl ? 1 : 0);
}

// ---------------------------------------------------------------------------
// Residual update + first half of RMSNorm, as a flat elementwise kernel.
//   h[r] += the partial tiles a residual GEMM left in scratch (fixed order: ascending CTA index)
//   x[r]  = h[r] * g as bf16 planes (hi, lo; plus a third plane on request) -- NOT yet divided by the row's RMS
//   ss[r][w] = sum of h[r][c]^2 over the 128 columns of warp w
// The division by sqrt(mean(h^2) + eps) commutes with the GEMM that consumes x, so that GEMM's
// finisher applies it to the fp32 sums (it adds the ss[r][*] in a fixed order).  This kernel then
// has no reduction across threads beyond a warp, no barrier, and every thread is independent.
// A thread owns 4 neighbouring columns of one row; d must be a multiple of 128.
// ---------------------------------------------------------------------------
constexpr int kNormThreads = 256;

__global__ void __launch_bounds__(kNormThreads)
rmsnorm_kernel(Rows rw, int v0, int nv, float *h, Partials pend, const bf16 *__restrict__ g, int d, bf16 *x,
               size_t x_lo_off, int planes, float *ss, int pdl) {
  if (pdl) { griddep_launch(); griddep_wait(); }
  rmsnorm_item(rw, v0, nv, h, pend, g, d, x, x_lo_off, planes, ss, blockIdx.x * kNormThreads + threadIdx.x);
}

cudaError_t launch_rmsnorm(const Rows &rw, int v0, int v1, float *h, const Partials &pending, const bf16 *g, int d,
                           bf16 *x, size_t x_lo_off, int planes, float *ss, bool pdl, cudaStream_t st) {
  const int nv = v1 - v0;
  if (nv <= 0) return cudaSuccess;
  const int threads = rw.n_seq * nv * (d >> 2);
  return launch_k(rmsnorm_kernel, dim3((threads + kNormThreads - 1) / kNormThreads), dim3(kNormThreads), 0, st, pdl, rw,
                  v0, nv, h, pending, g, d, x, x_lo_off, planes, ss, pdl ? 1 : 0);
}

// ---------------------------------------------------------------------------
// Pseudo hidden states, Eq. 3: h~_i = W_i h[anchor] + b_i on the raw fp32 residual stream.  The k maps are
// one [k d][d] weight matrix for the stream-K GEMM; this kernel prepares its operand: the anchor row of every
// sequence, untouched by any norm, as (hi, lo) bf16 planes in row s of xp.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
root_split_kernel(Rows rw, const float *h, const bf16 *g, int d, bf16 *xp, size_t xp_lo_off, int pdl) {
  if (pdl) { griddep_launch(); griddep_wait(); }
  root_split_item(rw, h, g, d, xp, xp_lo_off, blockIdx.x * 256 + threadIdx.x);
}

void launch_root_split(const Rows &rw, const float *h, const bf16 *g, int d, bf16 *xp, size_t xp_lo_off, bool pdl, cudaStream_t st) {
  const int threads = rw.n_seq * (rw.chains ? rw.T : 1) * (d >> 2);
  launch_k(root_split_kernel, dim3((threads + 255) / 256), dim3(256), 0, st, pdl, rw, h, g, d, xp, xp_lo_off, pdl ? 1 : 0);
}

// ---------------------------------------------------------------------------
// Top-B of each logits row by (value descending, id ascending), in two passes of one kernel:
//   pass 1  every (row, segment of kTopSeg logits) leaves its B best as candidates in scratch
//   pass 2  every row picks its B best among its candidates
// Selecting by the same total order in both passes gives exactly the top-B of the whole row.
// ---------------------------------------------------------------------------
constexpr int kTopThreads = 256;

__device__ __forceinline__ bool better(float va, int ia, float vb, int ib) { return va > vb || (va == vb && ia < ib); }

// grid = (segments, rows).  Element t of the segment has value vals[row * row_stride + seg * seg_len + t] and
// id ids[same index] (ids == NULL: its position in the row).  Output slot (row * segments + seg) gets B pairs;
// a segment with fewer than B elements pads with (-inf, INT_MAX).
__global__ void __launch_bounds__(kTopThreads)
topb_kernel(const float *vals, const int32_t *ids, int row_stride, int seg_len, int row_len, int B, int32_t *out_ids,
            float *out_vals, int pdl) {
  __shared__ float sval[32];
  __shared__ int sid[32];
  __shared__ int swin;
  if (pdl) { griddep_launch(); griddep_wait(); }
  const int seg = blockIdx.x, r = blockIdx.y;
  const size_t base = (size_t)r * row_stride + (size_t)seg * seg_len;
  const int n = min(seg_len, row_len - seg * seg_len);
  float lv[kMaxTopB];
  int li[kMaxTopB];
#pragma unroll
  for (int j = 0; j < kMaxTopB; ++j) { lv[j] = -INFINITY; li[j] = 0x7fffffff; }
  for (int t = threadIdx.x; t < n; t += kTopThreads) {
    const float v = vals[base + t];
    const int id = ids ? ids[base + t] : seg * seg_len + t;
    if (better(v, id, lv[kMaxTopB - 1], li[kMaxTopB - 1])) {
      lv[kMaxTopB - 1] = v; li[kMaxTopB - 1] = id;
#pragma unroll
      for (int j = kMaxTopB - 1; j > 0; --j) {
        if (better(lv[j], li[j], lv[j - 1], li[j - 1])) {
          const float tv = lv[j]; lv[j] = lv[j - 1]; lv[j - 1] = tv;
          const int ti = li[j]; li[j] = li[j - 1]; li[j - 1] = ti;
        }
      }
    }
  }
  const size_t o = ((size_t)r * gridDim.x + seg) * B;
  int head = 0;
  for (int b = 0; b < B; ++b) {
    float cv = -INFINITY; int ci = 0x7fffffff;
#pragma unroll
    for (int j = 0; j < kMaxTopB; ++j) if (j == head) { cv = lv[j]; ci = li[j]; }
    float bv = cv; int bi = ci;
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, s);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, s);
      if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
    }
    if ((threadIdx.x & 31) == 0) { sval[threadIdx.x >> 5] = bv; sid[threadIdx.x >> 5] = bi; }
    __syncthreads();
    if (threadIdx.x < 32) {
      float v = (threadIdx.x < kTopThreads / 32) ? sval[threadIdx.x] : -INFINITY;
      int i = (threadIdx.x < kTopThreads / 32) ? sid[threadIdx.x] : 0x7fffffff;
#pragma unroll
      for (int s = 16; s > 0; s >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, v, s);
        const int oi = __shfl_xor_sync(0xffffffffu, i, s);
        if (better(ov, oi, v, i)) { v = ov; i = oi; }
      }
      if (threadIdx.x == 0) {
        swin = i;
        out_ids[o + b] = i;
        out_vals[o + b] = v;
      }
    }
    __syncthreads();
    if (ci == swin && ci != 0x7fffffff && head < kMaxTopB) ++head;   // ids are unique: exactly one thread advances
    __syncthreads();
  }
}

int topb_segments(int V) { return (V + kTopSeg - 1) / kTopSeg; }

void launch_topb(const float *logits, int R, int V, int B, int32_t *cand_ids, float *cand_vals, int32_t *ids, float *vals,
                 bool pdl, cudaStream_t st) {
  const int segs = topb_segments(V);
  launch_k(topb_kernel, dim3(segs, R), dim3(kTopThreads), 0, st, pdl, logits, (const int32_t *)nullptr, V, kTopSeg, V, B,
           cand_ids, cand_vals, pdl ? 1 : 0);
  launch_k(topb_kernel, dim3(1, R), dim3(kTopThreads), 0, st, pdl, (const float *)cand_vals, (const int32_t *)cand_ids,
           segs * B, segs * B, segs * B, B, ids, vals, pdl ? 1 : 0);
}

// ---------------------------------------------------------------------------
// Greedy acceptance walk and next tree (Section 3.4).  One CTA per sequence.
// ---------------------------------------------------------------------------
__global__ void accept_kernel(Rows rw, AcceptArgs a, int pdl) {
  __shared__ int32_t s_best[kMaxTreeRows];
  __shared__ int32_t s_bonus, s_end;
  if (pdl) { griddep_launch(); griddep_wait(); }
  const int s = blockIdx.x, tid = threadIdx.x;
  const int32_t *tok = a.tokens + (size_t)s * rw.T;
  // own tree of the sequence (rows beyond its size are padding and can neither be accepted nor take a candidate)
  const int32_t *parents = a.parents + (size_t)s * a.parents_stride, *next_parents = a.next_parents + (size_t)s * a.parents_stride;
  const int Ts = a.sizes ? min(a.sizes[s], rw.T) : rw.T, Tn = a.sizes ? min(a.sizes[s], a.T_next) : a.T_next;
  for (int v = tid; v < rw.T; v += blockDim.x) {
    const int32_t b = a.top_ids[(size_t)(s * rw.Ms + v) * a.B];
    s_best[v] = b;
    if (a.o_best) a.o_best[(size_t)s * rw.T + v] = b;
  }
  __syncthreads();
  if (tid == 0) {
    int32_t *path = a.path + (size_t)s * a.S, *acc = a.accepted + (size_t)s * a.S;
    int cur = 0, na = 0;
    path[0] = 0;
    if (a.prefill_last_row >= 0) {
      cur = a.prefill_last_row;
    } else {
      while (na + 1 < a.S) {
        int next = -1;
        for (int ch = cur + 1; ch < Ts; ++ch)
          if (parents[ch] == cur && tok[ch] == s_best[cur]) { next = ch; break; }
        if (next < 0) break;
        acc[na] = tok[next];
        path[++na] = next;
        cur = next;
      }
    }
    acc[na] = s_best[cur];
    s_bonus = s_best[cur];
    s_end = cur;
    a.n_accepted[s] = na + 1;
    if (a.o_n_accepted) a.o_n_accepted[s] = na + 1;
    for (int j = 0; j <= na; ++j) {
      if (a.o_path) a.o_path[(size_t)s * a.S + j] = path[j];
      if (a.o_accepted) a.o_accepted[(size_t)s * a.S + j] = acc[j];
    }
  }
  __syncthreads();
  // the pseudo row that holds the candidates of depth j (1-based): row j of the one chain, or of the chain
  // under the node the walk ended on
  const int steps = rw.chains ? rw.kc : rw.k;
  const size_t row0 = (size_t)s * rw.Ms + rw.T + (rw.chains ? s_end : 0);
  const int row_step = rw.chains ? rw.T : 1;
  if (a.o_topb_ids || a.o_topb_vals) {
    for (int i = tid; i < steps * a.B; i += blockDim.x) {
      const size_t src = (row0 + (size_t)(i / a.B) * row_step) * a.B + i % a.B;
      if (a.o_topb_ids) a.o_topb_ids[(size_t)s * steps * a.B + i] = a.top_ids[src];
      if (a.o_topb_vals) a.o_topb_vals[(size_t)s * steps * a.B + i] = a.top_vals[src];
    }
  }
  for (int v = tid; v < a.T_next; v += blockDim.x) {
    int32_t t;
    if (v == 0 || v >= Tn) {
      t = s_bonus;
    } else {
      int dep = 0;
      for (int u = v; u > 0 && dep <= a.T_next; u = next_parents[u]) ++dep;
      int rank = 0;
      for (int u = 1; u < v; ++u) rank += (next_parents[u] == next_parents[v]);
      dep = min(dep, max(steps, 1));
      rank = min(rank, a.B - 1);
      t = (steps > 0) ? a.top_ids[(row0 + (size_t)(dep - 1) * row_step) * a.B + rank] : s_bonus;
    }
    a.next_tokens[(size_t)s * a.T_next + v] = t;
    if (a.o_next_tokens) a.o_next_tokens[(size_t)s * a.T_next + v] = t;
  }
}

void launch_accept(const Rows &rw, const AcceptArgs &a, bool pdl, cudaStream_t st) {
  launch_k(accept_kernel, dim3(rw.n_seq), dim3(128), 0, st, pdl, rw, a, pdl ? 1 : 0);
}

// ---------------------------------------------------------------------------
// KV compaction of the accepted path.  Each thread owns one 16-byte column slice of a
// (layer, K|V) plane and moves it for every path entry: it loads all source rows before
// storing any, so a destination slot that is another entry's source is never clobbered.
// ---------------------------------------------------------------------------
constexpr int kMaxPath = 16;

__global__ void __launch_bounds__(128) commit_kernel(CommitArgs a, int pdl) {
  if (pdl) { griddep_launch(); griddep_wait(); }
  const int s = blockIdx.y, plane = blockIdx.x;     // plane = layer * 2 + (0 K, 1 V)
  const int slot = a.seq_ids[s];
  const int n = a.ctx_len[slot];
  const int len = min(a.path_len[s], kMaxPath);
  const int32_t *path = a.path + (size_t)s * a.S;
  bf16 *base = a.kv + (size_t)(plane >> 1) * a.layer_stride + (size_t)(plane & 1) * a.kv_stride;
  const int nvec = a.nkv >> 3;
  size_t src_row[kMaxPath], dst_row[kMaxPath];
#pragma unroll
  for (int j = 0; j < kMaxPath; ++j) {
    if (j < len) { src_row[j] = kv_row(a.pages, slot, n + path[j], a.max_ctx); dst_row[j] = kv_row(a.pages, slot, n + j, a.max_ctx); }
  }
  for (int c = threadIdx.x; c < nvec; c += blockDim.x) {
    uint4 tmp[kMaxPath];
#pragma unroll
    for (int j = 0; j < kMaxPath; ++j)
      if (j < len) tmp[j] = reinterpret_cast<const uint4 *>(base + src_row[j] * a.nkv)[c];
#pragma unroll
    for (int j = 0; j < kMaxPath; ++j)
      if (j < len && path[j] != j) reinterpret_cast<uint4 *>(base + dst_row[j] * a.nkv)[c] = tmp[j];
  }
}

__global__ void advance_ctx_kernel(int n_seq, const int32_t *seq_ids, int32_t *ctx_len, const int32_t *path_len,
                                   int amount, int pdl) {
  if (pdl) { griddep_launch(); griddep_wait(); }
  const int s = threadIdx.x;
  if (s < n_seq) ctx_len[seq_ids[s]] += path_len ? min(path_len[s], kMaxPath) : amount;
}

void launch_commit(int n_seq, const CommitArgs &a, bool pdl, cudaStream_t st) {
  launch_k(commit_kernel, dim3(a.n_layers * 2, n_seq), dim3(128), 0, st, pdl, a, pdl ? 1 : 0);
  launch_k(advance_ctx_kernel, dim3(1), dim3(32), 0, st, pdl, n_seq, a.seq_ids, a.ctx_len, a.path_len, 0, pdl ? 1 : 0);
}

void launch_advance_ctx(int n_seq, const int32_t *seq_ids, int32_t *ctx_len, int amount, bool pdl, cudaStream_t st) {
  launch_k(advance_ctx_kernel, dim3(1), dim3(32), 0, st, pdl, n_seq, seq_ids, ctx_len, (const int32_t *)nullptr, amount,
           pdl ? 1 : 0);
}

}  // namespace firp
