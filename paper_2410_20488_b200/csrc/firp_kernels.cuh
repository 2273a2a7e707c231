// Internal launcher interface between the step scheduler and the sm_100a kernels.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace firp {

typedef __nv_bfloat16 bf16;

constexpr int kMaxSeq = 16;        // sequences per step
constexpr int kMaxTreeRows = 144;  // rows per sequence: T + k (128 + 8), or T (1 + k) with a chain under every node
constexpr int kMaskWords = 5;      // ceil(136 / 32)
constexpr int kMaxTopB = 8;
constexpr int kAttnTile = 64;      // kv positions per attention tile
constexpr int kGemmBN = 64;        // weight rows per GEMM tile
constexpr int kGemmBK = 64;        // k elements per pipeline stage

// Per-step row geometry shared by every kernel.  Row r = s * Ms + v.
struct Rows {
  int n_seq;   // sequences in this step
  int T;       // tree rows per sequence
  int k;       // pseudo rows per sequence
  int Ms;      // T + k
  int R;       // n_seq * Ms
  int anchor;  // tree row the pseudo chain hangs off (one chain)
  int chains;  // != 0: a chain under every tree node; chain row i (1-based) of node v is row T + (i-1) T + v
  int kc;      // prediction steps per chain (k = kc with one chain, k = T * kc with a chain per node)
  int masked;  // != 0: a pseudo row sees no other pseudo row (the "Masked" ablation of Section 4.3)
};

// Rows of the KV cache.  A (layer, K|V) plane holds max_batch * max_ctx rows of Hkv * dh elements.  Without a
// page table position `pos` of slot `slot` is row slot * max_ctx + pos; with one (pages of kKvPage positions,
// table[slot * pages_per_seq + pos / kKvPage] = physical page) it is row page * kKvPage + pos % kKvPage.
constexpr int kKvPage = 64;               // = kAttnTile: an attention tile never straddles two pages
struct KvPages { const int32_t *table; int pages_per_seq; };
__device__ __forceinline__ size_t kv_row(const KvPages &pg, int slot, int pos, int max_ctx) {
  if (pg.table == nullptr) return (size_t)slot * max_ctx + pos;
  return (size_t)pg.table[slot * pg.pages_per_seq + pos / kKvPage] * kKvPage + (pos % kKvPage);
}

constexpr int kGemmMaxCtas = 192;         // scratch slots are provided for this many CTAs
constexpr int kGemmSlots = 3;             // partial tiles (segments) per CTA

// Stream-K schedule of one GEMM launch.  Unit u = supertile * KB + k block (supertile = 256 weight
// rows, k block = 64 elements); CTA c owns units [sk_begin(c), sk_begin(c + 1)) and its s-th segment
// is the part of supertile sk_begin(c) / KB + s inside that range.
struct StreamK {
  int U;        // units (supertiles x k blocks; U * G stays far below 2^31 for every supported shape)
  int KB;       // k blocks per supertile
  int G;        // CTAs (<= U, so no range is empty)
};
__host__ __device__ __forceinline__ int sk_begin(const StreamK &s, int c) { return (int)(((unsigned)s.U * (unsigned)c) / (unsigned)s.G); }
// CTA whose range holds unit u: the largest c with floor(U c / G) <= u, i.e. c < (u + 1) G / U
__host__ __device__ __forceinline__ int sk_owner(const StreamK &s, int u) {
  return (int)((((unsigned)u + 1u) * (unsigned)s.G + (unsigned)s.U - 1u) / (unsigned)s.U) - 1;
}
// The CTAs c_first..c_last that hold a piece of supertile st.  Every one but the first starts its range
// inside st, so its piece is its segment 0; the first one's piece is segment ord_first.
struct SkContrib { int c_first, c_last, ord_first; };
__host__ __device__ __forceinline__ SkContrib sk_contributors(const StreamK &s, int st) {
  SkContrib k;
  k.c_first = sk_owner(s, st * s.KB);
  k.c_last = sk_owner(s, (st + 1) * s.KB - 1);
  k.ord_first = st - sk_begin(s, k.c_first) / s.KB;
  return k;
}

// ---- tree bookkeeping (Section 3.4) ---------------------------------------
struct TreeMeta {
  int32_t *depth;      // [R]
  int32_t *pos;        // [R] absolute position = ctx_len + depth
  uint32_t *mask;      // [R][kMaskWords] bit u: row v attends to new row u of its sequence
  float2 *rope;        // [R][dh/2] (cos, sin) of pos * theta^(-2c/dh)
};
// d_parents: [T] shared by the sequences (parents_stride 0) or [n_seq][T] (parents_stride T).
// zero_word (may be NULL): a device word the kernel clears (the arrival counter of the fused decoder kernel)
void launch_tree_prep(const Rows &rw, const int32_t *d_parents, int parents_stride, const int32_t *d_seq_ids, const int32_t *d_ctx_len,
                      int dh, float theta, TreeMeta meta, int32_t *out_depth, uint32_t *out_mask, int out_mask_words,
                      unsigned *zero_word, bool pdl, cudaStream_t st);

// h[r] = embed[token] for tree rows, 0 for pseudo rows
void launch_embed(const Rows &rw, const int32_t *d_tokens, const bf16 *embed, int d, int vocab, float *h, bool pdl,
                  cudaStream_t st);

// Activations that feed a GEMM or the attention are stored as two bf16 planes (hi, lo) with
// hi + lo = the fp32 value to ~16 mantissa bits; the lo plane starts *_lo_off elements after hi.

// Partial tiles a stream-K GEMM left in scratch: slot (c, s) = segment s of CTA c, laid out
// [2 tiles][ws_rows token rows][128 lanes] fp32; whoever consumes the GEMM sums them in CTA order.
struct Partials {
  StreamK sk;        // schedule of the GEMM that wrote the tiles (U = 0: nothing pending)
  const float *ws;   // its scratch slots
  int ws_rows;       // token rows per scratch tile
};
// For rows with v in [v0, v1): if `pending` has units, first h[r] += the partial tiles of a residual GEMM;
// then x[r] = h[r] * g as `planes` bf16 planes (hi, lo or hi, mid, lo) and ss[r][w] = sum of squares of the
// 128 columns of warp w.
// The 1 / sqrt(mean(h^2) + eps) of RMSNorm is applied by the finisher of the GEMM that consumes x.
constexpr int kNormMaxWarps = 64;   // d <= 8192
cudaError_t launch_rmsnorm(const Rows &rw, int v0, int v1, float *h, const Partials &pending, const bf16 *g, int d,
                           bf16 *x, size_t x_lo_off, int planes, float *ss, bool pdl, cudaStream_t st);

// Eq. 3, h[s*Ms + T + i] = W_i h[s*Ms + anchor] + b_i, as a GEMM of the k maps stacked into one [k d][d] matrix:
// launch_root_split writes the raw residual rows Eq. 3 reads (every sequence's anchor, or all its T tree rows when
// every node carries a chain: row s * T + v) as (hi, lo) bf16 planes; one chain: into row s of
// xp; the GEMM (EPI_PSEUDO) multiplies; launch_gemm_finish(EPI_PSEUDO) sums the partial tiles, adds the bias and
// stores the k new residual rows (GemmArgs: h_rows = residual stream, pred_b = bias or NULL, R = n_seq).
// g (may be NULL): gain vector of the pre-norm variant: the planes then hold h * g and the finisher divides by the
// source row's RMS (GemmArgs::ss of the EPI_PSEUDO finisher)
void launch_root_split(const Rows &rw, const float *h, const bf16 *g, int d, bf16 *xp, size_t xp_lo_off, bool pdl, cudaStream_t st);

// top-B of every row of logits by (value desc, id asc)
// Two passes: per 2048-logit segment candidates (scratch cand_*: [R][topb_segments(V)][B]), then the row's top-B.
constexpr int kTopSeg = 2048;
int topb_segments(int V);
void launch_topb(const float *logits, int R, int V, int B, int32_t *cand_ids, float *cand_vals, int32_t *ids, float *vals,
                 bool pdl, cudaStream_t st);

struct AcceptArgs {
  const int32_t *tokens;        // [n_seq][T]
  const int32_t *parents;       // [T], or [n_seq][T] with parents_stride = T
  const int32_t *next_parents;  // [T_next], likewise
  int parents_stride;           // 0: one template for every sequence
  const int32_t *sizes;         // NULL, or [n_seq]: nodes of each sequence's own tree (the rest of its T rows is padding)
  const int32_t *top_ids;       // [R][B] (row r's candidates; [0] is the argmax)
  const float *top_vals;        // [R][B]
  int T_next, B, S;             // S = path stride
  int prefill_last_row;         // >= 0: prefill mode, the root is the argmax of this row; -1: verify walk
  int32_t *path, *n_accepted, *accepted;  // internal copies [n_seq][S], [n_seq], [n_seq][S]
  int32_t *next_tokens;                   // [n_seq][T_next]
  // optional caller buffers (may be NULL)
  int32_t *o_path, *o_n_accepted, *o_accepted, *o_next_tokens, *o_best, *o_topb_ids;
  float *o_topb_vals;
};
void launch_accept(const Rows &rw, const AcceptArgs &a, bool pdl, cudaStream_t st);

// KV compaction: rows path[j] -> slot n + j in every layer; then ctx_len += len
struct CommitArgs {
  bf16 *kv;                 // cache base
  size_t seq_stride;        // elements per sequence
  size_t layer_stride;      // elements per layer (2 * max_ctx * nkv)
  size_t kv_stride;         // elements per K or V plane (max_ctx * nkv)
  int n_layers, nkv;        // nkv = Hkv * dh
  const int32_t *seq_ids;   // [n_seq] device
  const int32_t *path;      // [n_seq][S] device
  const int32_t *path_len;  // [n_seq] device
  int S;
  int32_t *ctx_len;         // [max_batch] device
  int max_ctx; KvPages pages;
};
void launch_commit(int n_seq, const CommitArgs &a, bool pdl, cudaStream_t st);
void launch_advance_ctx(int n_seq, const int32_t *seq_ids, int32_t *ctx_len, int amount, bool pdl, cudaStream_t st);

// ---- skinny weight-streaming GEMM ------------------------------------------
enum GemmEpilogue { EPI_RESIDUAL = 0, EPI_QKV_ROPE = 1, EPI_SWIGLU = 2, EPI_LOGITS = 3, EPI_PSEUDO = 4 };

struct GemmArgs {
  const bf16 *X;    // [R][K] activations, first (hi) plane (row-major, K contiguous)
  size_t x_lo_off;  // elements from one plane to the next ( = plane_rows * K )
  int plane_rows;   // rows per plane of X
  int planes;       // 2: hi + lo (~16 mantissa bits), 3: hi + mid + lo (~24 bits)
  const bf16 *W;    // [N][K] weights
  int R;            // valid rows
  int *err;         // device status word (set to a non-zero code if a bounded wait gives up)
  unsigned long long wait_ns;   // bounded waits give up after this many nanoseconds (0: the default of 2 s)
  int N, K;
  Rows rw; int rows_active;      // rows with v < rows_active are written, the others skipped
  // stream-K scratch: partial tiles [kGemmMaxCtas][kGemmSlots][2][plane_rows][128] fp32
  float *ws;
  int l2_ahead;     // 32 KB units each CTA prefetches into L2 beyond its shared-memory ring while it waits
  // The GEMM that follows this one in the step (NULL: none).  Once a CTA has issued its own last load it
  // prefetches the first next_units units of the same CTA's range of THAT GEMM into L2, so that HBM keeps
  // streaming through this kernel's tail and the hand-over, and the next kernel's ring fills from L2.
  const bf16 *next_W; int next_epi, next_N, next_K, next_F, next_heads, next_dh, next_units;
  // finishers: X holds h * g, not yet divided by the RMS: row m of the result is scaled by
  // 1 / sqrt(sum_w ss[m][w] / K + eps) (ss == NULL: X is used as it is)
  const float *ss; float eps;
  // EPI_QKV_ROPE
  int H, Hkv, dh;
  const float2 *rope; const int32_t *seq_ids; const int32_t *ctx_len; const int32_t *pos;   // pos[R]: row positions
  bf16 *q; size_t q_lo_off;      // [R][H*dh] hi plane, lo plane
  bf16 *kcache; size_t seq_stride, kv_stride; int max_ctx;  // kcache points at this layer's K plane (row 0)
  KvPages pages;
  // EPI_SWIGLU: y[R][F], N = 2F
  bf16 *y; size_t y_lo_off; int F;
  // EPI_LOGITS: logits[R][N]
  float *logits;
  // EPI_PSEUDO: output n = i * K + o of map pseudo0 + i (+ pred_b[n]).  One chain: row m = sequence m, result to
  // h_rows[(m * Ms + T + pseudo0 + i) * K + o].  A chain per node: row m = s * T + v, result to
  // h_rows[(s * Ms + T + (pseudo0 + i) * T + v) * K + o].
  float *h_rows; const bf16 *pred_b; int pseudo0;
};
// The GEMM leaves partial tiles in a.ws under the schedule *sk_out, to be finished by launch_gemm_finish
// (or, for EPI_RESIDUAL, by launch_rmsnorm).  `epi` only selects how weight rows are grouped into supertiles.
// pdl: launch with programmatic stream serialization (the kernel waits on its predecessor itself).
cudaError_t launch_gemm_tc(GemmEpilogue epi, const GemmArgs &a, bool pdl, cudaStream_t st, StreamK *sk_out);
cudaError_t launch_gemm_finish(GemmEpilogue epi, const Partials &p, const GemmArgs &a, bool pdl, cudaStream_t st);
bool gemm_tc_available();         // the driver entry point for tensor-map encoding was found

// ---- tree-masked split-KV attention ---------------------------------------
constexpr int kAttnMaxSplits = 8;   // kv splits = CTAs per cluster (portable cluster size limit)
struct AttnArgs {
  Rows rw; int rows_active;
  int H, Hkv, dh;
  const bf16 *q; size_t q_lo_off;   // [R][H*dh] rotated queries, hi and lo planes
  const bf16 *kcache;         // this layer's K plane of slot 0; V plane = kcache + kv_stride
  size_t seq_stride, kv_stride; int max_ctx;
  KvPages pages;
  const int32_t *seq_ids, *ctx_len;
  const int32_t *pos;         // [R] absolute position of every row (row 0 of a sequence: its committed length)
  const uint32_t *mask;       // [R][kMaskWords]
  int splits;                 // kv splits (grid.x = cluster size): 1, 2, 4 or 8
  int q_planes, p_planes;     // bf16 planes of the queries / of the probabilities that enter the tensor cores: 2 (hi, lo) or 1
  bf16 *o; size_t o_lo_off;   // [R][H*dh] hi plane, lo plane
  int *err; unsigned long long wait_ns;   // status word and bound of the device-side waits (tensor-core kernel; 0: default)
};
// kv splits for `groups` = sequences x kv heads x query blocks and `kv_tiles` 64-position tiles
int attention_splits(int groups, int kv_tiles);
cudaError_t launch_attention(const AttnArgs &a, bool pdl, cudaStream_t st);
// The tcgen05 kernel (head dimension 128): 128-position tiles, query blocks of at most kAttnTcMaxCols columns
// (query rows x heads of the group), a.splits from attention_tc_splits.
constexpr int kAttnTcTile = 128, kAttnTcMaxCols = 48;
void attention_tc_blocks(int qrows, int *qblocks, int *qper);
int attention_tc_splits(int groups, int kv_tiles, int sm_count);
cudaError_t launch_attention_tc(const AttnArgs &a, bool pdl, cudaStream_t st);

// ---- the decoder layers of a step as one persistent kernel (fused_step.cu) ------------------------------
struct FusedShape { int L, d, H, Hkv, dh, F, V, max_ctx; float eps; };
struct FusedStep {
  FusedShape shape;
  Rows rw;
  int tl[8];                 // insertion layer of each prediction step (non-decreasing)
  bool want_head;            // final norm + lm-head
  bool prenorm;              // Eq. 3 reads the anchor through the insertion layer's input RMSNorm
  int Rp;                    // rows per activation plane
  int n_hi_max;              // upper bound of the longest committed context among the sequences
  int max_batch;             // of the configuration (sizes the attention scratch)
  uint64_t weights_gen;      // changes whenever the weight pointers change
  unsigned long long wait_ns;   // bound of every device-side wait (0: default)
  // weights (device pointers; the per-layer arrays are host arrays of L pointers)
  const void *const *wqkv, *const *wo, *const *wgu, *const *wd, *const *g_attn, *const *g_mlp;
  const void *g_final, *lm_head, *pred_w, *pred_b;
  // workspace
  float *h, *ws, *ss, *logits, *attn_ws;
  bf16 *x, *xp, *q, *o, *y, *kv;
  size_t kv_seq, kv_layer, kv_plane;
  KvPages pages;
  const float2 *rope; const int32_t *pos, *seq_ids, *ctx_len; const uint32_t *mask;
  int *err; unsigned *bar;   // status word; arrival counter of the grid barrier (zero before the launch)
  void *d_maps;              // device room for the tensor maps: fused_map_bytes(L) bytes, 128-byte aligned
};
struct FusedPlan;            // host-side cache of the phase list and the tensor maps of one step shape
FusedPlan *fused_plan_create();
void fused_plan_destroy(FusedPlan *p);
size_t fused_map_bytes(int n_layers);
size_t fused_attn_ws_floats(int max_batch, int H, int Hkv, int dh);   // scratch of the attention splits
// whether the fused kernel can run this step (at most 48 rows; every GEMM's stream-K schedule fits its scratch)
bool fused_eligible(const FusedShape &sh, const Rows &rw);
// Runs everything between the embedding and the top-B: all decoder layers, Eq. 3 at its layers, and (want_head)
// the final norm and the lm-head.  Cooperative launch, one CTA per SM.
cudaError_t launch_fused_layers(FusedPlan *plan, const FusedStep &fs, bool pdl, cudaStream_t st, int *launches);
// one CTA waits (bounded by wait_ns, 0 = default) on a barrier nobody arrives on, sets *err and returns
cudaError_t launch_wait_selftest(int *err, unsigned long long wait_ns, cudaStream_t st);

}  // namespace firp
