// C ABI of the FIRP draft+verify step: context, argument validation, workspace layout and
// the per-step launch sequence (Section 3.4 inference loop).  Host code only; every step of
// the path runs in the kernels declared in firp_kernels.cuh.
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <string>
#include <vector>

#include "../../include/firp.h"
#include "firp_kernels.cuh"

using namespace firp;

namespace {

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Carver {
  uint8_t *base; size_t off;
  template <typename T> T *take(size_t count) {
    off = align_up(off, 256);
    T *p = base ? reinterpret_cast<T *>(base + off) : nullptr;
    off += count * sizeof(T);
    return p;
  }
};

}  // namespace

// Kernel classes of the per-kernel timing aid (firp_profile_*).
enum KernelClass {
  KC_TREE_PREP = 0, KC_EMBED, KC_RMSNORM, KC_PSEUDO_PROJ, KC_GEMM_QKV, KC_QKV_FINISH, KC_ATTENTION, KC_GEMM_O,
  KC_GEMM_GATE_UP, KC_SWIGLU_FINISH, KC_GEMM_DOWN, KC_GEMM_LM_HEAD, KC_LOGITS_FINISH, KC_TOPB, KC_ACCEPT, KC_COMMIT, KC_FUSED_LAYERS, KC_COUNT
};
static const char *const kClassNames[KC_COUNT] = {
    "tree_prep", "embed", "residual_rmsnorm", "pseudo_proj", "gemm_qkv", "qkv_rope_finish", "tree_attention", "gemm_o",
    "gemm_gate_up", "swiglu_finish", "gemm_down", "gemm_lm_head", "logits_finish", "topb", "accept_next_tree", "kv_commit",
    "fused_decoder_layers"};

struct firp_ctx {
  firp_model_cfg cfg{};
  // per-kernel timing aid: event pairs recorded around launches while enabled
  bool profiling = false;
  std::vector<cudaEvent_t> ev_pool;           // events created so far (reused after each read)
  std::vector<int> ev_class;                  // class of pair i (events 2i, 2i+1)
  size_t ev_used = 0;                         // pairs in use
  std::string err;
  int launches = 0;
  bool bound = false, have_weights = false, stepped = false;
  int Rmax = 0, S = 0;                  // rows the workspace holds (a prefill chunk), path stride
  int row_cap = 0;                      // rows one step may carry (max_rows of the configuration)
  int sm_count = 148;                   // of the device the buffers were bound on
  bool use_pdl = true;                  // programmatic dependent launch
  bool use_fused = false;               // firp_set_fused: steps of at most 48 rows run their layers as one persistent kernel
  unsigned long long wait_ns = 0;       // bound of device-side waits (0: the kernels' default)
  uint64_t weights_gen = 0;             // bumped by firp_init_weights
  FusedPlan *plan_step = nullptr, *plan_prefill = nullptr;
  int *dev_status = nullptr;            // device status word (bounded waits report here)
  unsigned *grid_bar = nullptr;         // arrival counter of the fused kernel's grid barrier
  float *attn_ws = nullptr;             // partial results of its attention splits
  uint8_t *d_maps = nullptr;            // its tensor maps
  int32_t *d_pages = nullptr;           // page table of the KV cache (device copy), [max_batch][pages_per_seq]
  bool paged = false;
  int pages_per_seq() const { return (cfg.max_ctx + kKvPage - 1) / kKvPage; }
  KvPages pages() const { return KvPages{paged ? d_pages : nullptr, pages_per_seq()}; }
  // weights
  firp_weights w{};
  std::vector<const void *> wqkv, wo, wgu, wd, g_attn, g_mlp;
  // device buffers (carved from the caller's workspace)
  bf16 *kv = nullptr;
  float *h = nullptr, *gemm_ws = nullptr, *ss = nullptr, *logits = nullptr, *top_vals = nullptr, *cand_vals = nullptr;
  int32_t *cand_ids = nullptr;
  bf16 *x = nullptr, *xp = nullptr, *q = nullptr, *o = nullptr, *y = nullptr;
  int32_t *ctx_len = nullptr, *seq_ids = nullptr, *parents = nullptr, *next_parents = nullptr, *chain = nullptr;
  int32_t *top_ids = nullptr, *path = nullptr, *n_acc = nullptr, *accepted = nullptr, *next_tokens = nullptr;
  int32_t *exp_path = nullptr, *exp_len = nullptr, *tree_sizes = nullptr;
  TreeMeta meta{};
  size_t ws_bytes = 0;
  // host mirrors
  std::vector<int32_t> n_hi;           // upper bound of each slot's committed length
  std::vector<int32_t> last_parents, last_next_parents, last_seq_ids, last_sizes;
  int last_n_seq = 0, last_T = 0, last_k = 0;
  int pseudo_masked = 0;     // Section 4.3 "Masked": pseudo rows do not see one another
  int pred_prenorm = 0;      // Eq. 3 reads the anchor through the insertion layer's input RMSNorm
  int planes[5] = {2, 2, 2, 2, 2};
  int attn_tc = -1;                  // head dimension 128: 1 the tcgen05 attention kernel, 0 the mma.sync one, -1 by the step's shape
  int attn_planes[2] = {2, 2};       // of the queries and of the probabilities in the attention   // bf16 planes of the activations per GEMM class: qkv, o, gate/up, down, lm-head

  // cache layout [layer][K|V][row][kv_head][head_dim]; row = slot * max_ctx + position, or through the page table
  size_t kv_seq() const { return (size_t)cfg.max_ctx * cfg.n_kv_heads * cfg.head_dim; }      // elements per slot of a plane
  size_t kv_plane() const { return (size_t)cfg.max_batch * kv_seq(); }                        // one K or V plane of a layer
  size_t kv_layer() const { return 2 * kv_plane(); }

  size_t carve(void *base) {
    Carver c{reinterpret_cast<uint8_t *>(base), 0};
    const int d = cfg.d_model, nq = cfg.n_heads * cfg.head_dim, half = cfg.head_dim / 2;
    const size_t R = Rmax;
    h = c.take<float>(R * d);
    xp = c.take<bf16>(2 * R * d);           // the rows Eq. 3 reads (anchor of each sequence, or all tree rows): hi plane, lo plane
    x = c.take<bf16>(3 * R * d);            // normalised activations: hi plane, lo plane, third plane (QKV input)
    q = c.take<bf16>(2 * R * nq);
    o = c.take<bf16>(2 * R * nq);
    y = c.take<bf16>(2 * R * cfg.d_ffn);
    gemm_ws = c.take<float>((size_t)kGemmMaxCtas * kGemmSlots * 2 * R * 128);
    ss = c.take<float>(R * kNormMaxWarps);
    logits = c.take<float>(R * cfg.vocab);
    top_ids = c.take<int32_t>(R * kMaxTopB);
    top_vals = c.take<float>(R * kMaxTopB);
    cand_ids = c.take<int32_t>(R * (size_t)topb_segments(cfg.vocab) * kMaxTopB);
    cand_vals = c.take<float>(R * (size_t)topb_segments(cfg.vocab) * kMaxTopB);
    meta.depth = c.take<int32_t>(R);
    meta.pos = c.take<int32_t>(R);
    meta.mask = c.take<uint32_t>(R * kMaskWords);
    meta.rope = c.take<float2>(R * half);
    ctx_len = c.take<int32_t>(cfg.max_batch);
    seq_ids = c.take<int32_t>(kMaxSeq);
    parents = c.take<int32_t>(kMaxTreeRows);
    next_parents = c.take<int32_t>(kMaxTreeRows);
    chain = c.take<int32_t>(kMaxTreeRows);
    path = c.take<int32_t>((size_t)kMaxSeq * S);
    n_acc = c.take<int32_t>(kMaxSeq);
    accepted = c.take<int32_t>((size_t)kMaxSeq * S);
    next_tokens = c.take<int32_t>((size_t)kMaxSeq * kMaxTreeRows);
    exp_path = c.take<int32_t>((size_t)kMaxSeq * S);
    exp_len = c.take<int32_t>(kMaxSeq);
    tree_sizes = c.take<int32_t>(kMaxSeq);
    dev_status = c.take<int>(1);
    grid_bar = c.take<unsigned>(1);
    attn_ws = c.take<float>(fused_attn_ws_floats(cfg.max_batch, cfg.n_heads, cfg.n_kv_heads, cfg.head_dim));
    d_pages = c.take<int32_t>((size_t)cfg.max_batch * pages_per_seq());
    d_maps = c.take<uint8_t>(2 * fused_map_bytes(cfg.n_layers));   // one set for the step plan, one for the prefill plan
    return align_up(c.off, 256);
  }
};

namespace {

int fail(firp_ctx *ctx, int code, const char *fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof(buf), fmt, ap);
  va_end(ap);
  if (ctx) ctx->err = buf;
  return code;
}

#define FIRP_CUDA(ctx, call)                                                                            \
  do {                                                                                                  \
    cudaError_t e__ = (call);                                                                           \
    if (e__ != cudaSuccess) return fail(ctx, FIRP_ERR_CUDA, "%s: %s", #call, cudaGetErrorString(e__)); \
  } while (0)

// Brackets the launches issued during its lifetime with an event pair when profiling is on.
struct Bracket {
  firp_ctx *c; cudaStream_t st; cudaEvent_t stop = nullptr;
  Bracket(firp_ctx *ctx, int cls, cudaStream_t s) : c(ctx), st(s) {
    if (!c->profiling) return;
    while (c->ev_pool.size() < 2 * (c->ev_used + 1)) {
      cudaEvent_t e;
      if (cudaEventCreate(&e) != cudaSuccess) return;
      c->ev_pool.push_back(e);
    }
    if (c->ev_class.size() <= c->ev_used) c->ev_class.resize(c->ev_used + 1);
    c->ev_class[c->ev_used] = cls;
    cudaEventRecord(c->ev_pool[2 * c->ev_used], st);
    stop = c->ev_pool[2 * c->ev_used + 1];
    ++c->ev_used;
  }
  ~Bracket() { if (stop) cudaEventRecord(stop, st); }
};
#define FIRP_TIMED(cls) Bracket bracket__(c, cls, st)

// depth of every node of a validated tree; returns max depth or -1 if malformed
int tree_depths(const int32_t *parents, int T, std::vector<int> &depth) {
  depth.assign(T, 0);
  if (T < 1 || parents[0] != -1) return -1;
  int mx = 0;
  for (int v = 1; v < T; ++v) {
    if (parents[v] < 0 || parents[v] >= v) return -1;
    depth[v] = depth[parents[v]] + 1;
    mx = depth[v] > mx ? depth[v] : mx;
  }
  return mx;
}

// sibling rank must stay below top_b for every node that takes a candidate
int max_sibling_rank(const int32_t *parents, int T) {
  int mx = 0;
  for (int v = 1; v < T; ++v) {
    int r = 0;
    for (int u = 1; u < v; ++u) r += (parents[u] == parents[v]);
    mx = r > mx ? r : mx;
  }
  return mx;
}

int upload_i32(firp_ctx *ctx, int32_t *dst, const int32_t *src, int n, std::vector<int32_t> &mirror, cudaStream_t st) {
  if ((int)mirror.size() == n && memcmp(mirror.data(), src, sizeof(int32_t) * n) == 0) return FIRP_OK;
  mirror.assign(src, src + n);
  FIRP_CUDA(ctx, cudaMemcpyAsync(dst, mirror.data(), sizeof(int32_t) * n, cudaMemcpyHostToDevice, st));
  return FIRP_OK;
}

// The launch sequence shared by firp_step and firp_prefill chunks.
struct RunArgs {
  Rows rw;
  const int32_t *d_tokens;   // [n_seq][T]
  int tl[8];                 // insertion layer of each prediction step (non-decreasing), Section 3.3
  bool want_head;            // run final norm + lm-head + top-B + accept
  int prefill_last_row;      // -1: verify walk
  int T_next;
  const firp_step_out *out;
  float *logits_dst;         // where the lm-head writes (workspace or caller buffer)
  int n_hi_max;              // upper bound of the longest committed context among the sequences
  int parents_stride;        // 0: one tree template for all sequences; T: a tree per sequence
  const int32_t *d_sizes;    // per-sequence tree sizes (device) or NULL
};

int run_rows(firp_ctx *c, const RunArgs &ra, cudaStream_t st) {
  const firp_model_cfg &cfg = c->cfg;
  const Rows &rw = ra.rw;
  const int d = cfg.d_model, H = cfg.n_heads, Hkv = cfg.n_kv_heads, dh = cfg.head_dim, F = cfg.d_ffn;
  const int nq = H * dh;
  const size_t Rp = (size_t)c->Rmax;          // rows per activation plane
  const firp_step_out *out = ra.out;
  int &nl = c->launches;
  const bool pdl = c->use_pdl;
  // L2 lookahead per GEMM class (32 KB units beyond the ring): qkv, o, gate/up, down, lm-head.  Measured at the
  // 7B shape: it pays before the GEMMs whose predecessor is short or cannot share the SM (o, gate/up) and
  // costs before the down projection, whose finisher it slows by more than it saves.
  static const int ahead[5] = {0, 48, 48, 0, 48};

  const int mw_out = (rw.Ms + 31) / 32;
  { FIRP_TIMED(KC_TREE_PREP);
    launch_tree_prep(rw, c->parents, ra.parents_stride, c->seq_ids, c->ctx_len, dh, cfg.rope_theta, c->meta, out ? out->depth : nullptr,
                     out ? out->mask : nullptr, mw_out, c->grid_bar, pdl, st); ++nl; }
  { FIRP_TIMED(KC_EMBED);
    launch_embed(rw, ra.d_tokens, (const bf16 *)c->w.embed, d, cfg.vocab, c->h, pdl, st); ++nl; }

  const FusedShape fshape{cfg.n_layers, d, H, Hkv, dh, F, cfg.vocab, cfg.max_ctx, cfg.rms_eps};
  const bool fused = c->use_fused && fused_eligible(fshape, rw);
  if (fused) {      // all decoder layers (and the lm-head) as one persistent kernel
    FusedStep fs{};
    fs.shape = fshape; fs.rw = rw; memcpy(fs.tl, ra.tl, sizeof(fs.tl)); fs.want_head = ra.want_head; fs.prenorm = c->pred_prenorm != 0; fs.Rp = (int)Rp;
    fs.n_hi_max = ra.n_hi_max; fs.max_batch = cfg.max_batch; fs.weights_gen = c->weights_gen; fs.wait_ns = c->wait_ns;
    fs.wqkv = c->wqkv.data(); fs.wo = c->wo.data(); fs.wgu = c->wgu.data(); fs.wd = c->wd.data();
    fs.g_attn = c->g_attn.data(); fs.g_mlp = c->g_mlp.data();
    fs.g_final = c->w.g_final; fs.lm_head = c->w.lm_head; fs.pred_w = c->w.pred_w; fs.pred_b = c->w.pred_b;
    fs.h = c->h; fs.ws = c->gemm_ws; fs.ss = c->ss; fs.logits = ra.logits_dst; fs.attn_ws = c->attn_ws;
    fs.x = c->x; fs.xp = c->xp; fs.q = c->q; fs.o = c->o; fs.y = c->y; fs.kv = c->kv;
    fs.kv_seq = c->kv_seq(); fs.kv_layer = c->kv_layer(); fs.kv_plane = c->kv_plane(); fs.pages = c->pages();
    fs.rope = c->meta.rope; fs.pos = c->meta.pos; fs.seq_ids = c->seq_ids; fs.ctx_len = c->ctx_len; fs.mask = c->meta.mask;
    // each cached plan owns its tensor maps on the device: a prefill between two steps must not replace the step's
    const bool for_prefill = ra.prefill_last_row >= 0;
    fs.err = c->dev_status; fs.bar = c->grid_bar; fs.d_maps = c->d_maps + (for_prefill ? fused_map_bytes(cfg.n_layers) : 0);
    FusedPlan *&plan = for_prefill ? c->plan_prefill : c->plan_step;
    if (!plan) plan = fused_plan_create();
    FIRP_TIMED(KC_FUSED_LAYERS);
    FIRP_CUDA(c, launch_fused_layers(plan, fs, pdl, st, &nl));
  }

  auto gemm_base = [&](const bf16 *X, size_t lo_off, const void *W, int N, int K, int act) {
    GemmArgs g{};
    g.X = X; g.x_lo_off = lo_off; g.plane_rows = (int)Rp; g.err = c->dev_status; g.wait_ns = c->wait_ns;
    g.W = (const bf16 *)W; g.R = rw.R; g.N = N; g.K = K; g.rw = rw; g.rows_active = act; g.planes = 2;
    g.ws = c->gemm_ws; g.l2_ahead = 48;
    if (X == c->x) { g.ss = c->ss; g.eps = cfg.rms_eps; }   // x = h * g: the finisher divides by the row's RMS
    return g;
  };
  // partial tiles a residual GEMM left behind: the next RMSNorm adds them into the residual stream
  Partials pending{};
  pending.ws = c->gemm_ws; pending.ws_rows = (int)Rp;
  const Partials none{};
  // every GEMM names its successor, whose first units it prefetches into L2 at its own tail
  // (32 KB units per CTA, by the GEMM that issues the prefetch: qkv, o, gate/up, down; 3 and 8 measured worse)
  static const int next_units[4] = {5, 5, 5, 5};
  auto set_next = [&](GemmArgs &g, int cls, GemmEpilogue epi, const void *W, int N, int K) {
    g.next_W = (const bf16 *)W; g.next_epi = epi; g.next_N = N; g.next_K = K; g.next_F = F; g.next_heads = H + 2 * Hkv;
    g.next_dh = dh; g.next_units = next_units[cls];
  };
  int alive = 0;   // prediction steps appended below this layer
  const int per_step = rw.chains ? rw.T : 1;                   // pseudo rows one prediction step adds per sequence
  for (int j = 0; j < cfg.n_layers && !fused; ++j) {
    int ins = 0;     // prediction steps whose layer this is
    while (alive + ins < rw.kc && ra.tl[alive + ins] == j) ++ins;
    const bool insert = ins > 0;
    // the rows that took part in the last residual GEMM get its pending sums; new pseudo rows have none
    const int carried = rw.T + alive * per_step;
    const int act = carried + ins * per_step;                  // rows alive in this layer
    { FIRP_TIMED(KC_RMSNORM);
      FIRP_CUDA(c, launch_rmsnorm(rw, 0, carried, c->h, pending, (const bf16 *)c->g_attn[j], d, c->x, Rp * d, c->planes[0] == 3 ? 3 : 2, c->ss, pdl, st)); ++nl; }
    pending.sk.U = 0;
    if (insert) {   // Eq. 3 on the raw (now complete) residual row of the root, then the norm of the new rows
      { FIRP_TIMED(KC_PSEUDO_PROJ);      // this layer's maps as one [ins d][d] GEMM on the source rows (the anchor of
                                         // each sequence, or every tree row when each node carries a chain)
        launch_root_split(rw, c->h, c->pred_prenorm ? (const bf16 *)c->g_attn[j] : nullptr, d, c->xp, Rp * d, pdl, st); ++nl;
        GemmArgs g{};
        g.X = c->xp; g.x_lo_off = Rp * d; g.plane_rows = (int)Rp; g.planes = 2; g.err = c->dev_status; g.wait_ns = c->wait_ns;
        g.W = (const bf16 *)c->w.pred_w + (size_t)alive * d * d; g.R = rw.n_seq * per_step; g.N = ins * d; g.K = d; g.rw = rw;
        g.rows_active = act;
        g.ws = c->gemm_ws; g.l2_ahead = 48;
        g.h_rows = c->h; g.pseudo0 = alive;      // map i of this GEMM is prediction step alive + i
        if (c->pred_prenorm) { g.ss = c->ss; g.eps = cfg.rms_eps; }   // the finisher divides by the source row's RMS
        g.pred_b = c->w.pred_b ? (const bf16 *)c->w.pred_b + (size_t)alive * d : nullptr;
        Partials p = pending;
        FIRP_CUDA(c, launch_gemm_tc(EPI_PSEUDO, g, pdl, st, &p.sk)); ++nl;
        p.ws_rows = (int)Rp;
        FIRP_CUDA(c, launch_gemm_finish(EPI_PSEUDO, p, g, pdl, st)); ++nl; }
      FIRP_TIMED(KC_RMSNORM);
      FIRP_CUDA(c, launch_rmsnorm(rw, carried, act, c->h, none, (const bf16 *)c->g_attn[j], d, c->x, Rp * d, c->planes[0] == 3 ? 3 : 2, c->ss, pdl, st)); ++nl;
      alive += ins;
    }
    bf16 *kplane = c->kv + (size_t)j * c->kv_layer();
    {
      GemmArgs g = gemm_base(c->x, Rp * d, c->wqkv[j], (H + 2 * Hkv) * dh, d, act);
      g.H = H; g.Hkv = Hkv; g.dh = dh;
      g.l2_ahead = ahead[0];
      set_next(g, 0, EPI_RESIDUAL, c->wo[j], d, nq);
      g.planes = c->planes[0];
      g.rope = c->meta.rope; g.seq_ids = c->seq_ids; g.ctx_len = c->ctx_len; g.pos = c->meta.pos;
      g.q = c->q; g.q_lo_off = Rp * nq; g.kcache = kplane; g.seq_stride = c->kv_seq(); g.kv_stride = c->kv_plane(); g.max_ctx = cfg.max_ctx; g.pages = c->pages();
      Partials p = pending;
      { FIRP_TIMED(KC_GEMM_QKV);
        FIRP_CUDA(c, launch_gemm_tc(EPI_QKV_ROPE, g, pdl, st, &p.sk)); ++nl; }
      FIRP_TIMED(KC_QKV_FINISH);
      FIRP_CUDA(c, launch_gemm_finish(EPI_QKV_ROPE, p, g, pdl, st)); ++nl;
    }
    {
      AttnArgs a{};
      a.rw = rw; a.rows_active = act; a.H = H; a.Hkv = Hkv; a.dh = dh;
      a.q = c->q; a.q_lo_off = Rp * nq; a.kcache = kplane; a.seq_stride = c->kv_seq(); a.kv_stride = c->kv_plane(); a.max_ctx = cfg.max_ctx; a.pages = c->pages();
      a.seq_ids = c->seq_ids; a.ctx_len = c->ctx_len; a.pos = c->meta.pos; a.mask = c->meta.mask;
      a.q_planes = c->attn_planes[0]; a.p_planes = c->attn_planes[1];
      const int tiles = (ra.n_hi_max + act + kAttnTile - 1) / kAttnTile;
      const int G = H / Hkv, qblocks = (act * G + 63) / 64;
      a.splits = attention_splits(rw.n_seq * Hkv * qblocks, tiles);
      a.o = c->o; a.o_lo_off = Rp * nq; a.err = c->dev_status; a.wait_ns = c->wait_ns;
      // Early (programmatic) launch of the mma.sync attention pays only when the rotary finisher before it has well
      // over one CTA per SM (5/4).  Measured at the 7B shape, ms per step with / without it: 35 rows 3.61 / 3.76 at
      // 512 cached tokens and 5.25 / 5.44 at 8192; 67 and 131 rows likewise 0.1 ms better with it; but 27 rows (162
      // CTAs on 148 SMs) 3.70 / 3.66 and 6.30 / 5.33, 19 rows 3.68 / 3.60 and 6.36 / 5.26, 1 row 3.52 / 3.43 and
      // 6.27 / 5.11.  The tensor-core kernel (one CTA per SM, all of them resident and set up before the finisher
      // ends) gains from it at every size: 1 row 3.27 / 3.14 at 512, 27 rows 3.60 / 3.49, 35 rows 3.69 / 3.60.
      const int half_dh = dh / 2, qkv_st = (H + 2 * Hkv + 128 / half_dh - 1) / (128 / half_dh);
      const bool attn_early = pdl && (qkv_st * rw.R * 32 + 255) / 256 >= c->sm_count * 5 / 4;
      bool tc = false;
      if (dh == 128 && c->attn_tc != 0) {
        int qb_tc, qper_tc;
        attention_tc_blocks(act * G, &qb_tc, &qper_tc);
        const int tiles_tc = (ra.n_hi_max + act + kAttnTcTile - 1) / kAttnTcTile;
        // Left to itself the tensor-core kernel takes every step the other kernel would not be launched early for
        // and every step of at most 16 query columns; otherwise those whose longest context spans at least three of
        // its 128-position tiles (four when the query columns need more than one block, eight when several
        // sequences are stepped together): its fixed cost is higher, its tile loop faster.  Measured at the 7B
        // shape, ms per step mma.sync / tcgen05, one sequence: 1 column 3.23 / 3.06 at 64 cached tokens, 3.37 /
        // 3.28 at 512, 5.04 / 4.06 at 8192; 35 columns 3.57 / 3.61 at 64, 3.64 / 3.65 at 128, 3.72 / 3.65 at 512,
        // 5.23 / 4.48 at 8192; 131 columns (three blocks) 5.96 / 5.91 at 64, 6.09 / 6.07 at 256, 10.35 / 9.68 at
        // 8192; 4 sequences x 35 columns 5.77 / 5.88 at 256, 6.78 / 6.36 at 1024, 9.13 / 7.75 at 4096; 16 sequences
        // x 9 columns 6.77 / 6.56 at 256, 19.41 / 12.13 at 4096.
        const int min_tiles = qper_tc <= 16 ? 1 : (rw.n_seq > 1 ? 8 : (qb_tc == 1 ? 3 : 4));
        tc = c->attn_tc > 0 || !attn_early || tiles_tc >= min_tiles;
        if (tc) a.splits = attention_tc_splits(rw.n_seq * Hkv * qb_tc, tiles_tc, c->sm_count);
      }
      FIRP_TIMED(KC_ATTENTION);
      FIRP_CUDA(c, tc ? launch_attention_tc(a, pdl, st) : launch_attention(a, attn_early, st)); ++nl;
    }
    {
      GemmArgs g = gemm_base(c->o, Rp * nq, c->wo[j], d, nq, act);
      g.planes = c->planes[1];
      g.l2_ahead = ahead[1];
      set_next(g, 1, EPI_SWIGLU, c->wgu[j], 2 * F, d);
      FIRP_TIMED(KC_GEMM_O);
      FIRP_CUDA(c, launch_gemm_tc(EPI_RESIDUAL, g, pdl, st, &pending.sk)); ++nl;
    }
    { FIRP_TIMED(KC_RMSNORM);
      FIRP_CUDA(c, launch_rmsnorm(rw, 0, act, c->h, pending, (const bf16 *)c->g_mlp[j], d, c->x, Rp * d, 2, c->ss, pdl, st)); ++nl; }
    pending.sk.U = 0;
    {
      GemmArgs g = gemm_base(c->x, Rp * d, c->wgu[j], 2 * F, d, act);
      g.planes = c->planes[2];
      g.y = c->y; g.y_lo_off = Rp * F; g.F = F; g.l2_ahead = ahead[2];
      set_next(g, 2, EPI_RESIDUAL, c->wd[j], d, F);
      Partials p = pending;
      { FIRP_TIMED(KC_GEMM_GATE_UP);
        FIRP_CUDA(c, launch_gemm_tc(EPI_SWIGLU, g, pdl, st, &p.sk)); ++nl; }
      FIRP_TIMED(KC_SWIGLU_FINISH);
      FIRP_CUDA(c, launch_gemm_finish(EPI_SWIGLU, p, g, pdl, st)); ++nl;
    }
    {
      GemmArgs g = gemm_base(c->y, Rp * F, c->wd[j], d, F, act);
      g.planes = c->planes[3];
      g.l2_ahead = ahead[3];
      if (j + 1 < cfg.n_layers) set_next(g, 3, EPI_QKV_ROPE, c->wqkv[j + 1], (H + 2 * Hkv) * dh, d);
      else if (ra.want_head) set_next(g, 3, EPI_LOGITS, c->w.lm_head, cfg.vocab, d);
      FIRP_TIMED(KC_GEMM_DOWN);
      FIRP_CUDA(c, launch_gemm_tc(EPI_RESIDUAL, g, pdl, st, &pending.sk)); ++nl;
    }
  }
  if (ra.want_head) {
    if (!fused) {
      { FIRP_TIMED(KC_RMSNORM);
        FIRP_CUDA(c, launch_rmsnorm(rw, 0, rw.Ms, c->h, pending, (const bf16 *)c->w.g_final, d, c->x, Rp * d, 2, c->ss, pdl, st)); ++nl; }
      GemmArgs g = gemm_base(c->x, Rp * d, c->w.lm_head, cfg.vocab, d, rw.Ms);
      g.planes = c->planes[4];
      g.logits = ra.logits_dst; g.l2_ahead = ahead[4];
      Partials p = pending;
      { FIRP_TIMED(KC_GEMM_LM_HEAD);
        FIRP_CUDA(c, launch_gemm_tc(EPI_LOGITS, g, pdl, st, &p.sk)); ++nl; }
      FIRP_TIMED(KC_LOGITS_FINISH);
      FIRP_CUDA(c, launch_gemm_finish(EPI_LOGITS, p, g, pdl, st)); ++nl;
    }
    { FIRP_TIMED(KC_TOPB);
      launch_topb(ra.logits_dst, rw.R, cfg.vocab, cfg.top_b, c->cand_ids, c->cand_vals, c->top_ids, c->top_vals, pdl, st);
      nl += 2; }
    AcceptArgs a{};
    a.tokens = ra.d_tokens; a.parents = c->parents; a.next_parents = c->next_parents;
    a.parents_stride = ra.parents_stride; a.sizes = ra.d_sizes;
    a.top_ids = c->top_ids; a.top_vals = c->top_vals; a.T_next = ra.T_next; a.B = cfg.top_b; a.S = c->S;
    a.prefill_last_row = ra.prefill_last_row;
    a.path = c->path; a.n_accepted = c->n_acc; a.accepted = c->accepted; a.next_tokens = c->next_tokens;
    if (out) {
      a.o_path = out->path; a.o_n_accepted = out->n_accepted; a.o_accepted = out->accepted_tokens;
      a.o_next_tokens = out->next_tree_tokens; a.o_best = (ra.prefill_last_row < 0) ? out->best : nullptr;
      a.o_topb_ids = out->topb_ids; a.o_topb_vals = out->topb_vals;
    }
    FIRP_TIMED(KC_ACCEPT);
    launch_accept(rw, a, pdl, st); ++nl;
  }
  FIRP_CUDA(c, cudaGetLastError());
  return FIRP_OK;
}

}  // namespace

extern "C" {

int firp_create(const firp_model_cfg *cfg, firp_ctx **out) {
  if (!cfg || !out) return FIRP_ERR_BAD_ARG;
  *out = nullptr;
  firp_ctx *c = new firp_ctx();
  c->cfg = *cfg;
  auto bad = [&](const char *why) { delete c; fprintf(stderr, "firp_create: %s\n", why); return (int)FIRP_ERR_BAD_ARG; };
  if (cfg->n_layers < 1 || cfg->d_model < 128 || cfg->d_model % 128 || cfg->d_model > 8192) return bad("d_model must be a multiple of 128, <= 8192");
  if (cfg->head_dim != 64 && cfg->head_dim != 128) return bad("head_dim must be 64 or 128");
  if (cfg->n_heads < 1 || cfg->n_kv_heads < 1 || cfg->n_heads % cfg->n_kv_heads) return bad("n_heads must be a multiple of n_kv_heads");
  if (cfg->d_ffn < 8 || cfg->d_ffn % 8 || cfg->vocab < 8) return bad("d_ffn must be a multiple of 8");
  if ((cfg->n_heads * cfg->head_dim) % 8) return bad("bad head geometry");
  if (cfg->max_batch < 1 || cfg->max_batch > kMaxSeq) return bad("max_batch must be 1..16");
  if (cfg->max_tree < 1 || cfg->max_tree > 128 || cfg->max_k < 0 || cfg->max_k > 8) return bad("max_tree <= 128, max_k <= 8");
  if (cfg->max_depth < 0 || cfg->max_depth > 15) return bad("max_depth must be 0..15");
  if (cfg->top_b < 1 || cfg->top_b > kMaxTopB) return bad("top_b must be 1..8");
  if (cfg->max_ctx < cfg->max_tree + cfg->max_k) return bad("max_ctx too small");
  int rows = cfg->max_batch * (cfg->max_tree + cfg->max_k);
  if (rows > 144) return bad("max_batch * (max_tree + max_k) must be <= 144 rows");
  if (cfg->max_rows < 0 || cfg->max_rows > 144) return bad("max_rows must be 0..144");
  if (cfg->max_rows > rows) rows = cfg->max_rows;
  c->row_cap = (int)align_up(rows, 16);
  c->Rmax = 144;          // the workspace always holds the largest row count, so that a prompt is prefilled 141 rows at a time
  c->S = cfg->max_depth + 1;
  c->n_hi.assign(cfg->max_batch, 0);

  c->ws_bytes = c->carve(nullptr);
  *out = c;
  return FIRP_OK;
}

void firp_destroy(firp_ctx *ctx) {
  if (!ctx) return;
  for (cudaEvent_t e : ctx->ev_pool) cudaEventDestroy(e);
  if (ctx->plan_step) fused_plan_destroy(ctx->plan_step);
  if (ctx->plan_prefill) fused_plan_destroy(ctx->plan_prefill);
  delete ctx;
}

const char *firp_last_error(const firp_ctx *ctx) { return ctx ? ctx->err.c_str() : "null context"; }

size_t firp_workspace_bytes(const firp_ctx *ctx) { return ctx ? ctx->ws_bytes : 0; }

size_t firp_kv_bytes(const firp_ctx *ctx) {
  return ctx ? (size_t)ctx->cfg.n_layers * ctx->kv_layer() * sizeof(bf16) : 0;
}

int firp_bind_buffers(firp_ctx *ctx, void *workspace, void *kv_cache, void *stream) {
  if (!ctx) return FIRP_ERR_BAD_ARG;
  if (!workspace || !kv_cache || ((uintptr_t)workspace & 255) || ((uintptr_t)kv_cache & 255))
    return fail(ctx, FIRP_ERR_BAD_ARG, "workspace and kv_cache must be non-NULL and 256-byte aligned");
  cudaStream_t st = (cudaStream_t)stream;
  ctx->carve(workspace);
  ctx->kv = reinterpret_cast<bf16 *>(kv_cache);
  FIRP_CUDA(ctx, cudaMemsetAsync(workspace, 0, ctx->ws_bytes, st));
  std::vector<int32_t> chain(kMaxTreeRows);
  for (int i = 0; i < kMaxTreeRows; ++i) chain[i] = i - 1;
  FIRP_CUDA(ctx, cudaMemcpyAsync(ctx->chain, chain.data(), sizeof(int32_t) * kMaxTreeRows, cudaMemcpyHostToDevice, st));
  FIRP_CUDA(ctx, cudaStreamSynchronize(st));
  std::fill(ctx->n_hi.begin(), ctx->n_hi.end(), 0);
  ctx->last_parents.clear(); ctx->last_next_parents.clear(); ctx->last_seq_ids.clear(); ctx->last_sizes.clear();
  if (!gemm_tc_available())
    return fail(ctx, FIRP_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
  {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) ctx->sm_count = n;
  }
  ctx->bound = true; ctx->stepped = false;
  ++ctx->weights_gen;
  return FIRP_OK;
}

int firp_init_weights(firp_ctx *ctx, const firp_weights *w) {
  if (!ctx || !w) return FIRP_ERR_BAD_ARG;
  const int L = ctx->cfg.n_layers;
  if (!w->embed || !w->lm_head || !w->g_final || !w->wqkv || !w->wo || !w->wgu || !w->wd || !w->g_attn || !w->g_mlp)
    return fail(ctx, FIRP_ERR_BAD_ARG, "missing weight pointer");
  if (w->n_maps < 0 || (w->n_maps > 0 && !w->pred_w)) return fail(ctx, FIRP_ERR_BAD_ARG, "n_maps > 0 needs pred_w");
  auto misaligned = [](const void *p) { return ((uintptr_t)p & 15) != 0; };
  if (misaligned(w->embed) || misaligned(w->lm_head) || misaligned(w->pred_w) || misaligned(w->g_final))
    return fail(ctx, FIRP_ERR_BAD_ARG, "weights must be 16-byte aligned");
  for (int j = 0; j < L; ++j) {
    const void *p[6] = {w->wqkv[j], w->wo[j], w->wgu[j], w->wd[j], w->g_attn[j], w->g_mlp[j]};
    for (int i = 0; i < 6; ++i)
      if (!p[i] || misaligned(p[i])) return fail(ctx, FIRP_ERR_BAD_ARG, "layer %d: NULL or misaligned weight", j);
  }
  ctx->w = *w;
  ctx->wqkv.assign(w->wqkv, w->wqkv + L); ctx->wo.assign(w->wo, w->wo + L); ctx->wgu.assign(w->wgu, w->wgu + L);
  ctx->wd.assign(w->wd, w->wd + L); ctx->g_attn.assign(w->g_attn, w->g_attn + L); ctx->g_mlp.assign(w->g_mlp, w->g_mlp + L);
  ctx->have_weights = true;
  ++ctx->weights_gen;
  return FIRP_OK;
}

static int check_ready(firp_ctx *ctx) {
  if (!ctx) return FIRP_ERR_BAD_ARG;
  if (!ctx->bound) return fail(ctx, FIRP_ERR_STATE, "firp_bind_buffers has not been called");
  if (!ctx->have_weights) return fail(ctx, FIRP_ERR_STATE, "firp_init_weights has not been called");
  return FIRP_OK;
}

static int check_seq_ids(firp_ctx *ctx, int n_seq, const int32_t *seq_ids, std::vector<int32_t> &ids) {
  if (n_seq < 1 || n_seq > ctx->cfg.max_batch) return fail(ctx, FIRP_ERR_CAPACITY, "n_seq %d outside 1..max_batch", n_seq);
  ids.resize(n_seq);
  for (int s = 0; s < n_seq; ++s) {
    ids[s] = seq_ids ? seq_ids[s] : s;
    if (ids[s] < 0 || ids[s] >= ctx->cfg.max_batch) return fail(ctx, FIRP_ERR_BAD_ARG, "seq id %d out of range", ids[s]);
    for (int t = 0; t < s; ++t) if (ids[t] == ids[s]) return fail(ctx, FIRP_ERR_BAD_ARG, "duplicate seq id %d", ids[s]);
  }
  return FIRP_OK;
}

// layers of the prediction steps: non-decreasing and inside the decoder
static int check_layers(firp_ctx *ctx, int k, const int32_t *layers) {
  if (k > 0 && !layers) return fail(ctx, FIRP_ERR_BAD_ARG, "NULL insertion layers");
  for (int i = 0; i < k; ++i) {
    if (layers[i] < 0 || layers[i] >= ctx->cfg.n_layers) return fail(ctx, FIRP_ERR_BAD_ARG, "insertion layer %d outside 0..n_layers-1", layers[i]);
    if (i > 0 && layers[i] < layers[i - 1]) return fail(ctx, FIRP_ERR_BAD_ARG, "insertion layers must not decrease");
  }
  return FIRP_OK;
}

int firp_step(firp_ctx *ctx, int32_t n_seq, const int32_t *seq_ids, const int32_t *d_tree_tokens,
              const int32_t *tree_parents, int32_t T, int32_t k, int32_t l, const firp_step_out *out, void *stream) {
  int32_t layers[8];
  for (int i = 0; i < 8; ++i) layers[i] = l;
  return firp_step_layers(ctx, n_seq, seq_ids, d_tree_tokens, tree_parents, T, k, layers, out, stream);
}

// One chain of k pseudo rows under the root (chains = false) or under every tree node (chains = true).
static int step_impl(firp_ctx *ctx, int32_t n_seq, const int32_t *seq_ids, const int32_t *d_tree_tokens,
                     const int32_t *tree_parents, const int32_t *tree_sizes, int32_t T, int32_t k, const int32_t *layers,
                     bool chains, const firp_step_out *out, void *stream);

int firp_step_layers(firp_ctx *ctx, int32_t n_seq, const int32_t *seq_ids, const int32_t *d_tree_tokens,
                     const int32_t *tree_parents, int32_t T, int32_t k, const int32_t *layers, const firp_step_out *out,
                     void *stream) {
  return step_impl(ctx, n_seq, seq_ids, d_tree_tokens, tree_parents, nullptr, T, k, layers, false, out, stream);
}

int firp_step_chains(firp_ctx *ctx, int32_t n_seq, const int32_t *seq_ids, const int32_t *d_tree_tokens,
                     const int32_t *tree_parents, int32_t T, int32_t k, const int32_t *layers, const firp_step_out *out,
                     void *stream) {
  return step_impl(ctx, n_seq, seq_ids, d_tree_tokens, tree_parents, nullptr, T, k, layers, true, out, stream);
}

int firp_step_trees(firp_ctx *ctx, int32_t n_seq, const int32_t *seq_ids, const int32_t *d_tree_tokens,
                    const int32_t *tree_parents, const int32_t *tree_sizes, int32_t T, int32_t k, const int32_t *layers,
                    const firp_step_out *out, void *stream) {
  if (!tree_sizes) return ctx ? fail(ctx, FIRP_ERR_BAD_ARG, "NULL tree sizes") : (int)FIRP_ERR_BAD_ARG;
  return step_impl(ctx, n_seq, seq_ids, d_tree_tokens, tree_parents, tree_sizes, T, k, layers, false, out, stream);
}

// tree_sizes == NULL: one template tree_parents[T] for all sequences.  Otherwise tree_parents is [n_seq][T] and
// sequence s uses its first tree_sizes[s] entries; the remaining rows are padding, hung under the root.
static int step_impl(firp_ctx *ctx, int32_t n_seq, const int32_t *seq_ids, const int32_t *d_tree_tokens,
                     const int32_t *tree_parents, const int32_t *tree_sizes, int32_t T, int32_t k, const int32_t *layers,
                     bool chains, const firp_step_out *out, void *stream) {
  int rc = check_ready(ctx);
  if (rc) return rc;
  const firp_model_cfg &cfg = ctx->cfg;
  cudaStream_t st = (cudaStream_t)stream;
  if (!d_tree_tokens || !tree_parents) return fail(ctx, FIRP_ERR_BAD_ARG, "NULL tokens or parents");
  if (T < 1 || T > cfg.max_tree) return fail(ctx, FIRP_ERR_CAPACITY, "T %d outside 1..max_tree", T);
  if (k < 0 || k > cfg.max_k || k > ctx->w.n_maps) return fail(ctx, FIRP_ERR_CAPACITY, "k %d exceeds max_k or the loaded maps", k);
  if ((rc = check_layers(ctx, k, layers))) return rc;
  std::vector<int32_t> ids;
  if ((rc = check_seq_ids(ctx, n_seq, seq_ids, ids))) return rc;
  const int pseudo = chains ? T * k : k;       // pseudo rows per sequence
  const int Ms = T + pseudo;
  if (Ms > kMaxTreeRows || n_seq * Ms > ctx->row_cap)
    return fail(ctx, FIRP_ERR_CAPACITY, "%d sequences x %d rows exceed the row capacity %d (max_rows of the configuration)", n_seq, Ms, ctx->row_cap);
  // validate every tree (the shared template, or each sequence's own) and lay the parents out for the device
  const int n_trees = tree_sizes ? n_seq : 1;
  std::vector<int32_t> dev_parents((size_t)n_trees * T);
  for (int t = 0; t < n_trees; ++t) {
    const int32_t *par = tree_parents + (size_t)t * T;
    const int size = tree_sizes ? tree_sizes[t] : T;
    if (size < 1 || size > T) return fail(ctx, FIRP_ERR_BAD_TREE, "tree size %d outside 1..T", size);
    if (size < T && k == 0) return fail(ctx, FIRP_ERR_BAD_TREE, "trees of different sizes need k > 0");
    std::vector<int> depth;
    const int maxd = tree_depths(par, size, depth);
    if (maxd < 0) return fail(ctx, FIRP_ERR_BAD_TREE, "parents[0] must be -1 and 0 <= parents[v] < v");
    if (maxd > cfg.max_depth) return fail(ctx, FIRP_ERR_BAD_TREE, "tree depth %d exceeds max_depth", maxd);
    if (k > 0 && maxd > k) return fail(ctx, FIRP_ERR_BAD_TREE, "tree depth %d exceeds k = %d", maxd, k);
    if (k > 0 && max_sibling_rank(par, size) >= cfg.top_b) return fail(ctx, FIRP_ERR_BAD_TREE, "more siblings than top_b");
    for (int v = 0; v < T; ++v) dev_parents[(size_t)t * T + v] = v < size ? par[v] : 0;   // padding rows: children of the root
  }
  int n_hi_max = 0;
  for (int s = 0; s < n_seq; ++s) {
    if (ctx->n_hi[ids[s]] + Ms > cfg.max_ctx) {
      // the host only keeps an upper bound after device-side commits: before refusing, read the exact length
      int32_t n = 0;
      FIRP_CUDA(ctx, cudaMemcpyAsync(&n, ctx->ctx_len + ids[s], sizeof(int32_t), cudaMemcpyDeviceToHost, st));
      FIRP_CUDA(ctx, cudaStreamSynchronize(st));
      ctx->n_hi[ids[s]] = n;
      if (n + Ms > cfg.max_ctx) return fail(ctx, FIRP_ERR_CAPACITY, "slot %d: context + rows exceeds max_ctx", ids[s]);
    }
    n_hi_max = ctx->n_hi[ids[s]] > n_hi_max ? ctx->n_hi[ids[s]] : n_hi_max;
  }
  ctx->launches = 0;
  if ((rc = upload_i32(ctx, ctx->seq_ids, ids.data(), n_seq, ctx->last_seq_ids, st))) return rc;
  if ((rc = upload_i32(ctx, ctx->parents, dev_parents.data(), n_trees * T, ctx->last_parents, st))) return rc;
  const int32_t one = -1;
  const int T_next = (k > 0) ? T : 1;
  if ((rc = upload_i32(ctx, ctx->next_parents, k > 0 ? dev_parents.data() : &one, k > 0 ? n_trees * T : 1, ctx->last_next_parents, st))) return rc;
  if (tree_sizes && (rc = upload_i32(ctx, ctx->tree_sizes, tree_sizes, n_seq, ctx->last_sizes, st))) return rc;

  RunArgs ra{};
  ra.rw = Rows{n_seq, T, pseudo, Ms, n_seq * Ms, 0, chains ? 1 : 0, k, ctx->pseudo_masked};
  for (int i = 0; i < k; ++i) ra.tl[i] = layers[i];
  ra.d_tokens = d_tree_tokens; ra.want_head = true; ra.prefill_last_row = -1; ra.T_next = T_next;
  ra.out = out; ra.logits_dst = (out && out->logits) ? out->logits : ctx->logits; ra.n_hi_max = n_hi_max;
  ra.parents_stride = tree_sizes ? T : 0; ra.d_sizes = tree_sizes ? ctx->tree_sizes : nullptr;
  if ((rc = run_rows(ctx, ra, st))) return rc;
  ctx->stepped = true; ctx->last_n_seq = n_seq; ctx->last_T = T; ctx->last_k = k;
  return FIRP_OK;
}

int firp_prefill(firp_ctx *ctx, int32_t seq, const int32_t *d_prompt, int32_t P, int32_t k, int32_t l,
                 const int32_t *next_parents, int32_t T_next, const firp_step_out *out, void *stream) {
  int32_t layers[8];
  for (int i = 0; i < 8; ++i) layers[i] = l;
  return firp_prefill_layers(ctx, seq, d_prompt, P, k, layers, next_parents, T_next, out, stream);
}

int firp_prefill_layers(firp_ctx *ctx, int32_t seq, const int32_t *d_prompt, int32_t P, int32_t k, const int32_t *layers,
                        const int32_t *next_parents, int32_t T_next, const firp_step_out *out, void *stream) {
  int rc = check_ready(ctx);
  if (rc) return rc;
  const firp_model_cfg &cfg = ctx->cfg;
  cudaStream_t st = (cudaStream_t)stream;
  if (!d_prompt || P < 1) return fail(ctx, FIRP_ERR_BAD_ARG, "empty prompt");
  if (seq < 0 || seq >= cfg.max_batch) return fail(ctx, FIRP_ERR_BAD_ARG, "seq id out of range");
  if (k < 0 || k > cfg.max_k || k > ctx->w.n_maps) return fail(ctx, FIRP_ERR_CAPACITY, "k exceeds max_k or the loaded maps");
  if ((rc = check_layers(ctx, k, layers))) return rc;
  if (P + k > cfg.max_ctx) return fail(ctx, FIRP_ERR_CAPACITY, "prompt does not fit max_ctx");
  const int32_t one = -1;
  if (k == 0) { next_parents = &one; T_next = 1; }
  if (!next_parents || T_next < 1 || T_next > cfg.max_tree) return fail(ctx, FIRP_ERR_BAD_ARG, "bad next-tree template");
  std::vector<int> depth;
  const int maxd = tree_depths(next_parents, T_next, depth);
  if (maxd < 0 || maxd > k || maxd > cfg.max_depth) return fail(ctx, FIRP_ERR_BAD_TREE, "next-tree template malformed or deeper than k");
  if (k > 0 && max_sibling_rank(next_parents, T_next) >= cfg.top_b) return fail(ctx, FIRP_ERR_BAD_TREE, "more siblings than top_b");

  ctx->launches = 0;
  std::vector<int32_t> ids(1, seq);
  if ((rc = upload_i32(ctx, ctx->seq_ids, ids.data(), 1, ctx->last_seq_ids, st))) return rc;
  if ((rc = upload_i32(ctx, ctx->next_parents, next_parents, T_next, ctx->last_next_parents, st))) return rc;
  // chain template for the prompt rows
  // the prompt runs in chunks of as many rows as the kernels take at once (144 less the pseudo rows of the last
  // chunk): a 512-token prompt is four passes over the weights
  const int chunk = std::min(ctx->Rmax, kMaxTreeRows) - k;
  std::vector<int32_t> chain(chunk);
  for (int i = 0; i < chunk; ++i) chain[i] = i - 1;
  if ((rc = upload_i32(ctx, ctx->parents, chain.data(), chunk, ctx->last_parents, st))) return rc;
  FIRP_CUDA(ctx, cudaMemsetAsync(ctx->ctx_len + seq, 0, sizeof(int32_t), st));
  ctx->n_hi[seq] = 0;

  for (int p0 = 0; p0 < P; p0 += chunk) {
    const int Tc = (P - p0 < chunk) ? P - p0 : chunk;
    const bool last = (p0 + Tc == P);
    const int kc = last ? k : 0;
    RunArgs ra{};
    ra.rw = Rows{1, Tc, kc, Tc + kc, Tc + kc, Tc - 1, 0, kc, ctx->pseudo_masked};
    for (int i = 0; i < kc; ++i) ra.tl[i] = layers[i];
    ra.d_tokens = d_prompt + p0; ra.want_head = last; ra.prefill_last_row = Tc - 1; ra.T_next = T_next;
    ra.out = nullptr; ra.logits_dst = ctx->logits; ra.n_hi_max = ctx->n_hi[seq];
    firp_step_out o2{};
    if (last && out) {
      o2 = *out; o2.logits = nullptr; o2.depth = nullptr; o2.mask = nullptr; o2.best = nullptr; o2.path = nullptr;
      ra.out = &o2;
    }
    if ((rc = run_rows(ctx, ra, st))) return rc;
    if (last && out && out->logits)
      FIRP_CUDA(ctx, cudaMemcpyAsync(out->logits, ctx->logits + (size_t)(Tc - 1) * cfg.vocab,
                                     sizeof(float) * (size_t)(1 + k) * cfg.vocab, cudaMemcpyDeviceToDevice, st));
    launch_advance_ctx(1, ctx->seq_ids, ctx->ctx_len, Tc, ctx->use_pdl, st); ++ctx->launches;
    ctx->n_hi[seq] += Tc;
  }
  FIRP_CUDA(ctx, cudaGetLastError());
  ctx->stepped = false;
  return FIRP_OK;
}

int firp_set_pseudo_masked(firp_ctx *ctx, int32_t masked) {
  if (!ctx) return FIRP_ERR_BAD_ARG;
  ctx->pseudo_masked = masked ? 1 : 0;
  return FIRP_OK;
}

int firp_set_pred_prenorm(firp_ctx *ctx, int32_t on) {
  if (!ctx) return FIRP_ERR_BAD_ARG;
  ctx->pred_prenorm = on ? 1 : 0;
  ++ctx->weights_gen;      // cached launch plans depend on it
  return FIRP_OK;
}

int firp_set_kv_pages(firp_ctx *ctx, const int32_t *page_table, void *stream) {
  if (!ctx) return FIRP_ERR_BAD_ARG;
  if (!ctx->bound) return fail(ctx, FIRP_ERR_STATE, "firp_bind_buffers has not been called");
  cudaStream_t st = (cudaStream_t)stream;
  ++ctx->weights_gen;                      // cached launch plans carry the table pointer
  if (!page_table) { ctx->paged = false; return FIRP_OK; }
  const int pps = ctx->pages_per_seq(), total = ctx->cfg.max_batch * pps;
  if (ctx->cfg.max_ctx % kKvPage) return fail(ctx, FIRP_ERR_BAD_ARG, "a paged cache needs max_ctx to be a multiple of %d", kKvPage);
  std::vector<char> seen(total, 0);
  for (int i = 0; i < total; ++i) {
    const int32_t pg = page_table[i];
    if (pg < 0 || pg >= total || seen[pg]) return fail(ctx, FIRP_ERR_BAD_ARG, "page table entry %d: page %d out of range or used twice", i, pg);
    seen[pg] = 1;
  }
  FIRP_CUDA(ctx, cudaMemcpyAsync(ctx->d_pages, page_table, sizeof(int32_t) * total, cudaMemcpyHostToDevice, st));
  FIRP_CUDA(ctx, cudaStreamSynchronize(st));
  ctx->paged = true;
  return FIRP_OK;
}

int firp_set_activation_planes(firp_ctx *ctx, int32_t qkv, int32_t o, int32_t gate_up, int32_t down, int32_t lm_head) {
  if (!ctx) return FIRP_ERR_BAD_ARG;
  const int32_t p[5] = {qkv, o, gate_up, down, lm_head};
  for (int i = 0; i < 5; ++i)
    if (p[i] < 1 || p[i] > (i == 0 ? 3 : 2)) return fail(ctx, FIRP_ERR_BAD_ARG, "planes must be 1..2 (1..3 for the QKV projection)");
  for (int i = 0; i < 5; ++i) ctx->planes[i] = p[i];
  return FIRP_OK;
}

int firp_set_attention_planes(firp_ctx *ctx, int32_t q_planes, int32_t p_planes) {
  if (!ctx || q_planes < 1 || q_planes > 2 || p_planes < 1 || p_planes > 2) return FIRP_ERR_BAD_ARG;
  ctx->attn_planes[0] = q_planes; ctx->attn_planes[1] = p_planes;
  return FIRP_OK;
}

int firp_set_attention_kernel(firp_ctx *ctx, int32_t tensor_core) {
  if (!ctx || tensor_core < -1 || tensor_core > 1) return FIRP_ERR_BAD_ARG;
  ctx->attn_tc = tensor_core;
  return FIRP_OK;
}

int firp_set_fused(firp_ctx *ctx, int32_t on) {
  if (!ctx) return FIRP_ERR_BAD_ARG;
  ctx->use_fused = on != 0;
  return FIRP_OK;
}

int firp_set_wait_limit_us(firp_ctx *ctx, int64_t usec) {
  if (!ctx || usec < 0) return FIRP_ERR_BAD_ARG;
  ctx->wait_ns = (unsigned long long)usec * 1000ull;
  return FIRP_OK;
}

int firp_selftest_wait(firp_ctx *ctx, void *stream) {
  if (!ctx) return FIRP_ERR_BAD_ARG;
  if (!ctx->bound) return fail(ctx, FIRP_ERR_STATE, "firp_bind_buffers has not been called");
  FIRP_CUDA(ctx, launch_wait_selftest(ctx->dev_status, ctx->wait_ns, (cudaStream_t)stream));
  return FIRP_OK;
}

int firp_kv_commit(firp_ctx *ctx, int32_t n_seq, const int32_t *seq_ids, const int32_t *path, const int32_t *path_len,
                   void *stream) {
  int rc = check_ready(ctx);
  if (rc) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  if (!ctx->stepped) return fail(ctx, FIRP_ERR_STATE, "no step to commit");
  if ((path == nullptr) != (path_len == nullptr)) return fail(ctx, FIRP_ERR_BAD_ARG, "path and path_len go together");
  std::vector<int32_t> ids;
  if ((rc = check_seq_ids(ctx, n_seq, seq_ids, ids))) return rc;
  if (n_seq != ctx->last_n_seq || ids != ctx->last_seq_ids) return fail(ctx, FIRP_ERR_STATE, "commit must name the sequences of the last step");
  const int S = ctx->S;
  CommitArgs a{};
  a.kv = ctx->kv; a.seq_stride = ctx->kv_seq(); a.layer_stride = ctx->kv_layer(); a.kv_stride = ctx->kv_plane();
  a.max_ctx = ctx->cfg.max_ctx; a.pages = ctx->pages();
  a.n_layers = ctx->cfg.n_layers; a.nkv = ctx->cfg.n_kv_heads * ctx->cfg.head_dim; a.seq_ids = ctx->seq_ids;
  a.S = S; a.ctx_len = ctx->ctx_len;
  ctx->launches = 0;
  if (path) {
    for (int s = 0; s < n_seq; ++s) {
      const int len = path_len[s];
      if (len < 1 || len > S) return fail(ctx, FIRP_ERR_BAD_ARG, "path_len %d outside 1..max_depth+1", len);
      const int32_t *p = path + (size_t)s * S;
      if (p[0] != 0) return fail(ctx, FIRP_ERR_BAD_ARG, "path[0] must be the root");
      for (int j = 1; j < len; ++j)
        if (p[j] <= p[j - 1] || p[j] >= ctx->last_T) return fail(ctx, FIRP_ERR_BAD_ARG, "path must be strictly increasing tree rows");
    }
    FIRP_CUDA(ctx, cudaMemcpyAsync(ctx->exp_path, path, sizeof(int32_t) * (size_t)n_seq * S, cudaMemcpyHostToDevice, st));
    FIRP_CUDA(ctx, cudaMemcpyAsync(ctx->exp_len, path_len, sizeof(int32_t) * n_seq, cudaMemcpyHostToDevice, st));
    a.path = ctx->exp_path; a.path_len = ctx->exp_len;
    for (int s = 0; s < n_seq; ++s) ctx->n_hi[ids[s]] += path_len[s];
  } else {
    a.path = ctx->path; a.path_len = ctx->n_acc;
    for (int s = 0; s < n_seq; ++s) ctx->n_hi[ids[s]] += S;   // exact value is on the device; keep an upper bound
  }
  { firp_ctx *c = ctx; FIRP_TIMED(KC_COMMIT);
    launch_commit(n_seq, a, ctx->use_pdl, st); ctx->launches += 2; }
  FIRP_CUDA(ctx, cudaGetLastError());
  ctx->stepped = false;
  return FIRP_OK;
}

int firp_context_len(firp_ctx *ctx, int32_t seq, int32_t *n, void *stream) {
  if (!ctx || !n) return FIRP_ERR_BAD_ARG;
  if (!ctx->bound) return fail(ctx, FIRP_ERR_STATE, "firp_bind_buffers has not been called");
  if (seq < 0 || seq >= ctx->cfg.max_batch) return fail(ctx, FIRP_ERR_BAD_ARG, "seq id out of range");
  cudaStream_t st = (cudaStream_t)stream;
  int status = 0;
  FIRP_CUDA(ctx, cudaMemcpyAsync(n, ctx->ctx_len + seq, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  FIRP_CUDA(ctx, cudaMemcpyAsync(&status, ctx->dev_status, sizeof(int), cudaMemcpyDeviceToHost, st));
  FIRP_CUDA(ctx, cudaStreamSynchronize(st));
  ctx->n_hi[seq] = *n;
  if (status != 0) {   // report once and clear, so that the context can go on after the caller has dealt with it
    FIRP_CUDA(ctx, cudaMemsetAsync(ctx->dev_status, 0, sizeof(int), st));
    FIRP_CUDA(ctx, cudaStreamSynchronize(st));
    return fail(ctx, FIRP_ERR_DEVICE_TIMEOUT, "a kernel gave up a bounded wait (device status %d)", status);
  }
  return FIRP_OK;
}

int firp_set_context_len(firp_ctx *ctx, int32_t seq, int32_t n, void *stream) {
  if (!ctx) return FIRP_ERR_BAD_ARG;
  if (!ctx->bound) return fail(ctx, FIRP_ERR_STATE, "firp_bind_buffers has not been called");
  if (seq < 0 || seq >= ctx->cfg.max_batch || n < 0 || n > ctx->cfg.max_ctx) return fail(ctx, FIRP_ERR_BAD_ARG, "seq or n out of range");
  cudaStream_t st = (cudaStream_t)stream;
  FIRP_CUDA(ctx, cudaMemcpyAsync(ctx->ctx_len + seq, &n, sizeof(int32_t), cudaMemcpyHostToDevice, st));
  FIRP_CUDA(ctx, cudaStreamSynchronize(st));
  ctx->n_hi[seq] = n;
  ctx->stepped = false;
  return FIRP_OK;
}

int firp_last_launch_count(const firp_ctx *ctx) { return ctx ? ctx->launches : 0; }

int firp_profile_enable(firp_ctx *ctx, int32_t on) {
  if (!ctx) return FIRP_ERR_BAD_ARG;
  ctx->profiling = on != 0;
  ctx->ev_used = 0;
  return FIRP_OK;
}

int firp_profile_read(firp_ctx *ctx, void *stream, int32_t n_classes, int32_t *launches, float *usec) {
  if (!ctx || !launches || !usec || n_classes < 0) return FIRP_ERR_BAD_ARG;
  FIRP_CUDA(ctx, cudaStreamSynchronize((cudaStream_t)stream));
  for (int i = 0; i < n_classes; ++i) { launches[i] = 0; usec[i] = 0.f; }
  for (size_t i = 0; i < ctx->ev_used; ++i) {
    float ms = 0.f;
    FIRP_CUDA(ctx, cudaEventElapsedTime(&ms, ctx->ev_pool[2 * i], ctx->ev_pool[2 * i + 1]));
    const int k = ctx->ev_class[i];
    if (k < n_classes) { ++launches[k]; usec[k] += ms * 1e3f; }
  }
  ctx->ev_used = 0;
  return KC_COUNT;
}

const char *firp_kernel_class_name(int32_t c) { return (c >= 0 && c < KC_COUNT) ? kClassNames[c] : nullptr; }

}  // extern "C"
