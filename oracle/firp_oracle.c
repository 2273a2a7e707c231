/*
 * firp_oracle.c -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, single-purpose CPU statement of what one FIRP draft+verify
 * decoder step computes, written from the paper (arXiv 2410.20488) so that the
 * CUDA path can be compared against it.  Nothing in the product may call it:
 * only tests, the smoke check and the benchmark's CPU-baseline leg do.  It
 * shares no code with the CUDA path.
 *
 * Precision: activations and logits are stored as fp32; every reduction (dot
 * products, RMS, softmax, weighted sums) is accumulated in fp64; weights are
 * bf16 bit patterns widened exactly to fp32.  The KV cache is a storage format
 * of the workload, not of the arithmetic: the benchmark configurations fix it
 * as bf16, so with cfg.kv_bf16 != 0 (the default of the Python wrapper) rotated
 * keys and values are rounded once to bf16 (round-to-nearest-even) when they are
 * stored and every reader sees the stored value; with kv_bf16 == 0 the cache
 * holds fp32 (used by the pins that compare against an fp64 library decoder).
 * There is no blocking, fusion or reordering: each function is the formula
 * written out.
 *
 * What is computed, with the passage each part follows:
 *   - Llama-style decoder block (the paper builds on the HuggingFace Llama
 *     architecture, Section 4 "Setup"): RMSNorm, q/k/v projections, rotary
 *     embedding in the rotate-half pairing (c, c + dh/2), softmax attention,
 *     output projection, SwiGLU MLP, residual adds, final RMSNorm, untied
 *     lm-head.
 *   - Tree attention (Section 3.4 "Tree attention"): the flattened tree keeps
 *     each token's positional index n + depth, and a row attends to the
 *     committed prefix plus its own ancestors and itself.
 *   - Pseudo hidden states (Section 3.2, Section 3.3 Eq. 3): at the input of
 *     layer l, k rows h~_i = W_i h[anchor] + b_i are appended.  Section 3.3
 *     gives every prediction step i its own layer t_i (Section 4 "Setup" uses
 *     15/20/25 and 25/30/35): oracle_forward_layers() appends row i at the
 *     input of layer t_i, t_1 <= ... <= t_k, from the anchor's residual there;
 *     oracle_forward() is the case t_1 = ... = t_k = l.  Pseudo row i
 *     stands for position pos[anchor] + i; it sees the prefix, the anchor's
 *     ancestors and the anchor, the earlier pseudo rows ("No masked" setting
 *     of Section 4.3) and itself (Section 3.3, paragraph after Eq. 3).
 *     With one chain (oracle_forward, oracle_forward_layers) the rows hang off
 *     one tree node, the root by default.  oracle_forward_chains keeps such a
 *     chain under every tree node, so that the next candidates can be read from
 *     the chain of the node the acceptance walk ends on (Section 3.4 produces
 *     them from the accepted sequence; the paper does not say how a tree step
 *     does that before the sequence is known).
 *   - Greedy verification (Section 3.4, Section 4 "greedy sampling"): walk
 *     from the root, following the child whose token equals the argmax of the
 *     current row; the walk's nodes are the accepted path, the last argmax is
 *     the bonus token.
 *   - Next tree (Section 3.4): node v at depth j of a static template takes
 *     the rank[v]-th best token of pseudo row j.
 *   - KV compaction: the cache rows of the accepted path move to slots
 *     n .. n+a, and n grows by a+1.
 *
 * Readings where the paper is silent: W is stored [out][in] (h~[o] = sum_c
 * W[o][c] h[c] + b[o]); the map is applied to the raw residual stream; ties in
 * argmax/top-B go to the lowest token id, duplicate sibling tokens to the
 * lowest node index; tree rows never see pseudo rows.
 *
 * Pins: tests/test_oracle_pins.py checks this file against an independent
 * library implementation of the Llama decoder (autoregressive greedy decoding
 * for T=1,k=0; per-path causal forwards for tree rows; a causal forward with
 * rows replaced at layer l for the pseudo chain), closed forms for Eq. 3, and
 * the losslessness invariant of Eq. 1.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
  int32_t L, d, H, Hkv, dh, F, V;
  int32_t max_ctx;   /* cache slots per sequence (committed + one step's rows) */
  int32_t n_maps;    /* predictor maps available (k <= n_maps) */
  int32_t n_seq;     /* independent sequences, each with its own cache */
  int32_t kv_bf16;   /* != 0: keys/values are rounded to bf16 when stored (the cache's storage format) */
  float eps, theta;
} oracle_cfg;

typedef struct {
  const uint16_t *embed;    /* [V][d] */
  const uint16_t *lm_head;  /* [V][d] */
  const uint16_t *g_final;  /* [d] */
  const uint16_t *pred_w;   /* [n_maps][d][d], [out][in] */
  const uint16_t *pred_b;   /* [n_maps][d] or NULL */
  const uint16_t *const *wq, *const *wk, *const *wv;  /* per layer: [H*dh][d], [Hkv*dh][d] x2 */
  const uint16_t *const *wo;                          /* [d][H*dh] */
  const uint16_t *const *wgate, *const *wup;          /* [F][d] */
  const uint16_t *const *wdown;                       /* [d][F] */
  const uint16_t *const *g_attn, *const *g_mlp;       /* [d] */
} oracle_weights;

typedef struct {
  oracle_cfg cfg;
  oracle_weights w;
  int32_t masked;  /* != 0: the "Masked" setting of Section 4.3: a pseudo row does not see other pseudo rows */
  int32_t prenorm; /* != 0: Eq. 3 reads the anchor's state through the RMSNorm of the layer it is inserted at */
  int32_t *n;      /* committed length per sequence */
  float **kc;      /* per sequence: [L][max_ctx][Hkv*dh] */
  float **vc;
} oracle_t;

static inline float bf16f(uint16_t b) {
  union { uint32_t u; float f; } v; v.u = (uint32_t)b << 16; return v.f;
}

/* fp32 -> nearest bf16 (ties to even), returned widened back to fp32 */
static inline float round_bf16(float f) {
  union { float f; uint32_t u; } v; v.f = f;
  if ((v.u & 0x7FFFFFFFu) > 0x7F800000u) return f;
  v.u += 0x7FFFu + ((v.u >> 16) & 1u);
  v.u &= 0xFFFF0000u;
  return v.f;
}

void *oracle_create(const oracle_cfg *cfg) {
  oracle_t *o = (oracle_t *)calloc(1, sizeof(oracle_t));
  o->cfg = *cfg;
  o->n = (int32_t *)calloc(cfg->n_seq, sizeof(int32_t));
  o->kc = (float **)calloc(cfg->n_seq, sizeof(float *));
  o->vc = (float **)calloc(cfg->n_seq, sizeof(float *));
  size_t per = (size_t)cfg->L * cfg->max_ctx * cfg->Hkv * cfg->dh;
  for (int s = 0; s < cfg->n_seq; ++s) {
    o->kc[s] = (float *)calloc(per, sizeof(float));
    o->vc[s] = (float *)calloc(per, sizeof(float));
    if (!o->kc[s] || !o->vc[s]) return NULL;
  }
  return o;
}

void oracle_destroy(void *h) {
  oracle_t *o = (oracle_t *)h;
  if (!o) return;
  for (int s = 0; s < o->cfg.n_seq; ++s) { free(o->kc[s]); free(o->vc[s]); }
  free(o->kc); free(o->vc); free(o->n); free(o);
}

void oracle_set_weights(void *h, const oracle_weights *w) { ((oracle_t *)h)->w = *w; }
/* Section 4.3 compares "No masked" (a pseudo row sees the earlier rows of its chain; the default, what the paper
 * adopts) with "Masked" (it sees none of them: only the prefix, its node's ancestors and node, and itself). */
void oracle_set_masked(void *h, int32_t masked) { ((oracle_t *)h)->masked = masked; }

/* Eq. 3 applies the map to the hidden state h^{t_i} as it stands (Section 3.3; the default here).  A variant the
 * equation's wording leaves open feeds the map what the decoder layer itself would read: the state after the
 * input RMSNorm of layer t_i, h~_i = W_i rmsnorm(h^{t_i}; g_attn[t_i]) + b_i.  prenorm != 0 selects it. */
void oracle_set_prenorm(void *h, int32_t prenorm) { ((oracle_t *)h)->prenorm = prenorm; }

/* The "Masked" setting applied to a visibility matrix of T tree rows + pseudo rows: pseudo rows keep what they
 * see among the tree rows and themselves, and lose every other pseudo row. */
void oracle_mask_pseudo(uint8_t *mask, int32_t T, int32_t M) {
  for (int v = T; v < M; ++v)
    for (int u = T; u < M; ++u) if (u != v) mask[(size_t)v * M + u] = 0;
}
int32_t oracle_context_len(void *h, int32_t seq) { return ((oracle_t *)h)->n[seq]; }
/* Rewind the committed length (rows >= n become scratch again); n = 0 empties the cache. */
void oracle_set_context_len(void *h, int32_t seq, int32_t n) { ((oracle_t *)h)->n[seq] = n; }

/* y[m][o] = sum_c W[o][c] * x[m][c]   (W bf16 [n_out][n_in]; x rows ldx apart; y rows ldy apart) */
static void linear(const uint16_t *W, const float *x, int ldx, float *y, int ldy, int M, int n_in, int n_out) {
#pragma omp parallel
  {
    float *wrow = (float *)malloc(sizeof(float) * n_in);
#pragma omp for schedule(static)
    for (int o = 0; o < n_out; ++o) {
      for (int c = 0; c < n_in; ++c) wrow[c] = bf16f(W[(size_t)o * n_in + c]);
      for (int m = 0; m < M; ++m) {
        const float *xr = x + (size_t)m * ldx;
        double acc = 0.0;
#pragma omp simd reduction(+ : acc)
        for (int c = 0; c < n_in; ++c) acc += (double)wrow[c] * (double)xr[c];
        y[(size_t)m * ldy + o] = (float)acc;
      }
    }
    free(wrow);
  }
}

/* x[m][c] = h[m][c] / sqrt(mean_c h[m][c]^2 + eps) * g[c] */
static void rmsnorm(const float *h, const uint16_t *g, float eps, float *x, int M, int d) {
  for (int m = 0; m < M; ++m) {
    double ss = 0.0;
    for (int c = 0; c < d; ++c) ss += (double)h[(size_t)m * d + c] * (double)h[(size_t)m * d + c];
    double r = 1.0 / sqrt(ss / d + (double)eps);
    for (int c = 0; c < d; ++c) x[(size_t)m * d + c] = (float)((double)h[(size_t)m * d + c] * r * (double)bf16f(g[c]));
  }
}

/* Rotary embedding at position p on one head vector, rotate-half pairing (c, c+dh/2). */
static void rope(float *x, int dh, int p, double theta) {
  int half = dh / 2;
  for (int c = 0; c < half; ++c) {
    double inv_freq = pow(theta, -2.0 * c / dh);
    double ang = (double)p * inv_freq, cs = cos(ang), sn = sin(ang);
    double a = x[c], b = x[c + half];
    x[c] = (float)(a * cs - b * sn);
    x[c + half] = (float)(b * cs + a * sn);
  }
}

/*
 * Tree bookkeeping (Section 3.4 "Tree attention"; Section 3.3 for pseudo rows).
 * Rows 0..T-1 are tree nodes, rows T..T+k-1 the pseudo chain hanging off `anchor`.
 * depth[v], mask[v][u] = 1 iff u is v or an ancestor of v, rank[v] = ordinal of v
 * among its parent's children in index order (tree rows only; rank[0] = 0).
 * Returns 0, or -1 for a malformed tree.
 */
static int tree_ok(const int32_t *parents, int32_t T) {
  if (T < 1 || parents[0] != -1) return 0;
  for (int v = 1; v < T; ++v) if (parents[v] < 0 || parents[v] >= v) return 0;
  return 1;
}

/* depth and ancestor-or-self mask of M rows whose extended parents precede them */
static void closure(const int32_t *ext_parent, int M, int32_t *depth, uint8_t *mask) {
  memset(mask, 0, (size_t)M * M);
  for (int v = 0; v < M; ++v) {
    depth[v] = (ext_parent[v] < 0) ? 0 : depth[ext_parent[v]] + 1;
    for (int u = v; u >= 0; u = ext_parent[u]) mask[(size_t)v * M + u] = 1;
  }
}

static void sibling_ranks(const int32_t *parents, int32_t T, int32_t *rank) {
  for (int v = 0; v < T; ++v) {
    int r = 0;
    for (int u = 1; u < v; ++u) if (parents[u] == parents[v]) ++r;
    rank[v] = (v == 0) ? 0 : r;
  }
}

int32_t oracle_tree_prep(const int32_t *parents, int32_t T, int32_t k, int32_t anchor,
                         int32_t *ext_parent, int32_t *depth, uint8_t *mask, int32_t *rank) {
  if (!tree_ok(parents, T) || anchor < 0 || anchor >= T) return -1;
  for (int v = 0; v < T; ++v) ext_parent[v] = parents[v];
  for (int i = 1; i <= k; ++i) ext_parent[T + i - 1] = (i == 1) ? anchor : T + i - 2;
  closure(ext_parent, T + k, depth, mask);
  if (rank) sibling_ranks(parents, T, rank);
  return 0;
}

/*
 * The same bookkeeping when EVERY tree node v carries its own chain of k pseudo rows
 * (Section 3.4 generates the next candidates from the accepted sequence, which is only
 * known after the pass, so a chain is kept for every node the walk may end on; Section
 * 3.3: chain row i of node v stands for position pos[v] + i and sees what v sees, the
 * earlier rows of its own chain and itself).  Rows: 0..T-1 tree nodes, then step-major
 * row(v, i) = T + (i-1)*T + v for i = 1..k, so M = T*(1+k).
 */
int32_t oracle_tree_prep_chains(const int32_t *parents, int32_t T, int32_t k,
                                int32_t *ext_parent, int32_t *depth, uint8_t *mask, int32_t *rank) {
  if (!tree_ok(parents, T) || k < 0) return -1;
  for (int v = 0; v < T; ++v) ext_parent[v] = parents[v];
  for (int i = 1; i <= k; ++i)
    for (int v = 0; v < T; ++v) ext_parent[T + (i - 1) * T + v] = (i == 1) ? v : T + (i - 2) * T + v;
  closure(ext_parent, T * (1 + k), depth, mask);
  if (rank) sibling_ranks(parents, T, rank);
  return 0;
}

/*
 * One forward pass over the T tree rows and pn pseudo rows of sequence `seq`, on top of
 * its committed cache of n positions.  Pseudo row r (row T + r) is W_step h[src] + b_step
 * (Eq. 3) on the residual entering layer tl[step[r]] and is alive from that layer on; the
 * rows are ordered by that layer.  Cache slots n..n+T+pn-1 receive the rows' keys/values
 * (scratch until oracle_commit; a pseudo row has none below its own layer).
 *
 * depth, mask [M], [M][M]: position offset and visibility of every row (M = T + pn)
 * logits      [M][V] fp32 out; rows < logit_row0 are skipped (left untouched)
 * dump_layer, h_dump   optional [M][d]: residual stream entering layer dump_layer,
 *             after that layer's insertions (rows not yet alive are zero)
 * h_ins       optional [pn][d]: every pseudo row as it was appended
 * Returns 0 or -2 (capacity).
 */
static int32_t forward_core(oracle_t *o, int32_t seq, const int32_t *tokens, int32_t T, int32_t pn,
                            const int32_t *p_src, const int32_t *p_step, const int32_t *tl,
                            const int32_t *depth, const uint8_t *mask, int32_t logit_row0, float *logits,
                            int32_t dump_layer, float *h_dump, float *h_ins) {
  const oracle_cfg *c = &o->cfg;
  const oracle_weights *w = &o->w;
  const int d = c->d, H = c->H, Hkv = c->Hkv, dh = c->dh, F = c->F, V = c->V;
  const int nq = H * dh, nkv = Hkv * dh, M = T + pn, n = o->n[seq];
  if (n + M > c->max_ctx) return -2;

  float *h = (float *)calloc((size_t)M * d, sizeof(float));
  float *x = (float *)calloc((size_t)M * d, sizeof(float));
  float *q = (float *)calloc((size_t)M * nq, sizeof(float));
  float *att = (float *)calloc((size_t)M * nq, sizeof(float));
  float *delta = (float *)calloc((size_t)M * d, sizeof(float));
  float *gate = (float *)calloc((size_t)M * F, sizeof(float));
  float *up = (float *)calloc((size_t)M * F, sizeof(float));
  double *p = (double *)malloc(sizeof(double) * (n + M));

  /* token embeddings of the tree rows */
  for (int v = 0; v < T; ++v)
    for (int cc = 0; cc < d; ++cc) h[(size_t)v * d + cc] = bf16f(w->embed[(size_t)tokens[v] * d + cc]);

  int rows = T;  /* rows alive: the tree rows and the pseudo rows whose layer has been reached */
  for (int j = 0; j < c->L; ++j) {
    for (int r = 0; r < pn; ++r) {
      const int i = p_step[r];
      if (tl[i] != j) continue;
      /* Eq. 3: h~ = W_i h[src] + b_i on the residual entering layer t_i, appended as row T+r */
      float *dst = h + (size_t)(T + r) * d;
      const float *src = h + (size_t)p_src[r] * d;
      if (o->prenorm) {   /* variant: the map reads the anchor through layer j's input norm */
        rmsnorm(src, w->g_attn[j], c->eps, x, 1, d);
        src = x;
      }
      linear(w->pred_w + (size_t)i * d * d, src, d, dst, d, 1, d, d);
      if (w->pred_b) for (int cc = 0; cc < d; ++cc) dst[cc] += bf16f(w->pred_b[(size_t)i * d + cc]);
      if (h_ins) memcpy(h_ins + (size_t)r * d, dst, sizeof(float) * d);
      rows = T + r + 1;
    }
    if (h_dump && j == dump_layer) memcpy(h_dump, h, sizeof(float) * (size_t)M * d);

    float *kc = o->kc[seq] + (size_t)j * c->max_ctx * nkv;
    float *vc = o->vc[seq] + (size_t)j * c->max_ctx * nkv;

    /* attention block */
    rmsnorm(h, w->g_attn[j], c->eps, x, rows, d);
    linear(w->wq[j], x, d, q, nq, rows, d, nq);
    linear(w->wk[j], x, d, kc + (size_t)n * nkv, nkv, rows, d, nkv);
    linear(w->wv[j], x, d, vc + (size_t)n * nkv, nkv, rows, d, nkv);
    for (int v = 0; v < rows; ++v) {
      int pos = n + depth[v];
      for (int hd = 0; hd < H; ++hd) rope(q + (size_t)v * nq + hd * dh, dh, pos, c->theta);
      for (int hd = 0; hd < Hkv; ++hd) rope(kc + (size_t)(n + v) * nkv + hd * dh, dh, pos, c->theta);
    }
    if (c->kv_bf16) {   /* the cache stores bf16: round once, on store */
      for (size_t i = 0; i < (size_t)rows * nkv; ++i) {
        kc[(size_t)n * nkv + i] = round_bf16(kc[(size_t)n * nkv + i]);
        vc[(size_t)n * nkv + i] = round_bf16(vc[(size_t)n * nkv + i]);
      }
    }
    for (int v = 0; v < rows; ++v) {
      for (int hd = 0; hd < H; ++hd) {
        const int kvh = hd / (H / Hkv);
        const float *qv = q + (size_t)v * nq + hd * dh;
        /* scores over the committed prefix and the visible new rows */
        double mx = -INFINITY;
        for (int u = 0; u < n + rows; ++u) {
          int visible = (u < n) || mask[(size_t)v * M + (u - n)];
          if (!visible) { p[u] = -INFINITY; continue; }
          const float *ku = kc + (size_t)u * nkv + kvh * dh;
          double s = 0.0;
          for (int cc = 0; cc < dh; ++cc) s += (double)qv[cc] * (double)ku[cc];
          p[u] = s / sqrt((double)dh);
          if (p[u] > mx) mx = p[u];
        }
        double sum = 0.0;
        for (int u = 0; u < n + rows; ++u) { p[u] = (p[u] == -INFINITY) ? 0.0 : exp(p[u] - mx); sum += p[u]; }
        for (int cc = 0; cc < dh; ++cc) {
          double acc = 0.0;
          for (int u = 0; u < n + rows; ++u) acc += p[u] * (double)vc[(size_t)u * nkv + kvh * dh + cc];
          att[(size_t)v * nq + hd * dh + cc] = (float)(acc / sum);
        }
      }
    }
    linear(w->wo[j], att, nq, delta, d, rows, nq, d);
    for (size_t i = 0; i < (size_t)rows * d; ++i) h[i] += delta[i];

    /* SwiGLU MLP block */
    rmsnorm(h, w->g_mlp[j], c->eps, x, rows, d);
    linear(w->wgate[j], x, d, gate, F, rows, d, F);
    linear(w->wup[j], x, d, up, F, rows, d, F);
    for (size_t i = 0; i < (size_t)rows * F; ++i) {
      double g = gate[i];
      gate[i] = (float)(g / (1.0 + exp(-g)) * (double)up[i]);
    }
    linear(w->wdown[j], gate, F, delta, d, rows, F, d);
    for (size_t i = 0; i < (size_t)rows * d; ++i) h[i] += delta[i];
  }

  /* final norm + original lm-head on every row (Section 3.2) */
  rmsnorm(h, w->g_final, c->eps, x, M, d);
  if (logit_row0 < 0) logit_row0 = 0;
  if (logits && logit_row0 < M)
    linear(w->lm_head, x + (size_t)logit_row0 * d, d, logits + (size_t)logit_row0 * V, V, M - logit_row0, d, V);

  free(h); free(x); free(q); free(att); free(delta); free(gate); free(up); free(p);
  return 0;
}

static int layers_ok(const oracle_cfg *c, int32_t k, const int32_t *tl) {
  if (k < 0 || k > c->n_maps) return 0;
  for (int i = 0; i < k; ++i) if (tl[i] < 0 || tl[i] >= c->L || (i > 0 && tl[i] < tl[i - 1])) return 0;
  return 1;
}

/*
 * The step with one chain of k pseudo rows hanging off tree node `anchor`: pseudo row i
 * (row T+i) is appended at the input of layer tl[i] (non-decreasing, 0 <= tl[i] < L).
 * h_ins optional [k][d].  Returns 0, -1 malformed tree or layers, -2 capacity.
 */
int32_t oracle_forward_layers(void *hnd, int32_t seq, const int32_t *tokens, const int32_t *parents,
                              int32_t T, int32_t k, const int32_t *tl, int32_t anchor, int32_t logit_row0,
                              float *logits, int32_t *depth_out, uint8_t *mask_out,
                              int32_t dump_layer, float *h_dump, float *h_ins) {
  oracle_t *o = (oracle_t *)hnd;
  if (!layers_ok(&o->cfg, k, tl)) return -1;
  const int M = T + k;
  int32_t *ext_parent = (int32_t *)malloc(sizeof(int32_t) * M);
  int32_t *depth = (int32_t *)malloc(sizeof(int32_t) * M);
  uint8_t *mask = (uint8_t *)malloc((size_t)M * M);
  int32_t *src = (int32_t *)malloc(sizeof(int32_t) * (k + 1)), *step = (int32_t *)malloc(sizeof(int32_t) * (k + 1));
  int32_t rc = -1;
  if (oracle_tree_prep(parents, T, k, anchor, ext_parent, depth, mask, NULL) == 0) {
    if (o->masked) oracle_mask_pseudo(mask, T, M);
    for (int i = 0; i < k; ++i) { src[i] = anchor; step[i] = i; }
    rc = forward_core(o, seq, tokens, T, k, src, step, tl, depth, mask, logit_row0, logits, dump_layer, h_dump, h_ins);
    if (depth_out) memcpy(depth_out, depth, sizeof(int32_t) * M);
    if (mask_out) memcpy(mask_out, mask, (size_t)M * M);
  }
  free(ext_parent); free(depth); free(mask); free(src); free(step);
  return rc;
}

/*
 * The step with a chain of k pseudo rows under EVERY tree node (see oracle_tree_prep_chains
 * for the row order): chain row i of node v is W_i h[v] + b_i on v's residual entering
 * layer tl[i].  logits [T*(1+k)][V].  Returns 0, -1 malformed tree or layers, -2 capacity.
 */
int32_t oracle_forward_chains(void *hnd, int32_t seq, const int32_t *tokens, const int32_t *parents,
                              int32_t T, int32_t k, const int32_t *tl, int32_t logit_row0,
                              float *logits, int32_t *depth_out, uint8_t *mask_out, float *h_ins) {
  oracle_t *o = (oracle_t *)hnd;
  if (!layers_ok(&o->cfg, k, tl)) return -1;
  const int pn = T * k, M = T + pn;
  int32_t *ext_parent = (int32_t *)malloc(sizeof(int32_t) * M);
  int32_t *depth = (int32_t *)malloc(sizeof(int32_t) * M);
  uint8_t *mask = (uint8_t *)malloc((size_t)M * M);
  int32_t *src = (int32_t *)malloc(sizeof(int32_t) * (pn + 1)), *step = (int32_t *)malloc(sizeof(int32_t) * (pn + 1));
  int32_t rc = -1;
  if (oracle_tree_prep_chains(parents, T, k, ext_parent, depth, mask, NULL) == 0) {
    if (o->masked) oracle_mask_pseudo(mask, T, M);
    for (int i = 0; i < k; ++i)
      for (int v = 0; v < T; ++v) { src[i * T + v] = v; step[i * T + v] = i; }
    rc = forward_core(o, seq, tokens, T, pn, src, step, tl, depth, mask, logit_row0, logits, -1, NULL, h_ins);
    if (depth_out) memcpy(depth_out, depth, sizeof(int32_t) * M);
    if (mask_out) memcpy(mask_out, mask, (size_t)M * M);
  }
  free(ext_parent); free(depth); free(mask); free(src); free(step);
  return rc;
}

/* The single-layer case of the paper's overview (Section 3.2): every prediction step at layer l. */
int32_t oracle_forward(void *hnd, int32_t seq, const int32_t *tokens, const int32_t *parents,
                       int32_t T, int32_t k, int32_t l, int32_t anchor, int32_t logit_row0,
                       float *logits, int32_t *depth_out, uint8_t *mask_out, float *h_at_l) {
  int32_t tl[64];
  if (k < 0 || k > 64) return -1;
  for (int i = 0; i < k; ++i) tl[i] = l;
  return oracle_forward_layers(hnd, seq, tokens, parents, T, k, tl, anchor, logit_row0, logits, depth_out, mask_out,
                               l, h_at_l, NULL);
}

/* argmax with ties to the lowest index */
static int32_t argmax_row(const float *row, int V) {
  int32_t best = 0;
  for (int t = 1; t < V; ++t) if (row[t] > row[best]) best = t;
  return best;
}

/*
 * Greedy verification (Section 3.4): best[v] = argmax logits[v] for tree rows;
 * path[0] = 0; from cur, move to the lowest-index child whose token equals
 * best[cur]; stop when there is none.  accepted = tokens of path[1..a] followed
 * by the bonus token best[path[a]].  Returns a+1 (tokens emitted).
 */
int32_t oracle_verify(const float *logits, const int32_t *tokens, const int32_t *parents, int32_t T, int32_t V,
                      int32_t *best, int32_t *path, int32_t *accepted) {
  for (int v = 0; v < T; ++v) best[v] = argmax_row(logits + (size_t)v * V, V);
  int cur = 0, a = 0;
  path[0] = 0;
  for (;;) {
    int next = -1;
    for (int ch = cur + 1; ch < T; ++ch)
      if (parents[ch] == cur && tokens[ch] == best[cur]) { next = ch; break; }
    if (next < 0) break;
    accepted[a] = tokens[next];
    path[++a] = next;
    cur = next;
  }
  accepted[a] = best[cur];
  return a + 1;
}

/*
 * Top-B of each pseudo row, ordered by (value descending, id ascending), and the
 * next tree on a static template (Section 3.4): next[0] = bonus; a node at depth
 * j >= 1 with sibling rank r takes topb[j-1][r].  Returns 0, or -1 if the
 * template needs a depth beyond k or a rank beyond B.
 */
int32_t oracle_next_tree(const float *logits, int32_t T, int32_t k, int32_t V, int32_t B, int32_t bonus,
                         const int32_t *next_parents, int32_t T_next,
                         int32_t *topb_ids, float *topb_vals, int32_t *next_tokens) {
  for (int i = 0; i < k; ++i) {
    const float *row = logits + (size_t)(T + i) * V;
    for (int b = 0; b < B; ++b) {
      int32_t pick = -1;
      for (int t = 0; t < V; ++t) {
        int taken = 0;
        for (int e = 0; e < b; ++e) if (topb_ids[i * B + e] == t) taken = 1;
        if (taken) continue;
        if (pick < 0 || row[t] > row[pick]) pick = t;
      }
      topb_ids[i * B + b] = pick;
      topb_vals[i * B + b] = row[pick];
    }
  }
  int32_t *depth = (int32_t *)malloc(sizeof(int32_t) * T_next);
  int rc = 0;
  next_tokens[0] = bonus;
  depth[0] = 0;
  for (int v = 1; v < T_next; ++v) {
    depth[v] = depth[next_parents[v]] + 1;
    int r = 0;
    for (int u = 1; u < v; ++u) if (next_parents[u] == next_parents[v]) ++r;
    if (depth[v] > k || r >= B) { rc = -1; break; }
    next_tokens[v] = topb_ids[(depth[v] - 1) * B + r];
  }
  free(depth);
  return rc;
}

/*
 * Commit: cache rows of path[j] (row index within the last step) move to slot
 * n + j in every layer; n += len.  path is strictly increasing with path[j] >= j.
 */
int32_t oracle_commit(void *hnd, int32_t seq, const int32_t *path, int32_t len) {
  oracle_t *o = (oracle_t *)hnd;
  const oracle_cfg *c = &o->cfg;
  const int nkv = c->Hkv * c->dh, n = o->n[seq];
  if (n + len > c->max_ctx) return -2;
  for (int j = 0; j < len; ++j) if (path[j] < j || (j > 0 && path[j] <= path[j - 1])) return -1;
  for (int lay = 0; lay < c->L; ++lay) {
    float *kc = o->kc[seq] + (size_t)lay * c->max_ctx * nkv;
    float *vc = o->vc[seq] + (size_t)lay * c->max_ctx * nkv;
    for (int j = 0; j < len; ++j) {
      if (path[j] == j) continue;
      memmove(kc + (size_t)(n + j) * nkv, kc + (size_t)(n + path[j]) * nkv, sizeof(float) * nkv);
      memmove(vc + (size_t)(n + j) * nkv, vc + (size_t)(n + path[j]) * nkv, sizeof(float) * nkv);
    }
  }
  o->n[seq] = n + len;
  return 0;
}

/* Read one committed/scratch cache row (tests of the compaction). which: 0 = K, 1 = V. */
void oracle_read_cache(void *hnd, int32_t seq, int32_t layer, int32_t which, int32_t slot, float *out) {
  oracle_t *o = (oracle_t *)hnd;
  const oracle_cfg *c = &o->cfg;
  const int nkv = c->Hkv * c->dh;
  const float *base = (which ? o->vc[seq] : o->kc[seq]) + ((size_t)layer * c->max_ctx + slot) * nkv;
  memcpy(out, base, sizeof(float) * nkv);
}

/* Test aid: overwrite cache rows slot0 .. slot0+count-1 of one layer with given bf16 rows (widened exactly).
 * Lets a harness start both implementations from the same seeded prefix without running a prefill;
 * no arithmetic of the method is involved.  which: 0 keys, 1 values. */
void oracle_write_cache(void *hnd, int32_t seq, int32_t layer, int32_t which, int32_t slot0, int32_t count,
                        const uint16_t *rows) {
  oracle_t *o = (oracle_t *)hnd;
  const oracle_cfg *c = &o->cfg;
  const int nkv = c->Hkv * c->dh;
  float *base = (which ? o->vc[seq] : o->kc[seq]) + ((size_t)layer * c->max_ctx + slot0) * nkv;
  for (size_t i = 0; i < (size_t)count * nkv; ++i) base[i] = bf16f(rows[i]);
}
