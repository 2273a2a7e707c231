/*
 * firp.h -- C ABI of the B200 (sm_100a) FIRP draft+verify decoder step.
 *
 * FIRP (arXiv 2410.20488) is single-model speculative decoding: at an
 * intermediate layer l, k trainable linear maps predict pseudo hidden states of
 * the next k positions (Section 3.2, Section 3.3 Eq. 3); they pass through the
 * remaining layers and the original lm-head and yield the draft tokens of the
 * next round, while the same forward pass verifies the current draft tree with
 * tree attention (Section 3.4).
 *
 * Conventions
 *   - All calls return 0 (FIRP_OK) or a negative firp_status; firp_last_error()
 *     returns a message for the last failure on that context.
 *   - "device" pointers are CUDA device memory of the current device, "host"
 *     pointers ordinary host memory.  The library allocates NO device memory:
 *     the caller provides the workspace, the KV cache, the weights and every
 *     output buffer, and keeps them alive while the context uses them.
 *   - Work is enqueued on the given CUDA stream (a cudaStream_t passed as
 *     void*, NULL = the legacy default stream) and nothing synchronises unless
 *     stated.  One context must be driven from one stream at a time.
 *   - Weight matrices are bf16, row-major [out][in].  Token ids are int32.
 *   - Rows of a step: for each of the n_seq sequences, rows 0..T-1 are the tree
 *     nodes (row 0 = root = the last emitted, not yet cached token) and rows
 *     T..T+k-1 the pseudo hidden states, a chain hanging off the root.
 */
#ifndef FIRP_H_
#define FIRP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  FIRP_OK = 0,
  FIRP_ERR_BAD_ARG = -1,   /* NULL pointer, size out of range, misaligned buffer */
  FIRP_ERR_BAD_TREE = -2,  /* parents[0] != -1, parents[v] >= v, depth beyond the limit */
  FIRP_ERR_CAPACITY = -3,  /* context + rows would exceed max_ctx, or a max_* of the config */
  FIRP_ERR_CUDA = -4,      /* a CUDA runtime call failed (message has the CUDA error) */
  FIRP_ERR_STATE = -5,     /* call out of order (no buffers bound, no weights, no step to commit) */
  FIRP_ERR_DEVICE_TIMEOUT = -6 /* a kernel's bounded wait ran out; results since the last check are invalid */
} firp_status;

typedef struct firp_ctx firp_ctx;

/* Decoder shape and capacity limits (Llama-style block: RMSNorm, rotary embedding in
 * the rotate-half pairing, grouped-query attention, SwiGLU MLP, untied lm-head). */
typedef struct {
  int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab;
  float rms_eps, rope_theta;
  int32_t max_batch;  /* sequences with a KV cache (slots 0..max_batch-1) */
  int32_t max_ctx;    /* cache positions per sequence, committed + one step's rows */
  int32_t max_tree;   /* largest T (tree rows per sequence, root included), <= 128 */
  int32_t max_k;      /* largest k (pseudo rows per sequence), <= 8 */
  int32_t max_depth;  /* largest tree depth; paths and accepted lists hold max_depth+1 entries */
  int32_t top_b;      /* candidates kept per pseudo row, 1..8 */
  int32_t max_rows;   /* rows one step may carry over all its sequences, <= 144; 0 = max_batch * (max_tree +
                         max_k).  firp_step_chains needs n_seq * T * (1 + k) rows: raise it for that call. */
} firp_model_cfg;

/* Device pointers to bf16 weights.  wqkv..g_mlp are HOST arrays of n_layers device pointers.
 * wqkv: [(n_heads + 2 n_kv_heads) * head_dim][d_model], q rows, then k rows, then v rows.
 * wo:   [d_model][n_heads * head_dim].   wgu: [2 d_ffn][d_model], gate rows then up rows.
 * wd:   [d_model][d_ffn].   g_attn, g_mlp, g_final: [d_model] RMSNorm gains.
 * embed, lm_head: [vocab][d_model].
 * pred_w: [n_maps][d_model][d_model] maps of Eq. 3, [out][in]; pred_b: [n_maps][d_model] or NULL.
 * Every matrix pointer must be 16-byte aligned. */
typedef struct {
  const void *embed, *lm_head, *g_final;
  const void *pred_w, *pred_b;
  int32_t n_maps;
  const void *const *wqkv, *const *wo, *const *wgu, *const *wd, *const *g_attn, *const *g_mlp;
} firp_weights;

/* Caller-owned DEVICE output buffers of one step; S = max_depth + 1, B = top_b.
 * Any pointer may be NULL (that result is then kept internal or not produced). */
typedef struct {
  int32_t *accepted_tokens;   /* [n_seq][S]  tokens emitted: accepted drafts, then the bonus token; only the first
                                 n_accepted entries of a row are written */
  int32_t *n_accepted;        /* [n_seq]     a + 1 */
  int32_t *path;              /* [n_seq][S]  accepted row indices, path[0] = 0: the KV compaction indices */
  int32_t *next_tree_tokens;  /* [n_seq][T_next] tokens of the next draft tree on the template */
  int32_t *best;              /* [n_seq][T]  greedy token of every tree row */
  int32_t *topb_ids;          /* [n_seq][k][B] candidates of pseudo row i, by (value desc, id asc) */
  float *topb_vals;           /* [n_seq][k][B] */
  float *logits;              /* [n_seq][T+k][vocab] fp32 */
  int32_t *depth;             /* [n_seq][T+k] depth of every row (position = context length + depth) */
  uint32_t *mask;             /* [n_seq][T+k][ceil((T+k)/32)] bit u of row v: row v attends to new row u */
} firp_step_out;

/* Create / destroy a context (host object only). */
int firp_create(const firp_model_cfg *cfg, firp_ctx **out);
void firp_destroy(firp_ctx *ctx);
const char *firp_last_error(const firp_ctx *ctx);

/* Bytes of device memory the caller must provide: scratch workspace and bf16 KV cache
 * (layout [layer][K|V][row][kv_head][head_dim] with row = slot * max_ctx + position, or, with a page table
 * (firp_set_kv_pages), row = page * 64 + position % 64). */
size_t firp_workspace_bytes(const firp_ctx *ctx);
size_t firp_kv_bytes(const firp_ctx *ctx);

/* Bind caller-allocated device buffers (256-byte aligned, at least the sizes above).
 * Zeroes the workspace on `stream` and resets every sequence to an empty context. */
int firp_bind_buffers(firp_ctx *ctx, void *workspace, void *kv_cache, void *stream);

/* Register the weights (pointers are stored, data is not copied). */
int firp_init_weights(firp_ctx *ctx, const firp_weights *w);

/*
 * Prefill sequence slot `seq` from an empty context: runs the P prompt tokens as a chain
 * (the plain "n + k hidden states" picture of Section 3.2, anchor = last prompt token),
 * caches all P rows, and returns in `out`: accepted_tokens[0] = the first root token
 * (greedy next token), n_accepted = 1, next_tree_tokens = the first draft tree on the
 * template `next_parents` (HOST, [T_next]), topb_*; logits (if given) holds 1+k rows:
 * the last prompt row, then the pseudo rows.  d_prompt is a DEVICE array [P].
 * k = 0 gives plain prefill (T_next must then be 1).  The prompt is processed 144 - k rows at a time
 * (one pass over the weights per chunk), whatever max_rows is.
 */
int firp_prefill(firp_ctx *ctx, int32_t seq, const int32_t *d_prompt, int32_t P, int32_t k, int32_t l,
                 const int32_t *next_parents, int32_t T_next, const firp_step_out *out, void *stream);

/*
 * One fused draft+verify step (Section 3.4) for n_seq sequences.
 *   seq_ids        HOST [n_seq] cache slots taking part (NULL = 0..n_seq-1), distinct
 *   d_tree_tokens  DEVICE [n_seq][T] tokens of each draft tree, node 0 = root
 *   tree_parents   HOST [T]: static tree template shared by the sequences,
 *                  parents[0] = -1, parents[v] < v; depth <= k when k > 0
 *   k, l           pseudo rows and 0-based insertion layer (input of layer l), 0 <= l < n_layers
 * Verifies every tree greedily (a draft token is accepted iff it equals the argmax of its
 * parent row; ties to the lowest token id, duplicate siblings to the lowest node), and builds
 * the next tree on the same template from the top-B of the pseudo rows: a node at depth j
 * with sibling rank r takes candidate r of pseudo row j.  With k = 0 the next tree is the
 * bonus token alone.  Keys/values of the rows are written to cache slots n..n+T+k-1, which
 * stay scratch until firp_kv_commit; the committed context is not changed.
 */
int firp_step(firp_ctx *ctx, int32_t n_seq, const int32_t *seq_ids, const int32_t *d_tree_tokens,
              const int32_t *tree_parents, int32_t T, int32_t k, int32_t l, const firp_step_out *out,
              void *stream);

/*
 * The same two calls with one insertion layer per prediction step (Section 3.3: step i is
 * trained on, and its pseudo hidden state predicted at, its own layer t_i; Section 4 "Setup"
 * uses 15/20/25 for the 7B and 25/30/35 for the 13B models).
 *   layers   HOST [k], non-decreasing, 0 <= layers[i] < n_layers: pseudo row i is appended at the
 *            input of layer layers[i] as W_i h[anchor] + b_i on the anchor's residual entering that
 *            layer, and takes part in every layer from there on (it has no keys/values below it).
 * layers[i] = l for every i is firp_step / firp_prefill with that l.  FIRP_ERR_BAD_ARG if the
 * layers decrease or leave the decoder; everything else as in the calls above.
 */
int firp_prefill_layers(firp_ctx *ctx, int32_t seq, const int32_t *d_prompt, int32_t P, int32_t k,
                        const int32_t *layers, const int32_t *next_parents, int32_t T_next,
                        const firp_step_out *out, void *stream);
int firp_step_layers(firp_ctx *ctx, int32_t n_seq, const int32_t *seq_ids, const int32_t *d_tree_tokens,
                     const int32_t *tree_parents, int32_t T, int32_t k, const int32_t *layers,
                     const firp_step_out *out, void *stream);

/*
 * The step with a chain of k pseudo rows under EVERY tree node instead of one chain under the
 * root.  Section 3.4 draws the next candidates from the accepted sequence, which a tree step only
 * knows after the pass; with a chain per node the next tree is read from the chain of the node the
 * acceptance walk ends on, so depth-j candidates are predictions for exactly the position they
 * will occupy (with the single chain of firp_step they are predictions made from the root).
 * Rows per sequence: T tree rows, then chain row i (1-based) of node v at row T + (i-1) T + v,
 * T (1 + k) in all (depth, mask, logits of `out` have that many rows; best, path, accepted,
 * next_tree_tokens as in firp_step; topb_ids / topb_vals [n_seq][k][B] are those of the end node's
 * chain).  Chain row i of node v is W_i h[v] + b_i (Eq. 3) on v's residual entering layer
 * layers[i-1], stands for position pos[v] + i and sees what v sees, rows 1..i-1 of its own chain
 * and itself (Section 3.3).  layers as in firp_step_layers.  Needs n_seq * T * (1 + k) <= max_rows
 * and context + T (1 + k) <= max_ctx; prefill is firp_prefill / firp_prefill_layers (only the last
 * prompt row needs a chain).  firp_kv_commit follows as after firp_step.
 */
int firp_step_chains(firp_ctx *ctx, int32_t n_seq, const int32_t *seq_ids, const int32_t *d_tree_tokens,
                     const int32_t *tree_parents, int32_t T, int32_t k, const int32_t *layers,
                     const firp_step_out *out, void *stream);

/*
 * The step of firp_step_layers with a tree of its own for every sequence (Section 3.4 builds the tree from
 * each sequence's own candidates; sequences at different points of their generation need not share a shape).
 *   tree_parents  HOST [n_seq][T]: row s holds the parents of sequence s's tree in its first tree_sizes[s] entries
 *   tree_sizes    HOST [n_seq]: 1 <= tree_sizes[s] <= T nodes
 * Every sequence still occupies T + k rows: rows tree_sizes[s] .. T-1 are padding (their tokens are ignored, they
 * can neither be accepted nor take a candidate; what the outputs hold for them is unspecified), the pseudo rows
 * stay at rows T .. T+k-1.  Each tree is validated like the template of firp_step; the next tree of a sequence is
 * built on its own shape.  Needs k > 0 unless every size equals T.
 */
int firp_step_trees(firp_ctx *ctx, int32_t n_seq, const int32_t *seq_ids, const int32_t *d_tree_tokens,
                    const int32_t *tree_parents, const int32_t *tree_sizes, int32_t T, int32_t k,
                    const int32_t *layers, const firp_step_out *out, void *stream);

/*
 * Visibility among the pseudo rows (Section 4.3, ablation).  masked = 0 (default, the "No masked"
 * setting the paper adopts): chain row i sees rows 1..i-1 of its chain.  masked != 0 ("Masked"): a
 * pseudo row sees no other pseudo row, only the prefix, its node with its ancestors, and itself;
 * positions are unchanged.  Applies to every later firp_prefill* / firp_step* call of the context.
 */
int firp_set_pseudo_masked(firp_ctx *ctx, int32_t masked);

/*
 * Non-contiguous KV cache (the paper's loop, Section 3.4, only needs the accepted prefix to be addressable; how
 * it is stored is the serving system's business).  page_table: HOST [max_batch][max_ctx / 64]; entry
 * [slot][p] is the physical page (0 .. max_batch * max_ctx / 64 - 1, each used once) that holds positions
 * 64 p .. 64 p + 63 of that slot; inside a (layer, K|V) plane of the cache a page is 64 consecutive rows.
 * The table is checked and copied into the workspace (synchronises `stream`); NULL goes back to contiguous rows.
 * max_ctx must be a multiple of 64.  Cache contents are not moved: set the table before the slot is prefilled.
 */
int firp_set_kv_pages(firp_ctx *ctx, const int32_t *page_table, void *stream);

/*
 * What Eq. 3 reads (Section 3.3 writes W_i h^{t_i} + b_i and does not say whether h^{t_i} is taken before or
 * after the layer's normalisation).  on == 0 (default): the raw residual stream entering layer t_i.  on != 0: the
 * state the decoder layer itself reads, h~_i = W_i rmsnorm(h^{t_i}; g_attn[t_i]) + b_i.  Applies to every later
 * firp_prefill* / firp_step* call of the context.
 */
int firp_set_pred_prenorm(firp_ctx *ctx, int32_t on);

/*
 * Commit after a step: for each sequence move the cache rows of path[j] to slot n + j
 * (every layer, K and V) and advance n by path_len.  path (HOST [n_seq][max_depth+1]) and
 * path_len (HOST [n_seq]) give an explicit path (strictly increasing, path[0] = 0); NULL
 * for both commits the path the last firp_step found, read on the device.
 * After a device-side commit the host does not know how many tokens were accepted: it keeps
 * an upper bound of the committed length (+ max_depth + 1 per commit), which sizes the
 * attention launch and feeds the capacity check.  firp_context_len brings the bound back to
 * the exact value; a step whose bound would not fit max_ctx reads the exact length itself
 * (one stream synchronisation) before it refuses, so the bound never causes a spurious
 * FIRP_ERR_CAPACITY, but a loop that never calls firp_context_len pays that synchronisation
 * on every step once the bound has drifted past max_ctx.
 */
int firp_kv_commit(firp_ctx *ctx, int32_t n_seq, const int32_t *seq_ids, const int32_t *path,
                   const int32_t *path_len, void *stream);

/*
 * Precision of the activations that enter the five weight GEMMs (the paper runs its models in half precision,
 * Section 4 "Setup", and says nothing about the arithmetic of a step).  Every GEMM multiplies bf16 by bf16 into
 * fp32 on the tensor cores; an activation is split into 1, 2 or 3 bf16 planes (hi; hi + lo; hi + mid + lo =
 * 8, 16, 24 mantissa bits) whose products are summed.  Default: 2 everywhere; the step then tracks an fp32
 * reference to ~3e-3 in the logits over 32 layers (a third plane on the QKV projection changes nothing measurable
 * and costs 3 % of the step).  1 is the plain bf16 GEMM; it halves the tensor-core work and the activation
 * traffic, which matters for steps of more than ~80 rows, at the price of 0.07-0.09 logit error over 32 layers
 * when used on the O, gate/up or down projection (0.01-0.02 on the QKV projection or the lm-head alone).  Applies to the kernel-per-operation
 * mode; the persistent kernel keeps the defaults.
 */
int firp_set_activation_planes(firp_ctx *ctx, int32_t qkv, int32_t o, int32_t gate_up, int32_t down, int32_t lm_head);

/* The same for the attention's two contractions: planes of the rotated queries (Q K^T) and of the softmax
 * probabilities (P V); keys and values are the cache's bf16.  Default 2 and 2. */
int firp_set_attention_planes(firp_ctx *ctx, int32_t q_planes, int32_t p_planes);

/*
 * Which kernel computes the tree attention (Section 3.4) in the kernel-per-operation mode when head_dim is 128.
 * tensor_core = 1: tiles of 128 cached positions as the M dimension of tcgen05 MMAs (S^T = K Q^T, O^T = V^T P^T,
 * accumulators in tensor memory, K/V tiles by TMA, two warpgroups alternating over the tiles); 0: the warp-level
 * mma.sync kernel with 64-position tiles, which is also what head_dim 64 and the persistent kernel always use;
 * -1 (default): chosen per step -- the mma.sync kernel only for steps of more than 16 query columns (rows x heads
 * per kv head) and about 29 rows or more (7B shape) whose longest context spans fewer than three of the
 * tensor-core kernel's tiles (four when the columns need more than one block of 48, eight when several sequences
 * are stepped together), where its lower fixed cost wins.  Both compute the same masked softmax with (hi, lo) bf16 planes of Q
 * and P and fp32 accumulation; summation orders differ.  Other values: FIRP_ERR_BAD_ARG.
 */
int firp_set_attention_kernel(firp_ctx *ctx, int32_t tensor_core);

/*
 * How the decoder layers of a step are launched (Section 3.4 describes one forward pass per round; the
 * paper gives no kernel design).  on != 0: a step of at most 48 rows over all its sequences runs its
 * layers, Eq. 3 and the lm-head as ONE persistent kernel (6 launches per step instead of ~300) whose weight
 * stream never stops between operations; larger steps, and every step when on == 0 (the default: it
 * measured 2-3 % faster at the 7B shape), use one kernel per operation.  Both run the same
 * arithmetic; they may cut the cached positions into a different number of attention splits, so their
 * results agree to fp32 rounding, and each is identical from run to run.
 */
int firp_set_fused(firp_ctx *ctx, int32_t on);

/*
 * Bound of every wait inside the kernels (for a tile, for the other CTAs of the persistent kernel), in
 * microseconds; 0 restores the default of 2 s.  A wait that runs out sets a device status word and the
 * kernel runs to its end without waiting again; the next firp_context_len returns
 * FIRP_ERR_DEVICE_TIMEOUT (results since the last check are invalid) and clears the word.
 */
int firp_set_wait_limit_us(firp_ctx *ctx, int64_t usec);

/*
 * Exercise the time-out path without disturbing any computation (the paper has no counterpart): enqueues a
 * one-CTA kernel that waits, with the routine and the limit the product kernels use, on a barrier nobody
 * arrives on.  The wait runs out, the kernel sets the device status word and returns normally; the next
 * firp_context_len therefore returns FIRP_ERR_DEVICE_TIMEOUT once, after which the context works as before.
 * Set a short limit first (firp_set_wait_limit_us): with the default the kernel runs for 2 s.
 */
int firp_selftest_wait(firp_ctx *ctx, void *stream);

/* Committed context length of a slot.  Synchronises `stream` (it reads the device counter) and
 * also reads the device status word: FIRP_ERR_DEVICE_TIMEOUT if any kernel gave up a wait. */
int firp_context_len(firp_ctx *ctx, int32_t seq, int32_t *n, void *stream);

/* Set the committed length of a slot (0 = empty; a smaller value rewinds). */
int firp_set_context_len(firp_ctx *ctx, int32_t seq, int32_t n, void *stream);

/* Number of kernels the last firp_step / firp_prefill / firp_kv_commit call launched. */
int firp_last_launch_count(const firp_ctx *ctx);

/*
 * Per-kernel timing aid (measurement only; it changes no result).  While enabled, every kernel
 * launch of firp_step / firp_prefill / firp_kv_commit is bracketed by a pair of CUDA events on
 * the call's stream, grouped by kernel class (the steps of Section 3.2-3.4: tree bookkeeping,
 * embedding, residual + RMSNorm, Eq. 3 projection, the five weight-streaming GEMMs and their
 * finishers, tree attention, top-B, acceptance walk, KV compaction).  The events serialise launches that otherwise overlap, so a
 * profiled step is slower than an unprofiled one: use it for per-kernel durations, not for the
 * step latency.
 *   firp_profile_enable  on != 0 starts (and clears) the collection, 0 stops it.
 *   firp_profile_read    synchronises `stream`, then writes for each class c < n_classes the
 *                        number of bracketed launches and their summed duration in microseconds
 *                        (HOST arrays), and clears the collection.  Returns the number of classes.
 *   firp_kernel_class_name  static name of class c, NULL if c is out of range.
 */
int firp_profile_enable(firp_ctx *ctx, int32_t on);
int firp_profile_read(firp_ctx *ctx, void *stream, int32_t n_classes, int32_t *launches, float *usec);
const char *firp_kernel_class_name(int32_t c);

/*
 * Top-B of logits rows without any device allocation.  (This call has no counterpart in the paper;
 * it serves hosts that drive the decoder from places where cudaMalloc is off limits: inside a
 * latency-critical serving loop whose memory pool is fixed at start-up, or in a plug-in that is
 * handed buffers and a stream by its host application and owns no allocator of its own.)
 *
 * Computes, for each of `rows` rows of fp32 logits (DEVICE, [rows][vocab], row-major), the b best
 * entries ordered by (value descending, token id ascending) -- the same selection firp_step makes
 * for its rows -- and writes d_ids [rows][b] and d_vals [rows][b] (DEVICE, caller-owned).
 *
 * The intermediate candidates of the two-pass selection live in a 256 KiB array that is part of
 * the library image on every GPU that loads it; nothing is allocated or freed, by this call or by
 * anything it uses.  The array limits the problem size: rows * ceil(vocab / 2048) must not exceed
 * FIRP_TOPB_STATIC_MAX_SLOTS, otherwise FIRP_ERR_CAPACITY is returned (and a line on stderr says
 * which limit was hit); 1 <= b <= 8.
 *
 * The first call on a device looks up the array's device address (once per device, under a lock):
 * make that first call outside any stream capture.  All calls on a device share the one array and it
 * keeps whatever the previous call left; every entry a call reads it has written itself, so no clearing
 * is needed, but two calls whose kernels can overlap on the GPU (different streams, no ordering between
 * them) race on it and must be serialised by the caller.
 * Work is enqueued on `stream`; nothing synchronises.  Returns FIRP_OK or a negative firp_status.
 */
#define FIRP_TOPB_STATIC_MAX_SLOTS 4096
int firp_topb_static(const float *d_logits, int32_t rows, int32_t vocab, int32_t b, int32_t *d_ids, float *d_vals,
                     void *stream);

#ifdef __cplusplus
}
#endif
#endif /* FIRP_H_ */
