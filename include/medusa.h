/*
 * medusa.h -- C ABI of the B200-native Medusa tree-verification decode step (Medusa, arXiv 2401.10774).
 *
 * One decoding step = (1) Medusa heads propose tokens, (2) a static candidate tree of those tokens is run
 * through the backbone with tree-masked attention against the KV cache, (3) the longest accepted candidate
 * prefix is committed to the cache (paper Sec. 2, Fig. 1).
 *
 * Conventions
 *   - Every function returns an int32 status: MEDUSA_OK (0) or a negative MEDUSA_ERR_* code;
 *     medusa_last_error(ctx) gives a human-readable reason.  Nothing throws across this boundary.
 *   - Pointers are DEVICE pointers owned by the caller unless the name ends in `_host`.  Device tensors
 *     must be 16-byte aligned and densely packed in the stated row-major layout.
 *   - Element type of weights/activations is the context's dtype (MEDUSA_F32: float, MEDUSA_BF16:
 *     bfloat16); logits, log-sum-exps and top-k values are always float; indices are int32.
 *   - All work is enqueued on the stream given to medusa_create and is asynchronous with respect to the
 *     host; integer results land in device memory.  Arguments are validated on the host before any launch.
 *     Conditions only the device can see (a full cache) are reported through medusa_device_status().
 *   - The context owns its workspace, the uploaded tree buffers and (after medusa_load_weights) the KV
 *     cache and decode state.  It never takes ownership of caller memory.
 *   - No CPU fallback exists: without a CUDA device medusa_create fails with MEDUSA_ERR_CUDA.
 */
#ifndef MEDUSA_B200_H
#define MEDUSA_B200_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct medusa_ctx medusa_ctx;

enum {
    MEDUSA_OK = 0,
    MEDUSA_ERR_INVALID_ARG = -1, /* null pointer, bad enum, misaligned tensor */
    MEDUSA_ERR_SHAPE = -2,       /* a size outside what the kernels support */
    MEDUSA_ERR_UNSUPPORTED = -3, /* valid request with no kernel for it */
    MEDUSA_ERR_CACHE_FULL = -4,  /* committing would exceed L_max (nothing is written) */
    MEDUSA_ERR_CUDA = -5,        /* a CUDA runtime call failed */
    MEDUSA_ERR_TIMEOUT = -6,     /* a bounded device-side wait gave up */
    MEDUSA_ERR_STATE = -7,       /* call order: weights/tree not loaded yet */
    MEDUSA_ERR_NONFINITE = -8,   /* checked build only: a stage produced a NaN or an infinity (device status word) */
    MEDUSA_ERR_BOUNDS = -9       /* checked build only: a stage produced an index outside its range (device status word) */
};

enum { MEDUSA_F32 = 0, MEDUSA_BF16 = 1 };
enum { MEDUSA_GREEDY = 0, MEDUSA_TYPICAL = 1, MEDUSA_REJECTION = 2 };

/* Llama-style decoder shape (paper App. G names the operators: QKV/O linears, QK^T/PV, up/gate/down). */
typedef struct {
    int32_t n_layers, d, n_heads, head_dim, ffn, vocab;
    int32_t n_medusa; /* K heads (paper Sec. 2.1.1) */
    int32_t dtype;    /* MEDUSA_F32 | MEDUSA_BF16 */
    int32_t L_max;    /* KV-cache capacity in positions */
    int32_t n_kv_heads; /* key/value heads; 0 = n_heads.  Fewer (a divisor of n_heads) is grouped-query attention:
                         * query head h reads key/value head h / (n_heads / n_kv_heads), wk and wv have
                         * n_kv_heads*head_dim rows, and every K/V tensor below has n_kv_heads in place of H */
    float rms_eps, rope_theta;
    int32_t max_tree_nodes; /* largest tree (nodes incl. root) the context must hold; 0 = 64.  Up to 256 (paper Sec. 3.3.1 /
                             * Fig. 4 studies trees of that size): buffers are sized for ceil(max/64) tiles of 64 token
                             * rows, projections and attention then run tile by tile */
    int32_t max_batch;      /* sequences the context holds (batch > 1: paper Sec. 4 leaves batching to the serving layer; App. G
                             * studies the operators at batch 16); 0 = 1, at most 4.  Every sequence has its own KV cache,
                             * cache length, root token and last hidden state */
} medusa_model_desc;

/* Static tree buffers (paper Sec. 2.1.2, Fig. 2).  Host arrays owned by the caller:
 * pos/tree_idx/parent hold >= n_paths+1 entries, mask >= (n_paths+1)*ceil((n_paths+1)/64), retrieve >=
 * (n_paths+1)*(max_depth+1). */
typedef struct {
    int32_t T, P, depth, topk; /* out: nodes incl. root, leaves, deepest level, max rank+1 */
    uint64_t *mask;            /* [T][W], W = ceil(T/64) words per node: bit j of row i (word j/64, bit j%64) says node j is
                                * i or an ancestor of i.  Trees of up to 64 nodes: one word per node */
    int32_t *pos;              /* [T]  depth of the node = rotary position offset from the cache length */
    int32_t *tree_idx;         /* [T]  index into the candidate pool [root, head1 top-k, head2 top-k, ...] */
    int32_t *parent;           /* [T]  parent node, -1 for the root */
    int32_t *retrieve;         /* [P][depth+1] root-to-leaf node indices, -1 padded */
} medusa_tree_buffers;

/* Acceptance rule (paper Sec. 2.3.1).  temperature <= 0 or mode GREEDY: accept a child iff it is the
 * argmax of its parent's logits.  TYPICAL: iff p > min(eps, delta*exp(-H(p))), p = softmax(logits/temperature).
 * REJECTION (paper Sec. 1 and Sec. 2.3.1, first paragraph: the rejection sampling of speculative decoding, which keeps
 * the original model's distribution; the paper gives no algorithm for the tree, this is the reading taken): the tree's
 * candidates are deterministic drafts (point-mass proposals).  Starting at the root, the children of the current node
 * are tried in node order: child c with token x is accepted iff uniform[c] < p(x) / (1 - R), R = the mass of the
 * siblings rejected before it at this node; an accepted child becomes the current node; when all children are
 * rejected (or the node is a leaf) the next token is the Gumbel-max sample of the node's distribution without the
 * rejected tokens.  Needs temperature > 0 and a noise row of V + T floats: gumbel[V] followed by uniform[T] in [0, 1)
 * (eps and delta are ignored).  Decisions are taken in double precision. */
typedef struct {
    int32_t mode;
    float temperature, eps, delta;
} medusa_accept_params;

/* Device pointers to the model weights, all matrices [out][in] in the context's dtype.
 * layers_host: HOST array of n_layers*9 device pointers in the order
 * attn_norm[d], wq[HD][d], wk[HD][d], wv[HD][d], wo[d][HD], ffn_norm[d], w_gate[F][d], w_up[F][d], w_down[d][F]. */
typedef struct {
    const void *embed;      /* [V][d] */
    const void *final_norm; /* [d] */
    const void *lm_head;    /* [V][d] */
    const void *const *layers_host;
    const void *medusa_w1; /* [K][d][d]  (paper: W1^(k)) */
    const void *medusa_w2; /* [K][V][d]  (paper: W2^(k), stored vocabulary-major) */
} medusa_weights;

/* Names for medusa_workspace_ptr (read-only views of context-owned device buffers, for inspection). */
enum {
    MEDUSA_WS_LOGITS = 0,   /* float [T][V]   backbone logits of the last tree pass */
    MEDUSA_WS_HIDDEN = 1,   /* float [T][d]   final-norm output of the last tree pass */
    MEDUSA_WS_TREE_K = 2,   /* dtype [N_L][R][Hkv][D] rotated keys of the last tree pass (T rows used per layer); R = the
                             * context's token rows: 64, or 64*ceil(max_tree_nodes/64) -- also the row count of LOGITS,
                             * HIDDEN and the TAP buffers */
    MEDUSA_WS_TREE_V = 3,   /* dtype [N_L][R][Hkv][D] */
    MEDUSA_WS_K_CACHE = 4,  /* dtype [N_L][Hkv][L_max][D] */
    MEDUSA_WS_V_CACHE = 5,  /* dtype [N_L][Hkv][L_max][D] */
    MEDUSA_WS_HEAD_LOGITS = 6, /* float [K][V]  Medusa-head logits of the last step */
    MEDUSA_WS_TOPK_IDX = 7, /* int32 [K][topk] */
    MEDUSA_WS_TREE_TOK = 8, /* int32 [T] */
    MEDUSA_WS_ACC_NODES = 9, /* int32 [depth+1] */
    MEDUSA_WS_STATE = 10,   /* int32 [8]: cache_len, root, best, accept_len, next_root, n_emitted, status, steps */
    MEDUSA_WS_H_LAST = 11,  /* float [d] */
    MEDUSA_WS_EMITTED = 12, /* int32 [depth+1] */
    /* copies taken at the layer chosen with MEDUSA_OPT_LAYER_TAP during the last backbone pass (64 rows, T used): */
    MEDUSA_WS_TAP_X_IN = 13,   /* float [64][d]  residual stream entering the layer */
    MEDUSA_WS_TAP_X_OUT = 14,  /* float [64][d]  residual stream leaving it */
    MEDUSA_WS_TAP_ATT = 15,    /* dtype [P][64][H*D] the layer's attention output as the output projection reads it
                                * (bf16 model: P = 2 planes whose sum is the value; f32 model: P = 1) */
    MEDUSA_WS_TAP_XN_OUT = 16  /* dtype [P][64][d] RMSNorm of X_OUT with the gain of the norm that follows the layer
                                * (the next layer's attention norm, or the final norm after the last layer) */
};

/* Context options for medusa_set_option. */
enum {
    MEDUSA_OPT_STEP_GRAPHS = 0,      /* 1 (default): medusa_decode_step may capture and replay whole-step CUDA graphs; 0: never */
    MEDUSA_OPT_ATTENTION_KERNEL = 1, /* bf16 / head_dim 128 tree attention: 1 mma.sync, 2 tcgen05, 0 (default) automatic: the
                                      * tcgen05 kernel for trees of up to 64 nodes from 2048 cached keys on in
                                      * medusa_tree_attention (by the length hint) and from 1536 on inside a pass or step (by
                                      * the host's lower bound of the cache length: exact after prefill, +1 per step) */
    MEDUSA_OPT_ATTENTION_LENGTH_HINT = 2, /* host-side upper bound of *cache_len for medusa_tree_attention (kernel choice and
                                           * grid size follow it; a longer cache is still processed completely); < 0: L_max */
    MEDUSA_OPT_LAYER_TAP = 3,        /* layer whose input / attention output / output the next passes copy to the TAP
                                      * buffers (parity checks layer by layer); -1 (default) off */
    MEDUSA_OPT_SPIN_LIMIT = 4,       /* polls after which a bounded device-side wait gives up with MEDUSA_ERR_TIMEOUT;
                                      * 0 = the kernels' default (about 4 million) */
    MEDUSA_OPT_WITHHOLD_LOAD = 5,    /* failure-path test hook, one shot: 1 = in the next tensor-core GEMM launch, 2 = in the
                                      * next tcgen05 attention launch, one CTA's producer issues no load at all, so that its
                                      * consumers' bounded waits expire with nothing in flight; the launch returns, its output
                                      * is unusable and the device status becomes MEDUSA_ERR_TIMEOUT */
    MEDUSA_OPT_ACTIVATION_PLANES = 6, /* bf16 model: planes of every activation the projections read.  2 (default): a value
                                       * y is held as hi = bf16(y) and lo = bf16(y - hi) and a projection is W hi + W lo
                                       * (accurate to ~2^-17); 1: hi only -- half the tensor-core work and up to 256 token
                                       * rows per weight stream (large trees, batches), at bf16 accuracy of the inputs */
    MEDUSA_OPT_PACK_WEIGHTS = 7        /* bf16 model, read by medusa_load_weights: 1 (default) = the context keeps its own
                                       * copy of the backbone matrices and the LM head, re-laid tile by tile so that the
                                       * 16 KiB a CTA requests per k block are consecutive bytes (costs the size of those
                                       * weights in device memory a second time; same arithmetic, bit-identical results,
                                       * the projections about 3.5 % faster); 0 = the projections stream the caller's
                                       * row-major tensors and nothing is copied */
};

/* ---- lifetime ------------------------------------------------------------------------------------ */

/* Creates a context on CUDA device `device`; `stream` is a cudaStream_t.  With NULL the context creates a
 * blocking stream of its own (the legacy default stream cannot be captured into the whole-step graphs); like
 * every blocking stream it orders itself with work on the legacy default stream in both directions.
 * Shapes supported: head_dim in {64,128}, T <= max_tree_nodes <= 256, max_batch <= 4, d and ffn multiples of 8 (bf16) /
 * 4 (f32). */
int32_t medusa_create(medusa_ctx **out, const medusa_model_desc *desc, int32_t device, void *stream);
int32_t medusa_destroy(medusa_ctx *ctx);
const char *medusa_last_error(const medusa_ctx *ctx);
/* Synchronises the stream and returns the device status word (MEDUSA_OK, MEDUSA_ERR_CACHE_FULL, ...);
 * the word is sticky until medusa_reset. */
int32_t medusa_device_status(medusa_ctx *ctx);
const void *medusa_workspace_ptr(medusa_ctx *ctx, int32_t which);
/* Synchronises the stream, then copies `bytes` bytes from offset `offset_bytes` of a workspace buffer to
 * dst_host. */
int32_t medusa_read_workspace(medusa_ctx *ctx, int32_t which, int64_t offset_bytes, void *dst_host, int64_t bytes);

/* Sets one of the MEDUSA_OPT_* options.  Options that captured step graphs depend on synchronise the stream and drop
 * those graphs.  Errors: INVALID_ARG (unknown option, value out of range). */
int32_t medusa_set_option(medusa_ctx *ctx, int32_t option, int64_t value);

/* Kernel-launch accounting and optional per-category device timing (CUDA events around every launch; adds
 * event overhead, so leave it off when timing whole steps).  Categories: 0 GEMM, 1 tree attention,
 * 2 Medusa-head GEMV, 3 element-wise (embed, RMSNorm, RoPE, SwiGLU), 4 top-k + candidate expansion,
 * 5 acceptance, 6 KV commit.  medusa_get_profile synchronises the stream and writes accumulated
 * milliseconds and launch counts (host arrays of MEDUSA_PROF_CATEGORIES entries, nullable); reset != 0 clears them. */
#define MEDUSA_PROF_CATEGORIES 8
int32_t medusa_set_profiling(medusa_ctx *ctx, int32_t on);
/* Whole-step graphs of medusa_decode_step: graphs currently cached and steps replayed from a graph since the
 * context was created (host int, nullable). */
int32_t medusa_step_graph_info(const medusa_ctx *ctx, int32_t *n_graphs_host, int64_t *n_replays_host);
int32_t medusa_get_profile(medusa_ctx *ctx, double *ms_host, int64_t *launches_host, int32_t reset);

/* Measurement aid (the paper has no counterpart): enqueues on `stream` (a cudaStream_t on the calling thread's current
 * device) a kernel that reads the first `bytes` bytes of device buffer `buf` (16-byte aligned) once with 16-byte
 * streaming loads and writes at most `sink_floats` floats to device buffer `sink`.  Timed with CUDA events over a buffer
 * much larger than the L2 it gives the read-only DRAM bandwidth, the ceiling for kernels that read far more than
 * they write.  Errors: INVALID_ARG, CUDA. */
int32_t medusa_stream_read(const void *buf, int64_t bytes, float *sink, int32_t sink_floats, void *stream);

/* ---- a0: static tree (paper Sec. 2.1.2 Fig. 2; Sec. 2.3.3 for the sparse tree) -------------------- */

/* Greedy node adding of Sec. 2.3.3 with surrogate accuracies 1/(rank+1): writes the n_nodes-1 rank tuples
 * (row-major [n_nodes-1][depth], -1 padded) of the best tree cut from the Cartesian tree per_depth_topk.
 * Host-only; returns the number of paths or a negative error. */
int32_t medusa_default_tree_paths(const int32_t *per_depth_topk_host, int32_t depth, int32_t n_nodes,
                                  int32_t *paths_host_out);

/* Sparse-tree construction from measured accuracies (Sec. 2.3.3).  acc_host: [depth][topk] row-major doubles,
 * acc[k][i] = estimated probability that the rank-i prediction of head k+1 is correct, each in [0, 1] (the
 * caller measures them on calibration data; rows need not be sorted).  Treating the heads as independent, a
 * node (i_1..i_k) has accuracy prod_j acc[j][i_j] (formed root to leaf in double); starting from the root, the
 * connected node of highest accuracy is added n_nodes-1 times (ties: the smaller tuple, a prefix before its
 * extensions), which maximises the expected number of accepted tokens for that node budget.
 * paths_host_out: [n_nodes-1][depth] rank tuples in the order added, -1 padded (feed to
 * medusa_build_tree_buffers).  expected_len_host_out (nullable): the sum of the chosen nodes' accuracies, i.e.
 * the expected number of accepted speculated tokens per step under the independence assumption.
 * Host-only, allocates only host memory.  Returns the number of paths, or INVALID_ARG (null, sizes < 1, depth > 8,
 * an accuracy outside [0, 1] or NaN) / SHAPE (n_nodes > 256 or more nodes asked for than the Cartesian tree has). */
int32_t medusa_tree_paths_from_accuracies(const double *acc_host, int32_t depth, int32_t topk, int32_t n_nodes,
                                          int32_t *paths_host_out, double *expected_len_host_out);

/* paths_host: [n_paths][max_depth] rank tuples (0-based rank of head j's prediction at depth j), -1 padded,
 * distinct and prefix-closed; T = n_paths+1 <= 256 (and <= the context's max_tree_nodes, 64 by default).  Fills out_host (node 0 = root, others sorted by
 * (depth, tuple)) and, if ctx != NULL, uploads a device copy that the other calls use.
 * Errors: INVALID_ARG (null), SHAPE (T > 256 or > the context's capacity, depth > 8, depth > n_medusa), INVALID_ARG (not prefix-closed,
 * duplicate, hole in padding). */
int32_t medusa_build_tree_buffers(medusa_ctx *ctx, const int32_t *paths_host, int32_t n_paths, int32_t max_depth,
                                  medusa_tree_buffers *out_host);

/* ---- a1-a4: Medusa heads, top-k, candidate expansion (paper Sec. 2.1.1 head definition; Sec. 2.1.2) ---- */

/* For k = 1..K: x_k = h + SiLU(W1_k h), z_k = W2_k x_k; topk_idx[k] = indices of the `topk` largest z_k
 * ordered by (value desc, index asc); tree_tok[i] = pool[tree_idx[i]] with pool = [root, topk_idx...].
 * h: [d]; W1: [K][d][d]; W2: [K][V][d]; root_token: device int32*; topk_idx: [K][topk] int32;
 * topk_val (nullable): [K][topk] float; logits_dump (nullable): [K][V] float; tree_tok: [T] int32.
 * Needs a tree uploaded by medusa_build_tree_buffers (ERR_STATE otherwise). */
int32_t medusa_heads(medusa_ctx *ctx, const void *h, const void *W1, const void *W2, const int32_t *root_token,
                     int32_t *topk_idx, float *topk_val, float *logits_dump, int32_t *tree_tok);

/* ---- a6: tree attention (paper Sec. 2.1.2 Fig. 2; App. G Table 5 "parallel decoding" QK^T, PV) --------- */

/* q: [T][H][D]; k_new, v_new: [T][Hkv][D]; k_cache, v_cache: [Hkv][L_max][D] of ONE layer, keys stored already
 * rotated (Hkv = the context's key/value heads: H unless n_kv_heads says otherwise);
 * cache_len: device int32* (L, 0 <= L <= L_max).  Query i of head h attends to cache positions 0..L-1 and
 * to the tree nodes j with bit j of mask[i] set; scores q.k/sqrt(D), softmax in float.
 * apply_rope != 0: q[i] and k_new[i] are first rotated at position L + pos[i] (element e pairs with e+D/2,
 * angle (L+pos)*theta^(-2e/D)); the rotated k_new is used for the scores but k_new itself is not modified.
 * out: [T][H][D]; lse (nullable): [T][H] float log-sum-exp of the scaled scores. */
int32_t medusa_tree_attention(medusa_ctx *ctx, const void *q, const void *k_new, const void *v_new,
                              const void *k_cache, const void *v_cache, const int32_t *cache_len,
                              int32_t apply_rope, void *out, float *lse);

/* Tree attention without a context and without any allocation.  (The paper has no counterpart for this
 * entry point: it exists for callers of this library, not for the method.)
 *
 * Who needs it: callers that must not allocate device memory at the time of the call -- a runtime that has
 * given its whole memory budget to its own pool, code on a path where cudaMalloc's implicit device
 * synchronisation is unacceptable, or a caller that has no medusa_ctx at all.  The split-KV partial
 * results that medusa_tree_attention keeps in its context workspace live here in a fixed array inside the
 * library image (about 8.1 MiB, held by every GPU that loads the library until the process exits).
 *
 * Same operation as medusa_tree_attention with apply_rope = 0, bf16, head_dim 128 only:
 * q, k_new, v_new: [T][H][128] (already rotated); k_cache, v_cache: [H][L_max][128]; cache_len: device int32*;
 * mask: device uint64 [T] (bit j of mask[i]: tree node j visible to query i); out: [T][H][128] bf16;
 * lse (nullable): float [T][H]; L_hint: host-side upper bound of *cache_len used to size the grid
 * (negative or > L_max: L_max is used); stream: cudaStream_t.  Work is enqueued on `stream`, nothing is
 * synchronised.  The device used is the calling thread's current device.
 * Limits: 1 <= T <= 64, H <= 64 (the fixed array serves at most 64 heads); anything larger returns
 * MEDUSA_ERR_SHAPE and prints the reason to stderr.  Other errors: MEDUSA_ERR_INVALID_ARG (null or
 * misaligned tensor), MEDUSA_ERR_CUDA.
 * The first call on each device resolves the array's device address and raises the kernel's shared-memory
 * limit; make that first call outside any stream capture.  It calls no cudaMalloc/cudaFree.
 * All calls on a device share the one array and it keeps the previous call's contents: the entry point
 * clears the per-head arrival counters on `stream` before every launch, the partials are rewritten before
 * they are read.  Two calls whose kernels overlap on the GPU (different streams) race on the array: keep
 * calls on one stream, or order them with events. */
int32_t medusa_tree_attention_static(const void *q, const void *k_new, const void *v_new, const void *k_cache,
                                     const void *v_cache, const int32_t *cache_len, const uint64_t *mask, int32_t T,
                                     int32_t H, int32_t L_max, int32_t L_hint, void *out, float *lse, void *stream);

/* ---- a7: acceptance (paper Sec. 2.3.1; Fig. 1 "longest accepted candidate prefix") ------------------ */

/* logits: float [T][V]; tree_tok: [T].  Walks every retrieve row, accepts the longest prefix whose nodes
 * pass the rule in `params` against their parent's logits; ties between rows go to the lowest row.
 * Outputs (device): best (row), accept_len (speculated tokens accepted, 0..depth), acc_nodes [depth+1]
 * (-1 beyond accept_len), next_root = argmax logits[last accepted node] (ties: lower index), or, if
 * gumbel != NULL and TYPICAL with temperature > 0, argmax_v fl(fl(logit_v * fl(1/temperature)) + gumbel[v]).
 * Typical-mode statistics are evaluated in double precision.  REJECTION: gumbel holds V + T floats (see
 * medusa_accept_params), best = the lowest retrieve row that starts with the accepted path; INVALID_ARG without a
 * noise row or with temperature <= 0. */
int32_t medusa_evaluate_posterior(medusa_ctx *ctx, const float *logits, const int32_t *tree_tok,
                                  const medusa_accept_params *params, const float *gumbel, int32_t *best,
                                  int32_t *accept_len, int32_t *next_root, int32_t *acc_nodes);

/* ---- a8: commit the accepted path (the paper only implies a KV cache; this defines the update) ------- */

/* n = min(1 + *accept_len, max_commit).  For every layer: cache[:, L+j, :] <- tree[acc_nodes[j]], j < n;
 * emitted[j] = tree_tok[acc_nodes[j]]; *n_emitted = n; h_last <- hidden[acc_nodes[n-1]]; *cache_len += n.
 * tree_k, tree_v: [N_L][R][Hkv][D] (R = the context's token rows: 64 unless max_tree_nodes asks for more); caches:
 * [N_L][Hkv][L_max][D];
 * hidden: float [T][d]; h_last: float [d].  If L + n > L_max nothing is written and the device status becomes
 * MEDUSA_ERR_CACHE_FULL. */
int32_t medusa_accept_and_update_kv(medusa_ctx *ctx, const void *tree_k, const void *tree_v, void *k_cache,
                                    void *v_cache, const int32_t *acc_nodes, const int32_t *accept_len,
                                    int32_t max_commit, int32_t *cache_len, const float *hidden, float *h_last,
                                    const int32_t *tree_tok, int32_t *emitted, int32_t *n_emitted);

/* ---- driver (paper Sec. 2: the three sub-steps of one decoding step) ------------------------------- */

/* Registers the weights (pointers must outlive the context) and allocates the KV cache and decode state. */
int32_t medusa_load_weights(medusa_ctx *ctx, const medusa_weights *w);
/* Clears the decode state of every sequence: cache_len = 0, status = OK. */
int32_t medusa_reset(medusa_ctx *ctx);
/* Runs the prompt (device int32 [n]) through the backbone in chains of up to 64 tokens (a chain tree is
 * ordinary causal attention), commits every position, and leaves root = argmax of the last logits and
 * h_last = the last hidden state.  ERR_CACHE_FULL if n exceeds the remaining capacity (checked on the host). */
int32_t medusa_prefill(medusa_ctx *ctx, const int32_t *prompt, int32_t n);
/* One backbone pass over `tokens` (device int32 [T], T = uploaded tree's size) with the uploaded tree's
 * mask/positions against the context's cache; results stay in the workspace (LOGITS, HIDDEN, TREE_K/V). */
int32_t medusa_tree_pass(medusa_ctx *ctx, const int32_t *tokens);
/* One full step: heads on h_last -> top-k -> tree tokens -> tree pass -> acceptance -> commit.
 * max_commit clamps the tokens emitted (generation budget).  gumbel (nullable): float [V] noise for this step
 * (REJECTION: required, float [V + T]).
 * emitted_host / n_emitted_host (nullable, pinned host memory recommended): async copies of the emitted
 * tokens [depth+1] and their count, valid after the stream is synchronised.
 * Nothing is synchronised: the step is enqueued on the context's stream.  The second consecutive step with the
 * same launch configuration (acceptance parameters, min(max_commit, depth + 1), presence of gumbel, the two host
 * pointers; the cache length is read on the device) is captured into a CUDA graph, and later steps with that
 * configuration replay it (up to 16 graphs per context; pageable host pointers, a stream that is itself being
 * captured, profiling and MEDUSA_OPT_STEP_GRAPHS = 0 keep the plain launches).
 * When max_commit cuts the accepted path short, the next step's root is the path's next (already accepted) token,
 * so repeated calls with a small max_commit continue the same token stream.  A replayed step reads its noise row
 * from a buffer of the context, into which gumbel is copied first. */
int32_t medusa_decode_step(medusa_ctx *ctx, const medusa_accept_params *params, const float *gumbel,
                           int32_t max_commit, int32_t *emitted_host, int32_t *n_emitted_host);
/* Batch > 1.  A context created with max_batch = B holds B independent sequences.  medusa_select_sequence chooses the
 * sequence that the single-sequence calls (medusa_prefill, medusa_decode_step, medusa_tree_pass, medusa_generate and the
 * per-sequence workspace views STATE, K_CACHE, V_CACHE, H_LAST, HEAD_LOGITS, TOPK_IDX, ACC_NODES, EMITTED) work on;
 * medusa_reset clears all sequences.  Errors: INVALID_ARG (b outside [0, B)). */
int32_t medusa_select_sequence(medusa_ctx *ctx, int32_t b);
/* One decode step of ALL B sequences in one backbone pass: sequence b's tree tokens are rows 64 b .. 64 b + T - 1 of the
 * pass (LOGITS, HIDDEN, TREE_K/V, TREE_TOK use the same rows), the projections stream the weights once for all sequences,
 * the attention runs per sequence against that sequence's cache and cache length, and heads, top-k, acceptance and
 * commit run per sequence exactly as in medusa_decode_step (same acceptance rule for all).  The uploaded tree must have
 * at most 64 nodes (SHAPE otherwise).  gumbel (nullable): float [B][V] device noise rows ([B][V + T] for REJECTION); emitted_host [B][depth+1] and
 * n_emitted_host [B] (nullable, pinned host memory recommended): async copies, valid after the stream is synchronised.
 * Every sequence must have been prefilled.  Like medusa_decode_step, the second consecutive batched step with the same
 * launch configuration is captured into a CUDA graph and replayed afterwards (the noise rows are staged through a
 * buffer of the context). */
int32_t medusa_decode_step_batch(medusa_ctx *ctx, const medusa_accept_params *params, const float *gumbel,
                                 int32_t max_commit, int32_t *emitted_host, int32_t *n_emitted_host);

/* Convenience loop with HOST buffers: prefill prompt_host[n_prompt], then decode steps until G tokens are
 * emitted (one stream synchronisation per step to read the emitted tokens).  gumbel_host (nullable):
 * [max steps = G][V] ([G][V + T] for REJECTION, where it is required).  Writes out_tokens_host[G]; emitted_per_step_host (nullable) [G]; *steps_host. */
int32_t medusa_generate(medusa_ctx *ctx, const int32_t *prompt_host, int32_t n_prompt, int32_t G,
                        const medusa_accept_params *params, const float *gumbel_host, int32_t *out_tokens_host,
                        int32_t *emitted_per_step_host, int32_t *steps_host);

/* 1 if this library was built with -DMEDUSA_DEBUG_CHECKS (the "checked" flavour), else 0.  The checked flavour launches,
 * after the stages of a step, kernels that test what the stage produced -- head logits and backbone logits finite
 * (MEDUSA_ERR_NONFINITE); tree tokens inside the vocabulary, accepted nodes inside the tree, the chosen row among the
 * retrieve rows, the next root inside the vocabulary, the cache length inside [0, L_max] (MEDUSA_ERR_BOUNDS) -- and
 * record the FIRST failure in the device status word (medusa_device_status).  Nothing traps, nothing is skipped, and
 * the results are those of the default library.  It stands in for a memory checker where none can be run. */
int32_t medusa_debug_checks_enabled(void);

/* ---- training of the heads with a frozen backbone (paper Sec. 2.2.1, Eq. 1) --------------------------- */

/* Forward and backward pass of the Medusa-1 objective over N positions:
 *   L = sum_k lambda_k * mean_n( -log p_n^(k)(labels[k][n]) ),  p^(k) = softmax(W2_k (h + SiLU(W1_k h)))  (Sec. 2.1.1),
 * the mean taken over the positions whose label is >= 0 (the paper sums over the positions of a sequence; the mean is
 * the reading taken so that the value does not depend on N), and its gradient with respect to W1_k and W2_k of the
 * registered weights (the backbone is frozen: `hidden` is a constant).
 * hidden: device [N][d] in the context's dtype, the backbone's last hidden states (the heads' input); labels: device
 * int32 [K][N], labels[k][n] = the token head k + 1 should predict at position n (the token k + 2 positions after the
 * one that produced hidden[n]), -1 where there is none; lambda_host: HOST float [K], NULL = 0.8^(k+1).
 * Outputs (device, overwritten): loss float [K + 1] (per-head mean cross-entropy, then L); grad_w1 float [K][d][d];
 * grad_w2 float [K][V][d] (same [out][in] layout as the weights).
 * bf16 contexts with heads only, d a multiple of 256 and V a multiple of 128 (SHAPE otherwise).  Arithmetic: the five
 * projections per head run on the tensor cores with bf16 operands and float accumulation -- the operand that takes the
 * token position of the kernel is a split bf16 pair (h1, dz) or exact bf16 (h), the streamed operand one bf16 plane
 * (weights as stored; dz^T, da^T and h1^T rounded) -- everything else in float; positions are processed in chunks of up
 * to 1024 and the gradients accumulated chunk by chunk in position order.  Allocates its workspace (about 0.8 GB at the
 * 7B shape) on the first call; enqueued on the context's stream, nothing is synchronised. */
int32_t medusa_heads_loss_and_grads(medusa_ctx *ctx, const void *hidden, const int32_t *labels, int32_t N,
                                    const float *lambda_host, float *loss, float *grad_w1, float *grad_w2);

#ifdef __cplusplus
}
#endif
#endif /* MEDUSA_B200_H */
