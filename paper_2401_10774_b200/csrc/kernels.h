// Internal launch interface between the C-ABI layer (api.cu) and the kernel files.
// Every launcher enqueues on `s` and returns; errors surface through cudaGetLastError in the caller.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "gemm_tc.h"

namespace medusa {

enum GemmOut { GEMM_STORE_F32 = 1, GEMM_ADD_F32 = 2 };

// ---- simt_kernels.cu (any shape, both dtypes; the fp32 model runs entirely on these) ----
void launch_embed(int dtype, const int32_t *tok, const void *embed, float *x, int T, int d, int V, cudaStream_t s);
// GEMM inputs ("split activations"): in the bf16 model an activation y is stored as two bf16 planes,
// hi = bf16(y) and lo = bf16(y - hi); a product with bf16 weights is then W*hi + W*lo, accurate to ~2^-17.
// In the f32 model there is one float plane and lo is null.
// out/out_lo: [T][d] planes (out_lo nullable); out_f32 (nullable): the unrounded values
// Projections write partial results as float planes (PlaneDesc, gemm_tc.h); the kernels below that consume
// them add a column's planes in order before anything else.
// x (+= sum of planes, written back if pd.n_max > 0), then RMSNorm(x) -> out planes
void launch_add_rmsnorm(int dtype, float *x, const float *planes, const PlaneDesc &pd, const void *gain,
                        float eps, void *out, void *out_lo, float *out_f32, int T, int d, cudaStream_t s);
// Y[t][col0 + n] (float, row stride ldy) (+)= sum_k (X[t][k] + Xlo[t][k]) * W[n][k];  X planes [T][K], row stride ldx
void launch_gemm_simt(int dtype, const void *X, const void *Xlo, int ldx, const void *W, void *Y, int ldy, int col0,
                      int T, int N, int K, GemmOut mode, cudaStream_t s);
// cs[t][e] = (cos, sin) of (L + pos[t]) * theta^(-2e/D), e < D/2
void launch_rope_table(float2 *cs, const int32_t *cache_len, const int32_t *pos, int T, int D, float theta,
                       cudaStream_t s);
// qkv float [T][(H + 2*Hkv)*D] (GEMM accumulators, rounded once here) -> q rotated [T][H][D], tree_k rotated
// [T][Hkv][D], tree_v [T][Hkv][D].  q_lo (nullable, bf16 model): second plane of q, q = q + q_lo to ~2^-17.  pd_q / pd_kv: plane layout of the launch that produced the q columns / the k and v
// columns (the same launch when kv_col0 == 0, else the second launch's column 0 sits at row column kv_col0 = H*D).
void launch_rope_split(int dtype, const float *qkv, const PlaneDesc &pd_q, const PlaneDesc &pd_kv, int kv_col0, const float2 *cs,
                       void *q, void *q_lo, void *tree_k, void *tree_v, int T, int H, int Hkv, int D, cudaStream_t s);
// rotate q and k only (stand-alone attention operator with apply_rope): in [T][H][D] -> out [T][H][D]
void launch_rope_apply(int dtype, const void *in, const float2 *cs, void *out, int T, int H, int D, cudaStream_t s);
// gate_up float [T][2F] -> act[t][i] = SiLU(gate) * up, rounded once to the activation dtype
void launch_silu_mul(int dtype, const float *gate_up, const PlaneDesc &pd, void *act, void *act_lo, int T,
                     int F, cudaStream_t s);

// sums `bytes` bytes with 16-byte streaming loads (a pure DRAM read stream); sink: >= blocks floats
void launch_stream_read(const void *buf, long long bytes, float *sink, int blocks, cudaStream_t s);

// ---- attention.cu ----
// q,out: [T][H][D], k_new,v_new: [T][Hkv][D] (already rotated); caches [Hkv][L_max][D]; mask [T][mask_words] (bit j of
// row i: tree node j visible to query i; one word per 64 nodes); lse nullable [T][H];
// out_lo (nullable): second plane of the split output.  Hkv divides H: query head h reads key/value head h / (H / Hkv)
// (grouped-query attention; Hkv == H is ordinary multi-head attention).
void launch_tree_attention_simt(int dtype, const void *q, const void *k_new, const void *v_new, const void *k_cache,
                                const void *v_cache, const int32_t *cache_len, const uint64_t *mask, void *out,
                                void *out_lo, float *lse, int T, int H, int Hkv, int D, int L_max, cudaStream_t s,
                                int mask_words = 1);

// ---- attention_flash.cu (bf16, head_dim 128: tensor-core split-KV flash-decode kernel) ----
constexpr int FLASH_MAX_SPLITS = 32;
size_t tree_attention_flash_workspace_bytes(int H, int q_tiles = 1);  // q_tiles: tiles of 64 query rows (trees > 64 nodes)
// same contract as the kernel above; L_hint: host-side upper bound of *cache_len (the tcgen05 kernel sizes its grid
// with it; the mma.sync kernel picks its key ranges from *cache_len on the device);
// workspace: tree_attention_flash_workspace_bytes(H) bytes, zero-initialised once
// q_lo (nullable): second plane of q; with it the scores are q.k + q_lo.k.
// n_seq > 1: a batch -- q, k_new, v_new, out hold n_seq tiles of 64 rows (sequence b at rows 64 b..), every sequence with
// the same tree of T <= 64 nodes; sequence b's caches start cache_seq_stride elements after sequence b-1's and its cache
// length len_stride ints after sequence b-1's; the workspace must have been sized for n_seq query tiles.
cudaError_t launch_tree_attention_flash(const void *q, const void *k_new, const void *v_new, const void *k_cache,
                                        const void *v_cache, const int32_t *cache_len, const uint64_t *mask, void *out,
                                        void *out_lo, float *lse, void *workspace, int T, int H, int Hkv, int L_max,
                                        int L_hint, cudaStream_t s, const void *q_lo = nullptr, int mask_words = 1,
                                        int n_seq = 1, long long cache_seq_stride = 0, int len_stride = 0);
// The same operation and workspace on the tcgen05 tensor cores (attention_tc.cu): scores and P V accumulate in
// TMEM, softmax threads own one query row each.  status: device status word (MEDUSA_ERR_TIMEOUT on an expired wait).
cudaError_t launch_tree_attention_tc(const void *q, const void *k_new, const void *v_new, const void *k_cache,
                                     const void *v_cache, const int32_t *cache_len, const uint64_t *mask, void *out,
                                     void *out_lo, float *lse, void *workspace, int T, int H, int Hkv, int L_max,
                                     int L_hint, int32_t *status, cudaStream_t s, uint32_t spin_limit = 0, int withhold = 0,
                                     const void *q_lo = nullptr);

// ---- heads.cu ----
// x_k = h + SiLU(W1_k h) -> float [K][d];  h: float if h_is_f32 else the model dtype
void launch_heads_resblock(int dtype, const void *h, int h_is_f32, const void *W1, float *x, int K, int d, cudaStream_t s);
// the same two products for nb <= 4 sequences at once (batch > 1): every weight row is read once for all of them.
// h_all: float [nb][d] (h_stride floats apart); x_all: sequence b's float [K][d] block x_stride floats after b-1's;
// logits_all: sequence b's float [K][V] block z_stride floats after b-1's
cudaError_t launch_heads_resblock_batch(int dtype, const float *h_all, long long h_stride, const void *W1, float *x_all,
                                        long long x_stride, int K, int d, int nb, cudaStream_t s);
cudaError_t launch_heads_vocab_batch(int dtype, const float *x_all, long long x_stride, const void *W2, float *logits_all,
                                     long long z_stride, int K, int d, int V, int nb, cudaStream_t s);
// z_k = W2_k x_k  -> logits float [K][V]
void launch_heads_vocab(int dtype, const float *x, const void *W2, float *logits, int K, int d, int V, cudaStream_t s);
// per head: indices of the topk largest (value desc, index asc)
// scratch: topk_scratch_bytes(K) bytes of device memory (candidates of the first stage); without it, or for
// topk > 8, the one-block-per-row multi-pass kernel runs
size_t topk_scratch_bytes(int K);
void launch_topk(const float *logits, int K, int V, int topk, int32_t *idx, float *val, void *scratch, cudaStream_t s);
void launch_expand(const int32_t *root, const int32_t *topk_idx, const int32_t *tree_idx, int32_t *tree_tok, int T,
                   cudaStream_t s);

// ---- posterior.cu ----
constexpr int NODE_STAT_SLICES = 2;
constexpr int NODE_PART_BYTES = 32;
struct PosteriorArgs {
    const float *logits;      // [T][V]
    const int32_t *tree_tok;  // [T]
    const int32_t *retrieve;  // [P][depth+1]
    const int32_t *parent;    // [T]
    const float *gumbel;      // nullable [V]
    const float *uniform;     // [T] numbers in [0, 1): rejection sampling only
    int T, V, P, depth, mode;
    float temperature, eps, delta;
    // scratch
    int32_t *node_argmax;  // [T]
    double *node_lse;      // [T]
    double *node_ent;      // [T]
    void *node_part;       // [T][stat_slices] records of NODE_PART_BYTES bytes (typical acceptance only)
    int stat_slices;       // vocabulary slices per node in typical mode (NODE_STAT_SLICES)
    // outputs
    int32_t *best, *accept_len, *next_root, *acc_nodes;
};
void launch_evaluate_posterior(const PosteriorArgs &a, cudaStream_t s);

struct CommitArgs {
    const void *tree_k, *tree_v;  // [N_L][tree_rows][H][D]
    int tree_rows;                // row stride of the scratch per layer (the context's rows, 64 unless it holds larger trees)
    void *k_cache, *v_cache;      // [N_L][H][L_max][D]
    const int32_t *acc_nodes, *accept_len;
    int max_commit;
    int32_t *cache_len;
    const float *hidden;  // [T][d]
    float *h_last;        // [d]
    const int32_t *tree_tok;
    int32_t *emitted, *n_emitted;
    int32_t *status;            // device status word
    const int32_t *next_root;   // nullable: if set, *root_out = *next_root
    int32_t *root_out;          // nullable
    int n_layers, H, D, L_max, d, depth_plus1;
};
void launch_commit(int dtype, const CommitArgs &a, cudaStream_t s);
// chain commit used by prefill: acc_nodes = 0..T-1 is implied
void launch_iota(int32_t *p, int n, cudaStream_t s);
// out[0] = argmax of logits[row] (ties: lower index)
void launch_argmax_row(const float *logits, int V, int row, int32_t *out, cudaStream_t s);


// ---- training of the heads (paper Sec. 2.2.1, Eq. 1): the kernels around the projections, train_heads.cu
void launch_head_hidden_fwd(const float *A_planes, const PlaneDesc &pd, const void *H, float *A, void *h1_hi, void *h1_lo, int rows,
                            int d, cudaStream_t s);
void launch_head_hidden_bwd(const float *dH1_planes, const PlaneDesc &pd, const float *A, void *dA, int rows, int d, cudaStream_t s);
void launch_ce_grad(const float *Z, int V, const int32_t *labels, int rows, int rows_valid, const int32_t *n_valid, float lambda,
                    float *row_loss, void *dz_hi, void *dz_lo, cudaStream_t s);
void launch_loss_accumulate(const float *row_loss, int rows, const int32_t *n_valid, float lambda, float *loss_k, float *loss_total,
                            cudaStream_t s);
void launch_count_valid(const int32_t *labels, int K, int N, int32_t *n_valid, cudaStream_t s);
// out[c][r] = in[r][c] for a row-major [R][C] bf16 matrix
void launch_transpose_bf16(const void *in, int R, int Cc, long long ld_in, void *out, long long ld_out, cudaStream_t s);

}  // namespace medusa
