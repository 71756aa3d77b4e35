// C-ABI layer and host driver of the Medusa tree-verification step (declarations: include/medusa.h).
// Validates arguments on the host, owns the workspace / KV cache / decode state, and enqueues the kernels
// of one step on the context's stream.  No host round-trip happens inside a step: cache length, root token,
// accepted path and the last hidden state stay in device memory between kernels and between steps.
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <algorithm>
#include <string>
#include <vector>

#include "common.cuh"
#include "pdl.cuh"
#include "gemm_tc.h"
#include "kernels.h"
#include "tree_host.h"

using namespace medusa;

struct medusa_ctx {
    medusa_model_desc m{};
    int device = 0;
    int rows = TREE_ROWS;  // token rows the context's buffers hold: 64 * max(ceil(max_tree_nodes / 64), max_batch), at most MAX_T
    // Sequences (batch): every sequence has its own decode state, KV cache, last hidden state and per-step integer
    // outputs.  The members d_state, k_cache, v_cache, h_last, head_x, head_logits, topk_idx, acc_nodes, emitted,
    // gumbel_dev and L_upper below are VIEWS of the selected sequence `cur` into the *_all allocations
    // (medusa_select_sequence re-points them), so that every single-sequence call works on the selected sequence.
    int B = 1, cur = 0;
    int32_t *state_all = nullptr, *topk_idx_all = nullptr, *acc_nodes_all = nullptr, *emitted_all = nullptr;
    float *h_last_all = nullptr, *head_x_all = nullptr, *head_logits_all = nullptr, *gumbel_all = nullptr;
    char *k_cache_all = nullptr, *v_cache_all = nullptr;
    size_t cache_seq_bytes = 0;  // bytes of one sequence's K (or V) cache
    std::vector<int> L_upper_all, L_lower_all;
    int Hkv = 0;  // key/value heads: m.n_kv_heads, or m.n_heads when that is 0 (ordinary multi-head attention)
    cudaStream_t stream = nullptr;
    bool own_stream = false;
    mutable std::string err;
    size_t esz = 4;  // bytes per weight/activation element

    // static tree
    bool have_tree = false;
    TreeHost tree;
    uint64_t *d_mask = nullptr, *d_chain_mask = nullptr;
    int32_t *d_pos = nullptr, *d_tree_idx = nullptr, *d_parent = nullptr, *d_retrieve = nullptr, *d_chain_pos = nullptr;

    // weights
    bool have_weights = false;
    medusa_weights w{};
    std::vector<const void *> layers;

    // decode state + workspace (device)
    int32_t *d_state = nullptr;  // ST_WORDS ints
    float *x = nullptr;          // [64][d] residual stream, float
    // GEMM inputs are "split activations": [2][64][width] bf16 planes (hi, lo) in the bf16 model, one float
    // plane in the f32 model.  lo_off(width) gives the byte offset of the lo plane (0 = none).
    void *xn = nullptr, *att = nullptr, *act = nullptr, *hidden = nullptr;
    void *q = nullptr, *rot_k = nullptr;
    float *hidden_f32 = nullptr;  // final-norm output before it is split into planes
    float *h_last = nullptr, *head_x = nullptr;
    void *flash_ws = nullptr;  // split-KV partials of the flash attention kernels
    // bf16 / head dim 128 attention kernel: 0 = automatic (the tcgen05/TMEM kernel for the stand-alone operation from
    // ATTN_TC_MIN_L keys on, the mma.sync kernel otherwise), 1 = always mma.sync, 2 = always tcgen05
    // (MEDUSA_ATTENTION=mma_sync|tcgen05)
    int attn_mode = 0;
    int attn_len_hint = -1;  // host-side bound of the cache length for the stand-alone attention call (< 0: the capacity)
    // layer tap (MEDUSA_OPT_LAYER_TAP): copies of one layer's input, attention output and output, for parity checks
    int tap_layer = -1;
    float *tap_x_in = nullptr, *tap_x_out = nullptr;  // [64][d] residual stream before / after the layer
    void *tap_att = nullptr;                          // the layer's attention output as the o projection reads it
    void *tap_xn_out = nullptr;                       // normalised residual stream after the layer (next norm's gain)
    // test hooks for the bounded device-side waits (MEDUSA_OPT_SPIN_LIMIT, MEDUSA_OPT_WITHHOLD_LOAD)
    uint32_t spin_limit = 0;  // 0: the kernels' default
    int withhold = 0;         // one-shot: 1 = next tensor-core GEMM launch, 2 = next tcgen05 attention launch
    // host-side upper bound of the device-resident cache length (a hint for attention kernels that size their
    // grid on the host; grows by the most a commit can add, exact again after prefill / generate read the length)
    int L_upper = 0;
    // host-side LOWER bound of the cache length: exact after prefill / generate, and every step adds at least one token.
    // Which attention kernel a step uses is decided on it, so that the long-cache kernel is only chosen where the cache
    // really is long (the upper bound drifts away from the length when steps accept less than a full path).
    int L_lower = 0;
    size_t part_elems = 0;
    float *part = nullptr;  // k-split partial planes of the projection in flight: [planes][64][width]
    // tensor-core path (bf16 model): TMA descriptors of the activation planes and of every weight matrix
    bool use_tc = false;
    TensorMap map_xn, map_att, map_act, map_hidden, map_lm;
    std::vector<TensorMap> wmaps;  // per layer: wq, wk, wv, wo, w_gate, w_up, w_down
    // activation planes the projections read (MEDUSA_OPT_ACTIVATION_PLANES): 2 = hi + lo (default), 1 = hi only
    int act_planes = 2;
    // MEDUSA_OPT_PACK_WEIGHTS: the weight maps describe the context's own packed copies (packed_on: as loaded)
    bool pack_weights = true, packed_on = false;
    std::vector<void *> packed_copies;  // the context's packed matrices (also listed in allocs); replaced when weights are loaded anew
    // the lo plane of a split activation (null in the f32 model and when the projections read one plane only)
    void *lo(void *hi, size_t width) const { return m.dtype == MEDUSA_BF16 && act_planes == 2 ? (char *)hi + (size_t)rows * width * 2 : nullptr; }
    // the second plane of q, which the attention kernel reads whatever the projections do
    void *q_lo_plane(void *hi, size_t width) const { return m.dtype == MEDUSA_BF16 ? (char *)hi + (size_t)rows * width * 2 : nullptr; }
    float *logits = nullptr, *head_logits = nullptr;
    float2 *rope_cs = nullptr;
    void *tree_k = nullptr, *tree_v = nullptr, *k_cache = nullptr, *v_cache = nullptr;
    int32_t *topk_idx = nullptr, *tree_tok = nullptr, *acc_nodes = nullptr, *emitted = nullptr, *node_argmax = nullptr;
    int32_t *iota = nullptr, *tmp_i32 = nullptr, *prompt_dev = nullptr;
    double *node_lse = nullptr, *node_ent = nullptr;
    void *node_part = nullptr;  // per-slice records of the typical-acceptance statistics
    float *gumbel_dev = nullptr;
    void *topk_scratch = nullptr;  // first-stage candidates of the two-stage top-k
    int32_t *pinned = nullptr;  // host: [0..63] emitted, [64] n_emitted
    std::vector<void *> allocs;

    // launch accounting (always) and per-category event timing (opt-in, medusa_set_profiling)
    int64_t launches[MEDUSA_PROF_CATEGORIES] = {};
    bool prof = false;
    unsigned skip_mask = 0;
    struct Span { int cat; cudaEvent_t a, b; };
    std::vector<Span> spans;
    std::vector<cudaEvent_t> free_events;
    double prof_ms[MEDUSA_PROF_CATEGORIES] = {};

    // Whole-step CUDA graphs (medusa_decode_step).  Everything a step launches depends on the host only through
    // the values in StepKey (the cache length is read on the device); the second consecutive step with the same key is captured from the stream into an
    // executable graph, and later steps with that key replay it.  MEDUSA_OPT_STEP_GRAPHS = 0 turns this off.
    struct StepKey {
        int32_t max_commit, has_gumbel, seq;
        int32_t long_cache;  // whether the step's attention launches are the long-cache kernel's (follows L_lower)
        medusa_accept_params p;
        int32_t *emitted_host, *n_emitted_host;
    };
    struct StepGraph {
        StepKey key;
        cudaGraphExec_t exec;
        int64_t launches[MEDUSA_PROF_CATEGORIES];  // what one replay adds to the launch accounting
        uint64_t used;
    };
    // Workspace of the heads' training pass (medusa_heads_loss_and_grads), allocated on its first call for chunks of up
    // to 1024 positions (R below is the chunk size of the call).  "planes" buffers are split activations [2][rows][width] (hi plane, lo plane).
    struct TrainWs {
        bool ready = false;
        void *Hp = nullptr, *HT = nullptr;      // hidden states [2][R][d] (hi used) and their transpose [2][d][R]
        void *H1p = nullptr, *H1T = nullptr;    // h1 = h + SiLU(W1 h) [2][R][d]; transpose of its hi plane [2][d][R]
        float *A = nullptr, *part = nullptr;    // W1 h [R][d]; partial planes of the two stream-K projections
        float *Z = nullptr;                     // logits [R][V]
        void *dZp = nullptr, *dZT = nullptr;    // gradient of the logits [2][R][V]; transpose of its hi plane [V][R]
        void *W2T = nullptr;                    // W2_k transposed [d][V]
        void *dA = nullptr, *dAT = nullptr;     // gradient of W1 h [R][d] and transposed [d][R]
        float *row_loss = nullptr;
        int32_t *n_valid = nullptr;
        size_t part_planes = 0;
        TensorMap mHp, mHT, mH1p, mH1T, mdZp, mdZT, mW2T, mdAT;
        std::vector<TensorMap> mW1, mW2;        // per head
        const void *w1_of = nullptr, *w2_of = nullptr;  // the weight pointers those per-head maps were encoded for
        int R = 0;                              // chunk size the chunk buffers' maps were encoded for
    } train;
    std::vector<StepGraph> step_graphs;
    StepKey last_key{};
    bool have_last_key = false;
    bool step_graphs_on = true;
    uint64_t step_clock = 0;
};

namespace {

int32_t fail(const medusa_ctx *c, int32_t code, const char *fmt, ...)
{
    if (c) {
        char buf[512];
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(buf, sizeof buf, fmt, ap);
        va_end(ap);
        c->err = buf;
    }
    return code;
}

#define MEDUSA_CUDA(c, call)                                                                              \
    do {                                                                                                  \
        cudaError_t e_ = (call);                                                                          \
        if (e_ != cudaSuccess)                                                                            \
            return fail((c), MEDUSA_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e_));            \
    } while (0)

#define MEDUSA_LAUNCH_CHECK(c)                                                                            \
    do {                                                                                                  \
        cudaError_t e_ = cudaGetLastError();                                                              \
        if (e_ != cudaSuccess)                                                                            \
            return fail((c), MEDUSA_ERR_CUDA, "kernel launch failed at %s:%d: %s", __FILE__, __LINE__,    \
                        cudaGetErrorString(e_));                                                          \
    } while (0)

template <typename T> int32_t dev_alloc(medusa_ctx *c, T **p, size_t count)
{
    void *v = nullptr;
    size_t bytes = count * sizeof(T);
    if (bytes == 0) bytes = 16;
    MEDUSA_CUDA(c, cudaMalloc(&v, bytes));
    MEDUSA_CUDA(c, cudaMemsetAsync(v, 0, bytes, c->stream));
    c->allocs.push_back(v);
    *p = (T *)v;
    return MEDUSA_OK;
}

int32_t dev_alloc_bytes(medusa_ctx *c, void **p, size_t bytes) { return dev_alloc<char>(c, (char **)p, bytes); }

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

__global__ void set_i32_kernel(int32_t *p, int32_t v) {
    pdl_enter(); *p = v; }

// ---- the checked flavour (-DMEDUSA_DEBUG_CHECKS): validation kernels launched after the stages of a step.  They only
// read what the stage produced and record the first failure in the device status word; nothing traps or is skipped.
#ifdef MEDUSA_DEBUG_CHECKS
__global__ void __launch_bounds__(256) debug_finite_kernel(const float *__restrict__ p, size_t n, int32_t *status)
{
    bool bad = false;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        bad |= !isfinite(p[i]);
    if (bad) atomicCAS(status, MEDUSA_OK, MEDUSA_ERR_NONFINITE);
}
__global__ void __launch_bounds__(256) debug_range_kernel(const int32_t *__restrict__ p, int n, int lo, int hi, int32_t *status)
{
    bool bad = false;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x)
        bad |= p[i] < lo || p[i] > hi;
    if (bad) atomicCAS(status, MEDUSA_OK, MEDUSA_ERR_BOUNDS);
}
void debug_finite(medusa_ctx *c, const float *p, size_t n)
{
    if (n) debug_finite_kernel<<<(unsigned)((n + 255) / 256 < 1184 ? (n + 255) / 256 : 1184), 256, 0, c->stream>>>(p, n, c->d_state + ST_STATUS);
}
void debug_range(medusa_ctx *c, const int32_t *p, int n, int lo, int hi)
{
    if (n > 0) debug_range_kernel<<<(n + 255) / 256, 256, 0, c->stream>>>(p, n, lo, hi, c->d_state + ST_STATUS);
}
#define DEBUG_FINITE(c, p, n) debug_finite(c, p, n)
#define DEBUG_RANGE(c, p, n, lo, hi) debug_range(c, p, n, lo, hi)
#else
#define DEBUG_FINITE(c, p, n) ((void)0)
#define DEBUG_RANGE(c, p, n, lo, hi) ((void)0)
#endif

constexpr int ATTN_TC_MIN_L = 2048;       // measured crossover of the two attention kernels at T = 64, 32 heads, stand-alone
constexpr int ATTN_TC_STEP_MIN_L = 1536;  // and inside a decode step

enum { PC_GEMM = 0, PC_ATTENTION = 1, PC_HEADS = 2, PC_ELEMWISE = 3, PC_TOPK = 4, PC_POSTERIOR = 5, PC_COMMIT = 6 };

struct ProfScope {
    medusa_ctx *c;
    medusa_ctx::Span sp{};
    bool on;
    static cudaEvent_t get(medusa_ctx *c)
    {
        cudaEvent_t e = nullptr;
        if (!c->free_events.empty()) { e = c->free_events.back(); c->free_events.pop_back(); }
        else cudaEventCreate(&e);
        return e;
    }
    ProfScope(medusa_ctx *c_, int cat, int n_kernels) : c(c_), on(c_->prof)
    {
        c->launches[cat] += n_kernels;
        if (on) {
            sp.cat = cat;
            sp.a = get(c);
            sp.b = get(c);
            cudaEventRecord(sp.a, c->stream);
        }
    }
    ~ProfScope()
    {
        if (on) {
            cudaEventRecord(sp.b, c->stream);
            c->spans.push_back(sp);
        }
    }
};
#ifdef MEDUSA_TIMING_AIDS
// Timing-aid builds only: `skip_mask` (MEDUSA_DEBUG_SKIP, a bit per category) drops launches, to read a kernel class's
// cost inside the running pipeline; results are meaningless while it is set.
#define PROF(c, cat, nk, stmt)                      \
    do {                                            \
        if (!((c)->skip_mask & (1u << (cat)))) {    \
            ProfScope ps_((c), (cat), (nk));        \
            stmt;                                   \
        }                                           \
    } while (0)
#else
#define PROF(c, cat, nk, stmt)               \
    do {                                     \
        ProfScope ps_((c), (cat), (nk));     \
        stmt;                                \
    } while (0)
#endif

#define TRY(expr)                          \
    do {                                   \
        int32_t rc_ = (expr);              \
        if (rc_ != MEDUSA_OK) return rc_;  \
    } while (0)

// Tree attention of one layer: tensor-core flash kernel for bf16 / head_dim 128, CUDA-core kernel otherwise.
int32_t attention(medusa_ctx *c, const void *q, const void *k_new, const void *v_new, const void *kc, const void *vc,
                  const int32_t *cache_len, const uint64_t *mask, void *out, void *out_lo, float *lse, int T, int L_hint,
                  bool in_step, int mask_words, const void *q_lo = nullptr)
{
    const medusa_model_desc &m = c->m;
    if (c->flash_ws) {
        cudaError_t e = cudaSuccess;
        // The tcgen05 kernel is the faster one from ATTN_TC_MIN_L cached keys on as a stand-alone operation, and from
        // ATTN_TC_STEP_MIN_L on inside a decode step (measured at 7B and 13B width: 0.4 % of the step at 1540 keys, 3.6 % at
        // 2140, 4.6 % at 3900; slower below).  Inside a step the choice follows the host's LOWER bound of the cache length.
        // (the tcgen05 kernel holds one tile of 64 query rows: larger trees always take the mma.sync kernel)
        if (T <= TREE_ROWS && (c->attn_mode == 2 || (c->attn_mode == 0 && (in_step ? c->L_lower >= ATTN_TC_STEP_MIN_L : L_hint >= ATTN_TC_MIN_L))))
        {
            const int wh = c->withhold == 2 ? 1 : 0;
            if (wh) c->withhold = 0;
            PROF(c, PC_ATTENTION, 1, e = launch_tree_attention_tc(q, k_new, v_new, kc, vc, cache_len, mask, out, out_lo, lse, c->flash_ws,
                                                                  T, m.n_heads, c->Hkv, m.L_max, L_hint, c->d_state + ST_STATUS, c->stream,
                                                                  c->spin_limit, wh, q_lo));
        }
        else
            PROF(c, PC_ATTENTION, 1, e = launch_tree_attention_flash(q, k_new, v_new, kc, vc, cache_len, mask, out, out_lo, lse,
                                                                     c->flash_ws, T, m.n_heads, c->Hkv, m.L_max, L_hint, c->stream, q_lo, mask_words));
        if (e != cudaSuccess) return fail(c, MEDUSA_ERR_CUDA, "flash attention launch failed: %s", cudaGetErrorString(e));
        return MEDUSA_OK;
    }
    PROF(c, PC_ATTENTION, 1, launch_tree_attention_simt(m.dtype, q, k_new, v_new, kc, vc, cache_len, mask, out, out_lo, lse, T,
                                                        m.n_heads, c->Hkv, m.head_dim, m.L_max, c->stream, mask_words));
    MEDUSA_LAUNCH_CHECK(c);
    return MEDUSA_OK;
}

// One projection launch: up to three weight matrices of `seg_cols` rows each (the first of seg0_cols rows, if that is
// given) share the input X (a split activation of width K).  Results land as partial planes
// P[p][t][first column of the matrix + n] described by *pd, the matrices side by side in a row.
// The bf16 model runs the tcgen05 kernel, everything else the CUDA-core kernel (one plane).
int32_t project(medusa_ctx *c, const void *X, const TensorMap *mapX, const void *const *W, const TensorMap *mapW, int n_seg,
                int seg_cols, int K, float *P, size_t plane_stride, int ldy, int T, int row0, bool whole_tiles,
                PlaneDesc *pd, int seg0_cols = 0)
{
    if (seg0_cols <= 0) seg0_cols = seg_cols;
    if (c->use_tc && (n_seg == 1 || (seg_cols % 128 == 0 && seg0_cols % 128 == 0))) {
        const TensorMap *maps[3] = {mapW, mapW + (n_seg > 1 ? 1 : 0), mapW + (n_seg > 2 ? 2 : 0)};
        // up to 64 rows: one launch of one token tile; more: launches of two token tiles (128 rows) each, so that the
        // weights are streamed once per 128 rows
        const int RT = gemm_tc_row_tiles(T, c->act_planes), rows_per_launch = RT * TREE_ROWS;
        *pd = gemm_tc_plan(n_seg, seg_cols, K, whole_tiles, (long long)plane_stride, seg0_cols, RT, c->act_planes);
        if (!whole_tiles && (size_t)pd->n_max * plane_stride > c->part_elems)
            return fail(c, MEDUSA_ERR_SHAPE, "projection needs %d partial planes, more than the workspace holds", pd->n_max);
        // every launch of the projection uses the same plan, so the consumer finds the same pieces in every row
        for (int r0 = (row0 / rows_per_launch) * rows_per_launch; r0 < T; r0 += rows_per_launch) {
            cudaError_t e = cudaSuccess;
            const int wh = c->withhold == 1 ? 1 : 0;
            if (wh) c->withhold = 0;
            const int Tt = T - r0 < rows_per_launch ? T - r0 : rows_per_launch, row0t = row0 > r0 ? row0 - r0 : 0;
            PROF(c, PC_GEMM, 1, e = launch_gemm_tc(mapX, maps, n_seg, seg_cols, K, *pd, P + (size_t)r0 * ldy, ldy, Tt, row0t,
                                                   c->d_state + ST_STATUS, c->stream, seg0_cols, c->spin_limit, wh, r0, c->rows + r0, RT, c->act_planes, false, 0, 0,
                                                   c->packed_on));
            if (e != cudaSuccess) return fail(c, MEDUSA_ERR_CUDA, "tensor-core GEMM launch failed: %s", cudaGetErrorString(e));
        }
        return MEDUSA_OK;
    }
    const char *Xr = (const char *)X + (size_t)row0 * K * c->esz;
    const char *Xlo = c->m.dtype == MEDUSA_BF16 ? (const char *)c->lo((void *)X, (size_t)K) + (size_t)row0 * K * c->esz : nullptr;
    for (int sgm = 0; sgm < n_seg; ++sgm)
        PROF(c, PC_GEMM, 1, launch_gemm_simt(c->m.dtype, Xr, Xlo, K, W[sgm], P + (size_t)row0 * ldy, ldy,
                                             sgm == 0 ? 0 : seg0_cols + (sgm - 1) * seg_cols, T - row0,
                                             sgm == 0 ? seg0_cols : seg_cols, K, GEMM_STORE_F32, c->stream));
    MEDUSA_LAUNCH_CHECK(c);
    *pd = PlaneDesc{};
    pd->n_max = 1;
    pd->stride = (long long)plane_stride;
    return MEDUSA_OK;
}

// One backbone pass over T token rows (paper App. G Table 5, "parallel decoding" column).
// logits are produced for rows [lm_row0, T).
// n_seq == 1: the T tokens of the selected sequence occupy rows 0..T-1.  n_seq > 1 (a batched step): sequence b's T_seq
// tree tokens occupy rows 64 b .. 64 b + T_seq - 1 of every buffer; the row-wise kernels and the projections run over
// all 64 n_seq rows at once (the weights are streamed once for all sequences), the rotary table and the attention run
// per sequence against that sequence's own cache and cache length.
int32_t tree_pass(medusa_ctx *c, const int32_t *tokens, int T_seq, const uint64_t *mask, const int32_t *pos, int lm_row0,
                  int mask_words, int n_seq = 1)
{
    const medusa_model_desc &m = c->m;
    const int d = m.d, H = m.n_heads, Hkv = c->Hkv, D = m.head_dim, HD = H * D, HkvD = Hkv * D, F = m.ffn, dt = m.dtype;
    const int qkv_ld = HD + 2 * HkvD;  // a row of the QKV projection: [q | k | v]
    cudaStream_t s = c->stream;
    const int T = n_seq > 1 ? n_seq * TREE_ROWS : T_seq;  // rows of the pass
    int32_t *cache_len = c->d_state + ST_CACHE_LEN;
    for (int b = 0; b < n_seq; ++b) {  // (checked flavour) the pass's tokens and every sequence's cache length
        DEBUG_RANGE(c, tokens + (size_t)b * TREE_ROWS, T_seq, 0, m.vocab - 1);
        DEBUG_RANGE(c, n_seq > 1 ? c->state_all + (size_t)b * ST_WORDS + ST_CACHE_LEN : cache_len, 1, 0, m.L_max);
    }
    PROF(c, PC_ELEMWISE, 1, launch_embed(dt, tokens, c->w.embed, c->x, T, d, m.vocab, s));
    if (n_seq > 1) {
        for (int b = 0; b < n_seq; ++b)
            PROF(c, PC_ELEMWISE, 1, launch_rope_table(c->rope_cs + (size_t)b * TREE_ROWS * (D / 2), c->state_all + (size_t)b * ST_WORDS + ST_CACHE_LEN,
                                                      pos, T_seq, D, m.rope_theta, s));
    } else {
        PROF(c, PC_ELEMWISE, 1, launch_rope_table(c->rope_cs, cache_len, pos, T, D, m.rope_theta, s));
    }
    MEDUSA_LAUNCH_CHECK(c);
    PlaneDesc pd_prev{};  // planes of the previous projection still to be added to the residual stream
    for (int l = 0; l < m.n_layers; ++l) {
        const void *const *w = c->layers.data() + (size_t)l * 9;
        const TensorMap *wm = c->use_tc ? c->wmaps.data() + (size_t)l * 7 : nullptr;
        char *tk = (char *)c->tree_k + (size_t)l * c->rows * HkvD * c->esz;
        char *tv = (char *)c->tree_v + (size_t)l * c->rows * HkvD * c->esz;
        const char *kc = (const char *)c->k_cache + (size_t)l * Hkv * m.L_max * D * c->esz;
        const char *vc = (const char *)c->v_cache + (size_t)l * Hkv * m.L_max * D * c->esz;
        PlaneDesc pd{};
        // x += down-projection of the previous layer;  xn = RMSNorm(x)
        PROF(c, PC_ELEMWISE, 1, launch_add_rmsnorm(dt, c->x, c->part, pd_prev, w[0], m.rms_eps, c->xn, c->lo(c->xn, d), nullptr, T,
                                                   d, s));
        if (c->tap_layer >= 0) {
            const size_t planes = dt == MEDUSA_BF16 ? 2 : 1;
            if (l == c->tap_layer)
                MEDUSA_CUDA(c, cudaMemcpyAsync(c->tap_x_in, c->x, (size_t)c->rows * d * sizeof(float), cudaMemcpyDeviceToDevice, s));
            if (l == c->tap_layer + 1) {
                MEDUSA_CUDA(c, cudaMemcpyAsync(c->tap_x_out, c->x, (size_t)c->rows * d * sizeof(float), cudaMemcpyDeviceToDevice, s));
                MEDUSA_CUDA(c, cudaMemcpyAsync(c->tap_xn_out, c->xn, planes * c->rows * d * c->esz, cudaMemcpyDeviceToDevice, s));
            }
        }
        const void *wqkv[3] = {w[1], w[2], w[3]};
        if (Hkv == H || !c->use_tc || (HD % 128 == 0 && HkvD % 128 == 0)) {
            // one launch for [q | k | v]; with grouped-query attention the k and v matrices are narrower than q
            TRY(project(c, c->xn, &c->map_xn, wqkv, wm, 3, HkvD, d, c->part, (size_t)c->rows * qkv_ld, qkv_ld, T, 0, false, &pd, HD));
            PROF(c, PC_ELEMWISE, 1, launch_rope_split(dt, c->part, pd, pd, 0, c->rope_cs, c->q, c->q_lo_plane(c->q, HD), tk, tv, T, H, Hkv, D, s));
        } else {
            // widths that are not multiples of the 128-row tile: q alone (any width), then k and v on the CUDA-core
            // kernel, into disjoint columns of the same rows
            PlaneDesc pd_kv{};
            TRY(project(c, c->xn, &c->map_xn, wqkv, wm, 1, HD, d, c->part, (size_t)c->rows * qkv_ld, qkv_ld, T, 0, false, &pd));
            TRY(project(c, c->xn, &c->map_xn, wqkv + 1, wm ? wm + 1 : nullptr, 2, HkvD, d, c->part + HD, (size_t)c->rows * qkv_ld,
                        qkv_ld, T, 0, false, &pd_kv));
            PROF(c, PC_ELEMWISE, 1, launch_rope_split(dt, c->part, pd, pd_kv, HD, c->rope_cs, c->q, c->q_lo_plane(c->q, HD), tk, tv, T, H, Hkv, D, s));
        }
        MEDUSA_LAUNCH_CHECK(c);
        if (n_seq > 1 && c->flash_ws && c->attn_mode != 2) {
            // all sequences in one launch of the flash kernel: grid z = sequence, each against its own cache and length
            cudaError_t e = cudaSuccess;
            const size_t lay = (size_t)l * Hkv * m.L_max * D * c->esz;
            PROF(c, PC_ATTENTION, 1, e = launch_tree_attention_flash(c->q, tk, tv, c->k_cache_all + lay, c->v_cache_all + lay,
                                                                     c->state_all + ST_CACHE_LEN, mask, c->att, c->lo(c->att, HD), nullptr,
                                                                     c->flash_ws, T_seq, H, Hkv, m.L_max, m.L_max, s, c->q_lo_plane(c->q, HD),
                                                                     mask_words, n_seq, (long long)(c->cache_seq_bytes / c->esz), ST_WORDS));
            if (e != cudaSuccess) return fail(c, MEDUSA_ERR_CUDA, "batched flash attention launch failed: %s", cudaGetErrorString(e));
        } else if (n_seq > 1) {
            // every sequence's 64-row tile against its own cache (launches follow one another on the stream and each
            // waits for its predecessor before it touches anything, so they can share the split-KV workspace)
            for (int b = 0; b < n_seq; ++b) {
                const size_t ro = (size_t)b * TREE_ROWS;  // first row of the sequence
                const size_t lay = (size_t)l * Hkv * m.L_max * D * c->esz;
                const char *q_lo = (const char *)c->q_lo_plane(c->q, HD);
                char *att_lo = (char *)c->lo(c->att, HD);
                TRY(attention(c, (const char *)c->q + ro * HD * c->esz, tk + ro * HkvD * c->esz, tv + ro * HkvD * c->esz,
                              c->k_cache_all + (size_t)b * c->cache_seq_bytes + lay, c->v_cache_all + (size_t)b * c->cache_seq_bytes + lay,
                              c->state_all + (size_t)b * ST_WORDS + ST_CACHE_LEN, mask, (char *)c->att + ro * HD * c->esz,
                              att_lo ? att_lo + ro * HD * c->esz : nullptr, nullptr, T_seq, c->L_upper_all[b], true, mask_words,
                              q_lo ? q_lo + ro * HD * c->esz : nullptr));
            }
        } else {
            TRY(attention(c, c->q, tk, tv, kc, vc, cache_len, mask, c->att, c->lo(c->att, HD), nullptr, T, c->L_upper, true,
                          mask_words, c->q_lo_plane(c->q, HD)));
        }
        if (l == c->tap_layer)
            MEDUSA_CUDA(c, cudaMemcpyAsync(c->tap_att, c->att, (dt == MEDUSA_BF16 ? 2 : 1) * (size_t)c->rows * HD * c->esz,
                                           cudaMemcpyDeviceToDevice, s));
        const void *wo[1] = {w[4]};
        TRY(project(c, c->att, &c->map_att, wo, wm ? wm + 3 : nullptr, 1, d, HD, c->part, (size_t)c->rows * d, d, T, 0, false, &pd));
        // x += attention output projection;  xn = RMSNorm(x)
        PROF(c, PC_ELEMWISE, 1, launch_add_rmsnorm(dt, c->x, c->part, pd, w[5], m.rms_eps, c->xn, c->lo(c->xn, d), nullptr, T, d, s));
        const void *wgu[2] = {w[6], w[7]};
        TRY(project(c, c->xn, &c->map_xn, wgu, wm ? wm + 4 : nullptr, 2, F, d, c->part, (size_t)c->rows * 2 * F, 2 * F, T, 0, false, &pd));
        PROF(c, PC_ELEMWISE, 1, launch_silu_mul(dt, c->part, pd, c->act, c->lo(c->act, F), T, F, s));
        MEDUSA_LAUNCH_CHECK(c);
        const void *wd[1] = {w[8]};
        TRY(project(c, c->act, &c->map_act, wd, wm ? wm + 6 : nullptr, 1, d, F, c->part, (size_t)c->rows * d, d, T, 0, false, &pd_prev));
    }
    PROF(c, PC_ELEMWISE, 1, launch_add_rmsnorm(dt, c->x, c->part, pd_prev, c->w.final_norm, m.rms_eps, c->hidden,
                                               c->lo(c->hidden, d), c->hidden_f32, T, d, s));
    if (c->tap_layer >= 0 && c->tap_layer == m.n_layers - 1) {
        MEDUSA_CUDA(c, cudaMemcpyAsync(c->tap_x_out, c->x, (size_t)c->rows * d * sizeof(float), cudaMemcpyDeviceToDevice, s));
        MEDUSA_CUDA(c, cudaMemcpyAsync(c->tap_xn_out, c->hidden, (dt == MEDUSA_BF16 ? 2 : 1) * (size_t)c->rows * d * c->esz,
                                       cudaMemcpyDeviceToDevice, s));
    }
    MEDUSA_LAUNCH_CHECK(c);
    // LM head straight into the logits buffer: whole tiles, one plane
    const void *wl[1] = {c->w.lm_head};
    PlaneDesc pd{};
    TRY(project(c, c->hidden, &c->map_hidden, wl, c->use_tc ? &c->map_lm : nullptr, 1, m.vocab, d, c->logits, 0, m.vocab, T,
                lm_row0, true, &pd));
    for (int b = 0; b < n_seq; ++b) {  // (checked flavour) the logits of every row that holds a token
        const int r0 = b * TREE_ROWS + (b == 0 ? lm_row0 : 0), r1 = b * TREE_ROWS + T_seq;
        if (r1 > r0) DEBUG_FINITE(c, c->logits + (size_t)r0 * m.vocab, (size_t)(r1 - r0) * m.vocab);
    }
    return MEDUSA_OK;
}

int32_t check_ready(medusa_ctx *c, bool need_tree, bool need_weights)
{
    if (!c) return MEDUSA_ERR_INVALID_ARG;
    if (need_tree && !c->have_tree) return fail(c, MEDUSA_ERR_STATE, "no tree uploaded: call medusa_build_tree_buffers first");
    if (need_weights && !c->have_weights) return fail(c, MEDUSA_ERR_STATE, "no weights: call medusa_load_weights first");
    return MEDUSA_OK;
}

}  // namespace

// ============================================================================ lifetime

static void drop_step_graphs(medusa_ctx *c);

// Re-points the selected-sequence views at sequence b (host pointer arithmetic only).
static void point_at(medusa_ctx *c, int b)
{
    const medusa_model_desc &m = c->m;
    const size_t K = m.n_medusa ? m.n_medusa : 1, R = (size_t)c->rows;
    c->cur = b;
    c->d_state = c->state_all + (size_t)b * ST_WORDS;
    c->h_last = c->h_last_all + (size_t)b * m.d;
    c->head_x = c->head_x_all + (size_t)b * K * m.d;
    c->head_logits = c->head_logits_all + (size_t)b * K * m.vocab;
    c->topk_idx = c->topk_idx_all + (size_t)b * K * R;
    c->acc_nodes = c->acc_nodes_all + (size_t)b * TREE_ROWS;
    c->emitted = c->emitted_all + (size_t)b * TREE_ROWS;
    c->gumbel_dev = c->gumbel_all + (size_t)b * ((size_t)m.vocab + c->rows);
    c->k_cache = c->k_cache_all ? c->k_cache_all + (size_t)b * c->cache_seq_bytes : nullptr;
    c->v_cache = c->v_cache_all ? c->v_cache_all + (size_t)b * c->cache_seq_bytes : nullptr;
    if ((size_t)b < c->L_upper_all.size()) c->L_upper = c->L_upper_all[b];
    if ((size_t)b < c->L_lower_all.size()) c->L_lower = c->L_lower_all[b];
}

extern "C" int32_t medusa_create(medusa_ctx **out, const medusa_model_desc *desc, int32_t device, void *stream)
{
    if (!out || !desc) return MEDUSA_ERR_INVALID_ARG;
    *out = nullptr;
    const medusa_model_desc &m = *desc;
    if (m.dtype != MEDUSA_F32 && m.dtype != MEDUSA_BF16) return MEDUSA_ERR_INVALID_ARG;
    if (m.n_layers < 0 || m.d < 1 || m.n_heads < 1 || m.ffn < 1 || m.vocab < 1 || m.n_medusa < 0 || m.L_max < 0)
        return MEDUSA_ERR_INVALID_ARG;
    if (m.max_tree_nodes < 0 || m.max_tree_nodes > MAX_T)
        return MEDUSA_ERR_SHAPE;  // trees of up to MAX_T nodes
    if (m.max_batch < 0 || m.max_batch > MAX_T / TREE_ROWS)
        return MEDUSA_ERR_SHAPE;  // up to MAX_T / 64 sequences (one tile of 64 token rows each)
    if (m.n_kv_heads < 0 || (m.n_kv_heads > 0 && m.n_heads % m.n_kv_heads != 0))
        return MEDUSA_ERR_SHAPE;  // every key/value head serves the same number of query heads
    const int vn = m.dtype == MEDUSA_BF16 ? 8 : 4;
    if ((m.head_dim != 64 && m.head_dim != 128) || m.d % vn || m.ffn % vn || m.n_medusa > MAX_DEPTH)
        return MEDUSA_ERR_SHAPE;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) {
        (void)cudaGetLastError();
        return MEDUSA_ERR_CUDA;  // no CPU fallback exists
    }
    medusa_ctx *c = new (std::nothrow) medusa_ctx();
    if (!c) return MEDUSA_ERR_CUDA;
    c->m = m;
    c->device = device;
    c->rows = m.max_tree_nodes <= TREE_ROWS ? TREE_ROWS : ((m.max_tree_nodes + TREE_ROWS - 1) / TREE_ROWS) * TREE_ROWS;
    c->B = m.max_batch > 1 ? m.max_batch : 1;
    if (c->rows < c->B * TREE_ROWS) c->rows = c->B * TREE_ROWS;  // a batched pass gives every sequence one tile of 64 rows
    c->L_upper_all.assign(c->B, 0);
    c->L_lower_all.assign(c->B, 0);
    c->stream = (cudaStream_t)stream;
    if (!c->stream) {
        // The legacy default stream cannot be captured into a graph.  A blocking stream orders itself with the
        // default stream in both directions, so a caller that works on the default stream sees the same order.
        cudaSetDevice(device);
        if (cudaStreamCreateWithFlags(&c->stream, cudaStreamDefault) == cudaSuccess) c->own_stream = true;
        else { c->stream = nullptr; (void)cudaGetLastError(); }
    }
    c->esz = m.dtype == MEDUSA_BF16 ? 2 : 4;
    if (const char *sk = tuning_env("MEDUSA_DEBUG_SKIP")) c->skip_mask = (unsigned)atoi(sk);
    if (const char *sg = tuning_env("MEDUSA_STEP_GRAPH")) c->step_graphs_on = atoi(sg) != 0;
    *out = c;
    MEDUSA_CUDA(c, cudaSetDevice(device));
    c->Hkv = m.n_kv_heads > 0 ? m.n_kv_heads : m.n_heads;
    const size_t d = m.d, HD = (size_t)m.n_heads * m.head_dim, HkvD = (size_t)c->Hkv * m.head_dim, F = m.ffn, V = m.vocab,
                 K = m.n_medusa, R = (size_t)c->rows;
    const size_t NB = (size_t)c->B;
    TRY(dev_alloc(c, &c->state_all, NB * ST_WORDS));
    TRY(dev_alloc(c, &c->d_mask, R * (R / 64)));
    TRY(dev_alloc(c, &c->d_chain_mask, R));
    TRY(dev_alloc(c, &c->d_pos, R));
    TRY(dev_alloc(c, &c->d_chain_pos, R));
    TRY(dev_alloc(c, &c->d_tree_idx, R));
    TRY(dev_alloc(c, &c->d_parent, R));
    TRY(dev_alloc(c, &c->d_retrieve, R * (MAX_DEPTH + 1)));
    TRY(dev_alloc(c, &c->x, R * d));
    const size_t planes = m.dtype == MEDUSA_BF16 ? 2 : 1;
    TRY(dev_alloc_bytes(c, &c->xn, planes * R * d * c->esz));
    TRY(dev_alloc_bytes(c, &c->q, planes * R * HD * c->esz));
    TRY(dev_alloc_bytes(c, &c->rot_k, R * HkvD * c->esz));
    TRY(dev_alloc_bytes(c, &c->att, planes * R * HD * c->esz));
    TRY(dev_alloc(c, &c->hidden_f32, R * d));
    TRY(dev_alloc_bytes(c, &c->act, planes * R * F * c->esz));
    TRY(dev_alloc_bytes(c, &c->hidden, planes * R * d * c->esz));
    TRY(dev_alloc(c, &c->h_last_all, NB * d));
    TRY(dev_alloc(c, &c->head_x_all, NB * (K ? K : 1) * d));
    TRY(dev_alloc(c, &c->logits, R * V));
    TRY(dev_alloc(c, &c->head_logits_all, NB * (K ? K : 1) * V));
    TRY(dev_alloc(c, &c->rope_cs, R * (size_t)(m.head_dim / 2)));
    TRY(dev_alloc(c, &c->topk_idx_all, NB * (K ? K : 1) * R));
    TRY(dev_alloc(c, &c->tree_tok, R));
    TRY(dev_alloc(c, &c->acc_nodes_all, NB * TREE_ROWS));
    TRY(dev_alloc(c, &c->emitted_all, NB * TREE_ROWS));
    TRY(dev_alloc(c, &c->node_argmax, R));
    TRY(dev_alloc(c, &c->iota, R));
    TRY(dev_alloc(c, &c->tmp_i32, 8 * NB));
    TRY(dev_alloc(c, &c->node_lse, R));
    TRY(dev_alloc(c, &c->node_ent, R));
    TRY(dev_alloc_bytes(c, &c->node_part, R * NODE_STAT_SLICES * NODE_PART_BYTES));
    TRY(dev_alloc(c, &c->gumbel_all, NB * (V + R)));  // per sequence: Gumbel noise [V], then one uniform per token row
    point_at(c, 0);
    TRY(dev_alloc_bytes(c, &c->topk_scratch, topk_scratch_bytes(m.n_medusa > 0 ? m.n_medusa : 1)));
    TRY(dev_alloc(c, &c->tap_x_in, R * d));
    TRY(dev_alloc(c, &c->tap_x_out, R * d));
    TRY(dev_alloc_bytes(c, &c->tap_att, planes * R * HD * c->esz));
    TRY(dev_alloc_bytes(c, &c->tap_xn_out, planes * R * d * c->esz));
    if (m.dtype == MEDUSA_BF16 && m.head_dim == 128 && tuning_env("MEDUSA_FORCE_SIMT_ATTENTION") == nullptr)
        TRY(dev_alloc_bytes(c, &c->flash_ws, tree_attention_flash_workspace_bytes(m.n_heads, c->rows / TREE_ROWS)));
    if (const char *e = tuning_env("MEDUSA_ATTENTION"))
        c->attn_mode = strcmp(e, "tcgen05") == 0 ? 2 : (strcmp(e, "mma_sync") == 0 ? 1 : 0);
    c->use_tc = m.dtype == MEDUSA_BF16 && tuning_env("MEDUSA_FORCE_SIMT_GEMM") == nullptr && !(d % 8 || HD % 8 || HkvD % 8 || F % 8);
    {
        // partial planes: for each projection, its width times the most pieces any of its tiles is cut into
        const size_t qkv_ld = HD + 2 * HkvD;
        size_t need = qkv_ld > 2 * F ? qkv_ld : 2 * F;
        if (d > need) need = d;
        if (c->use_tc) {
            // {segments, rows per segment, K, row width of the planes}; with fewer key/value heads than query heads
            // the QKV projection is two launches into rows of the full [q | k | v] width
            // {segments, rows per segment, K, row width of the planes, rows of segment 0}; the last two entries are the
            // two-launch form of the QKV projection (head widths that are not multiples of 128)
            const size_t shp[6][5] = {{3, HkvD, d, qkv_ld, HD}, {1, d, HD, d, d}, {2, F, d, 2 * F, F}, {1, d, F, d, d},
                                      {1, HD, d, qkv_ld, HD}, {2, HkvD, d, qkv_ld, HkvD}};
            for (int i = 0; i < 6; ++i) {
                if (i == 0 && (HD % 128 || HkvD % 128) && c->Hkv != m.n_heads) continue;
                PlaneDesc pd = gemm_tc_plan((int)shp[i][0], (int)shp[i][1], (int)shp[i][2], false, 0, (int)shp[i][4]);
                const size_t n = (size_t)pd.n_max * shp[i][3];
                if (n > need) need = n;
            }
        }
        c->part_elems = R * need;
        TRY(dev_alloc(c, &c->part, R * need));
    }
    if (c->use_tc) {
        if (!make_act_map(&c->map_xn, c->xn, (int)d, c->rows) || !make_act_map(&c->map_att, c->att, (int)HD, c->rows) ||
            !make_act_map(&c->map_act, c->act, (int)F, c->rows) || !make_act_map(&c->map_hidden, c->hidden, (int)d, c->rows))
            return fail(c, MEDUSA_ERR_CUDA, "cuTensorMapEncodeTiled failed for the activation planes");
    }
    PROF(c, PC_ELEMWISE,1, launch_iota(c->iota, (int)R, c->stream));
    MEDUSA_LAUNCH_CHECK(c);
    // chain "tree" used by prefill: node i's parent is i-1 -> lower-triangular mask, positions 0..63
    uint64_t cm[TREE_ROWS];
    int32_t cp[TREE_ROWS];
    for (int i = 0; i < TREE_ROWS; ++i) {
        cm[i] = i == 63 ? ~0ull : ((1ull << (i + 1)) - 1ull);
        cp[i] = i;
    }
    MEDUSA_CUDA(c, cudaMemcpyAsync(c->d_chain_mask, cm, sizeof cm, cudaMemcpyHostToDevice, c->stream));
    MEDUSA_CUDA(c, cudaMemcpyAsync(c->d_chain_pos, cp, sizeof cp, cudaMemcpyHostToDevice, c->stream));
    MEDUSA_CUDA(c, cudaHostAlloc((void **)&c->pinned, (TREE_ROWS + 8) * sizeof(int32_t), cudaHostAllocDefault));  // depth + 1 <= 9 tokens per step
    MEDUSA_CUDA(c, cudaStreamSynchronize(c->stream));
    return MEDUSA_OK;
}

extern "C" int32_t medusa_destroy(medusa_ctx *c)
{
    if (!c) return MEDUSA_ERR_INVALID_ARG;
    cudaSetDevice(c->device);
    cudaStreamSynchronize(c->stream);
    drop_step_graphs(c);
    for (void *p : c->allocs) cudaFree(p);
    for (auto &sp : c->spans) { cudaEventDestroy(sp.a); cudaEventDestroy(sp.b); }
    for (cudaEvent_t e : c->free_events) cudaEventDestroy(e);
    if (c->pinned) cudaFreeHost(c->pinned);
    if (c->own_stream) cudaStreamDestroy(c->stream);
    delete c;
    return MEDUSA_OK;
}

extern "C" int32_t medusa_debug_checks_enabled(void)
{
#ifdef MEDUSA_DEBUG_CHECKS
    return 1;
#else
    return 0;
#endif
}

extern "C" const char *medusa_last_error(const medusa_ctx *c) { return c ? c->err.c_str() : "null context"; }

extern "C" int32_t medusa_device_status(medusa_ctx *c)
{
    if (!c) return MEDUSA_ERR_INVALID_ARG;
    int32_t st = 0;
    MEDUSA_CUDA(c, cudaMemcpyAsync(&st, c->d_state + ST_STATUS, sizeof st, cudaMemcpyDeviceToHost, c->stream));
    MEDUSA_CUDA(c, cudaStreamSynchronize(c->stream));
    if (st != MEDUSA_OK) fail(c, st, "device status %d", st);
    return st;
}

// Drops every captured step graph: called when something a graph has baked in changes (tree, weights).
static void drop_step_graphs(medusa_ctx *c)
{
    for (auto &g : c->step_graphs) cudaGraphExecDestroy(g.exec);
    c->step_graphs.clear();
    c->have_last_key = false;
}

// Context-owned buffer `which` and its size in bytes (0 bytes: not allocated yet).
static const void *workspace_view(medusa_ctx *c, int32_t which, size_t *bytes)
{
    const medusa_model_desc &m = c->m;
    const size_t R = (size_t)c->rows, d = m.d, V = m.vocab, K = m.n_medusa ? m.n_medusa : 1, HD = (size_t)m.n_heads * m.head_dim;
    const size_t HkvD = (size_t)c->Hkv * m.head_dim, planes = m.dtype == MEDUSA_BF16 ? 2 : 1;
    const size_t cache_bytes = c->cache_seq_bytes, tree_bytes = (size_t)m.n_layers * R * HkvD * c->esz;
    const void *p = nullptr;
    size_t n = 0;
    switch (which) {
    case MEDUSA_WS_LOGITS: p = c->logits; n = R * V * sizeof(float); break;
    case MEDUSA_WS_HIDDEN: p = c->hidden_f32; n = R * d * sizeof(float); break;
    case MEDUSA_WS_TREE_K: p = c->tree_k; n = tree_bytes; break;
    case MEDUSA_WS_TREE_V: p = c->tree_v; n = tree_bytes; break;
    case MEDUSA_WS_K_CACHE: p = c->k_cache; n = cache_bytes; break;
    case MEDUSA_WS_V_CACHE: p = c->v_cache; n = cache_bytes; break;
    case MEDUSA_WS_HEAD_LOGITS: p = c->head_logits; n = K * V * sizeof(float); break;
    case MEDUSA_WS_TOPK_IDX: p = c->topk_idx; n = K * R * sizeof(int32_t); break;
    case MEDUSA_WS_TREE_TOK: p = c->tree_tok; n = R * sizeof(int32_t); break;
    case MEDUSA_WS_ACC_NODES: p = c->acc_nodes; n = TREE_ROWS * sizeof(int32_t); break;
    case MEDUSA_WS_STATE: p = c->d_state; n = ST_WORDS * sizeof(int32_t); break;
    case MEDUSA_WS_H_LAST: p = c->h_last; n = d * sizeof(float); break;
    case MEDUSA_WS_EMITTED: p = c->emitted; n = TREE_ROWS * sizeof(int32_t); break;
    case MEDUSA_WS_TAP_X_IN: p = c->tap_x_in; n = R * d * sizeof(float); break;
    case MEDUSA_WS_TAP_X_OUT: p = c->tap_x_out; n = R * d * sizeof(float); break;
    case MEDUSA_WS_TAP_ATT: p = c->tap_att; n = planes * R * HD * c->esz; break;
    case MEDUSA_WS_TAP_XN_OUT: p = c->tap_xn_out; n = planes * R * d * c->esz; break;
    default: break;
    }
    if (bytes) *bytes = p ? n : 0;
    return p;
}

extern "C" const void *medusa_workspace_ptr(medusa_ctx *c, int32_t which)
{
    return c ? workspace_view(c, which, nullptr) : nullptr;
}

extern "C" int32_t medusa_set_option(medusa_ctx *c, int32_t option, int64_t value)
{
    if (!c) return MEDUSA_ERR_INVALID_ARG;
    switch (option) {
    case MEDUSA_OPT_STEP_GRAPHS:
        c->step_graphs_on = value != 0;
        if (!c->step_graphs_on) {
            MEDUSA_CUDA(c, cudaSetDevice(c->device));
            MEDUSA_CUDA(c, cudaStreamSynchronize(c->stream));
            drop_step_graphs(c);
        }
        return MEDUSA_OK;
    case MEDUSA_OPT_ATTENTION_KERNEL:
        if (value < 0 || value > 2) return fail(c, MEDUSA_ERR_INVALID_ARG, "attention kernel must be 0 (automatic), 1 (mma.sync) or 2 (tcgen05)");
        c->attn_mode = (int)value;
        return MEDUSA_OK;
    case MEDUSA_OPT_ATTENTION_LENGTH_HINT:
        c->attn_len_hint = value < 0 ? -1 : (value > c->m.L_max ? c->m.L_max : (int)value);
        return MEDUSA_OK;
    case MEDUSA_OPT_LAYER_TAP:
        if (value >= c->m.n_layers) return fail(c, MEDUSA_ERR_INVALID_ARG, "layer tap %lld: the model has %d layers", (long long)value, c->m.n_layers);
        MEDUSA_CUDA(c, cudaSetDevice(c->device));
        MEDUSA_CUDA(c, cudaStreamSynchronize(c->stream));
        drop_step_graphs(c);  // captured steps have the old tap baked in
        c->tap_layer = value < 0 ? -1 : (int)value;
        return MEDUSA_OK;
    case MEDUSA_OPT_SPIN_LIMIT:
        if (value < 0 || value > 0x7fffffffLL) return fail(c, MEDUSA_ERR_INVALID_ARG, "spin limit out of range");
        MEDUSA_CUDA(c, cudaSetDevice(c->device));
        MEDUSA_CUDA(c, cudaStreamSynchronize(c->stream));
        drop_step_graphs(c);  // captured launches carry the old limit
        c->spin_limit = (uint32_t)value;
        return MEDUSA_OK;
    case MEDUSA_OPT_ACTIVATION_PLANES:
        if (value != 1 && value != 2) return fail(c, MEDUSA_ERR_INVALID_ARG, "activation planes: 1 or 2");
        MEDUSA_CUDA(c, cudaSetDevice(c->device));
        MEDUSA_CUDA(c, cudaStreamSynchronize(c->stream));
        drop_step_graphs(c);
        c->act_planes = (int)value;
        return MEDUSA_OK;
    case MEDUSA_OPT_PACK_WEIGHTS:
        if (value != 0 && value != 1) return fail(c, MEDUSA_ERR_INVALID_ARG, "pack weights: 0 or 1");
        c->pack_weights = value == 1;  // takes effect with the next medusa_load_weights
        return MEDUSA_OK;
    case MEDUSA_OPT_WITHHOLD_LOAD:
        if (value < 0 || value > 2) return fail(c, MEDUSA_ERR_INVALID_ARG, "withhold: 0 (off), 1 (next tensor-core GEMM) or 2 (next tcgen05 attention)");
        c->withhold = (int)value;
        return MEDUSA_OK;
    default:
        return fail(c, MEDUSA_ERR_INVALID_ARG, "unknown option %d", option);
    }
}

extern "C" int32_t medusa_step_graph_info(const medusa_ctx *c, int32_t *n_graphs_host, int64_t *n_replays_host)
{
    if (!c) return MEDUSA_ERR_INVALID_ARG;
    if (n_graphs_host) *n_graphs_host = (int32_t)c->step_graphs.size();
    if (n_replays_host) *n_replays_host = (int64_t)c->step_clock;
    return MEDUSA_OK;
}

extern "C" int32_t medusa_set_profiling(medusa_ctx *c, int32_t on)
{
    if (!c) return MEDUSA_ERR_INVALID_ARG;
    c->prof = on != 0;
    return MEDUSA_OK;
}

extern "C" int32_t medusa_get_profile(medusa_ctx *c, double *ms_host, int64_t *launches_host, int32_t reset)
{
    if (!c) return MEDUSA_ERR_INVALID_ARG;
    MEDUSA_CUDA(c, cudaSetDevice(c->device));
    MEDUSA_CUDA(c, cudaStreamSynchronize(c->stream));
    for (auto &sp : c->spans) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, sp.a, sp.b) == cudaSuccess) c->prof_ms[sp.cat] += ms;
        c->free_events.push_back(sp.a);
        c->free_events.push_back(sp.b);
    }
    c->spans.clear();
    for (int i = 0; i < MEDUSA_PROF_CATEGORIES; ++i) {
        if (ms_host) ms_host[i] = c->prof_ms[i];
        if (launches_host) launches_host[i] = c->launches[i];
        if (reset) { c->prof_ms[i] = 0.0; c->launches[i] = 0; }
    }
    return MEDUSA_OK;
}

extern "C" int32_t medusa_read_workspace(medusa_ctx *c, int32_t which, int64_t offset_bytes, void *dst_host, int64_t bytes)
{
    if (!c || !dst_host || offset_bytes < 0 || bytes < 0) return MEDUSA_ERR_INVALID_ARG;
    size_t have = 0;
    const char *p = (const char *)workspace_view(c, which, &have);
    if (!p) return fail(c, MEDUSA_ERR_STATE, "workspace buffer %d does not exist (yet)", which);
    if ((uint64_t)offset_bytes + (uint64_t)bytes > have)
        return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_read_workspace: bytes [%lld, %lld) lie outside buffer %d of %zu bytes",
                    (long long)offset_bytes, (long long)(offset_bytes + bytes), which, have);
    MEDUSA_CUDA(c, cudaSetDevice(c->device));
    MEDUSA_CUDA(c, cudaStreamSynchronize(c->stream));
    MEDUSA_CUDA(c, cudaMemcpy(dst_host, p + offset_bytes, (size_t)bytes, cudaMemcpyDeviceToHost));
    return MEDUSA_OK;
}

// Measurement aid (no counterpart in the method): enqueues a kernel that reads `bytes` bytes of `buf` with 16-byte
// streaming loads and writes nothing but a few floats to `sink`.
extern "C" int32_t medusa_stream_read(const void *buf, int64_t bytes, float *sink, int32_t sink_floats, void *stream)
{
    if (!buf || !sink || bytes < 16 || sink_floats < 1 || ((uintptr_t)buf & 15u)) return MEDUSA_ERR_INVALID_ARG;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return MEDUSA_ERR_CUDA;
    int blocks = sms * 4;
    if (blocks > sink_floats) blocks = sink_floats;
    launch_stream_read(buf, (long long)bytes, sink, blocks, (cudaStream_t)stream);
    return cudaGetLastError() == cudaSuccess ? MEDUSA_OK : MEDUSA_ERR_CUDA;
}

// ============================================================================ a0: tree

extern "C" int32_t medusa_default_tree_paths(const int32_t *per_depth_topk_host, int32_t depth, int32_t n_nodes,
                                             int32_t *paths_host_out)
{
    return default_tree_paths(per_depth_topk_host, depth, n_nodes, paths_host_out);
}

extern "C" int32_t medusa_tree_paths_from_accuracies(const double *acc_host, int32_t depth, int32_t topk, int32_t n_nodes,
                                                     int32_t *paths_host_out, double *expected_len_host_out)
{
    return tree_paths_from_accuracies(acc_host, depth, topk, n_nodes, paths_host_out, expected_len_host_out);
}

extern "C" int32_t medusa_build_tree_buffers(medusa_ctx *c, const int32_t *paths_host, int32_t n_paths,
                                             int32_t max_depth, medusa_tree_buffers *out)
{
    TreeHost tr;
    int32_t rc = build_tree(paths_host, n_paths, max_depth, tr);
    if (rc != MEDUSA_OK) return fail(c, rc, "invalid tree: tuples must be distinct, prefix-closed, -1 padded, T <= %d", MAX_T);
    if (c && tr.depth > c->m.n_medusa) return fail(c, MEDUSA_ERR_SHAPE, "tree depth %d exceeds the %d Medusa heads", tr.depth, c->m.n_medusa);
    if (c && tr.T > c->rows)
        return fail(c, MEDUSA_ERR_SHAPE, "a tree of %d nodes does not fit this context (created for trees of up to %d nodes: "
                    "set max_tree_nodes in the model descriptor)", tr.T, c->rows);
    if (out) {
        out->T = tr.T; out->P = tr.P; out->depth = tr.depth; out->topk = tr.topk;
        if (out->mask) memcpy(out->mask, tr.mask.data(), tr.mask.size() * sizeof(uint64_t));
        if (out->pos) memcpy(out->pos, tr.pos.data(), tr.T * sizeof(int32_t));
        if (out->tree_idx) memcpy(out->tree_idx, tr.tree_idx.data(), tr.T * sizeof(int32_t));
        if (out->parent) memcpy(out->parent, tr.parent.data(), tr.T * sizeof(int32_t));
        if (out->retrieve) memcpy(out->retrieve, tr.retrieve.data(), tr.retrieve.size() * sizeof(int32_t));
    }
    if (c) {
        MEDUSA_CUDA(c, cudaSetDevice(c->device));
        MEDUSA_CUDA(c, cudaStreamSynchronize(c->stream));  // earlier work may still read the old tree
        MEDUSA_CUDA(c, cudaMemcpy(c->d_mask, tr.mask.data(), tr.mask.size() * sizeof(uint64_t), cudaMemcpyHostToDevice));
        MEDUSA_CUDA(c, cudaMemcpy(c->d_pos, tr.pos.data(), tr.T * sizeof(int32_t), cudaMemcpyHostToDevice));
        MEDUSA_CUDA(c, cudaMemcpy(c->d_tree_idx, tr.tree_idx.data(), tr.T * sizeof(int32_t), cudaMemcpyHostToDevice));
        MEDUSA_CUDA(c, cudaMemcpy(c->d_parent, tr.parent.data(), tr.T * sizeof(int32_t), cudaMemcpyHostToDevice));
        MEDUSA_CUDA(c, cudaMemcpy(c->d_retrieve, tr.retrieve.data(), tr.retrieve.size() * sizeof(int32_t), cudaMemcpyHostToDevice));
        drop_step_graphs(c);  // captured steps have the old tree's sizes baked in
        c->tree = tr;
        c->have_tree = true;
    }
    return MEDUSA_OK;
}

// ============================================================================ a1-a4: heads

static int32_t heads_impl(medusa_ctx *c, const void *h, int h_is_f32, const void *W1, const void *W2,
                          const int32_t *root_token, int32_t *topk_idx, float *topk_val, float *logits_dump,
                          int32_t *tree_tok)
{
    TRY(check_ready(c, true, false));
    const int K = c->tree.depth;  // heads deeper than the tree are unused (paper Sec. 2.2: no overhead)
    if (!h || !root_token || !tree_tok || (K > 0 && (!W1 || !W2 || !topk_idx)))
        return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_heads: null pointer");
    if (!aligned16(h) || !aligned16(W1) || !aligned16(W2))
        return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_heads: tensors must be 16-byte aligned");
    MEDUSA_CUDA(c, cudaSetDevice(c->device));
    float *z = logits_dump ? logits_dump : c->head_logits;
    if (K > 0) {
        PROF(c, PC_HEADS,1, launch_heads_resblock(c->m.dtype, h, h_is_f32, W1, c->head_x, K, c->m.d, c->stream));
        PROF(c, PC_HEADS,1, launch_heads_vocab(c->m.dtype, c->head_x, W2, z, K, c->m.d, c->m.vocab, c->stream));
        PROF(c, PC_TOPK, c->tree.topk <= 8 ? 2 : 1,
             launch_topk(z, K, c->m.vocab, c->tree.topk, topk_idx, topk_val, c->topk_scratch, c->stream));
    }
    PROF(c, PC_TOPK,1, launch_expand(root_token, topk_idx, c->d_tree_idx, tree_tok, c->tree.T, c->stream));
    if (K > 0) DEBUG_FINITE(c, z, (size_t)K * c->m.vocab);
    DEBUG_RANGE(c, tree_tok, c->tree.T, 0, c->m.vocab - 1);
    MEDUSA_LAUNCH_CHECK(c);
    return MEDUSA_OK;
}

extern "C" int32_t medusa_heads(medusa_ctx *c, const void *h, const void *W1, const void *W2, const int32_t *root_token,
                                int32_t *topk_idx, float *topk_val, float *logits_dump, int32_t *tree_tok)
{
    return heads_impl(c, h, 0, W1, W2, root_token, topk_idx, topk_val, logits_dump, tree_tok);
}

// ============================================================================ a6: tree attention

extern "C" int32_t medusa_tree_attention(medusa_ctx *c, const void *q, const void *k_new, const void *v_new,
                                         const void *k_cache, const void *v_cache, const int32_t *cache_len,
                                         int32_t apply_rope, void *out, float *lse)
{
    TRY(check_ready(c, true, false));
    if (!q || !k_new || !v_new || !cache_len || !out || (c->m.L_max > 0 && (!k_cache || !v_cache)))
        return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_tree_attention: null pointer");
    if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(out))
        return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_tree_attention: tensors must be 16-byte aligned");
    MEDUSA_CUDA(c, cudaSetDevice(c->device));
    DEBUG_RANGE(c, cache_len, 1, 0, c->m.L_max);
    const medusa_model_desc &m = c->m;
    const int T = c->tree.T;
    const void *qq = q, *kk = k_new;
    if (apply_rope) {
        PROF(c, PC_ELEMWISE,1, launch_rope_table(c->rope_cs, cache_len, c->d_pos, T, m.head_dim, m.rope_theta, c->stream));
        PROF(c, PC_ELEMWISE,1, launch_rope_apply(m.dtype, q, c->rope_cs, c->q, T, m.n_heads, m.head_dim, c->stream));
        PROF(c, PC_ELEMWISE,1, launch_rope_apply(m.dtype, k_new, c->rope_cs, c->rot_k, T, c->Hkv, m.head_dim, c->stream));
        qq = c->q;
        kk = c->rot_k;
    }
    MEDUSA_LAUNCH_CHECK(c);
    // the cache length lives on the device here: the kernel choice and the tcgen05 kernel's grid follow the caller's
    // bound (MEDUSA_OPT_ATTENTION_LENGTH_HINT), or the full capacity if none was given
    const int hint = c->attn_len_hint < 0 || c->attn_len_hint > m.L_max ? m.L_max : c->attn_len_hint;
    return attention(c, qq, kk, v_new, k_cache, v_cache, cache_len, c->d_mask, out, nullptr, lse, T, hint, false, c->tree.mask_words);
}

// ============================================================================ a7: acceptance

static bool known_mode(int32_t mode) { return mode == MEDUSA_GREEDY || mode == MEDUSA_TYPICAL || mode == MEDUSA_REJECTION; }
// floats of one step's noise row: Gumbel noise for the vocabulary, for rejection sampling also one uniform per tree node
static size_t noise_floats(const medusa_ctx *c, int32_t mode)
{
    return (size_t)c->m.vocab + (mode == MEDUSA_REJECTION ? (size_t)c->tree.T : 0);
}
// whether the acceptance kernels read the noise row in this mode
static bool mode_reads_noise(const medusa_accept_params *p) { return p->mode == MEDUSA_TYPICAL || p->mode == MEDUSA_REJECTION; }

extern "C" int32_t medusa_evaluate_posterior(medusa_ctx *c, const float *logits, const int32_t *tree_tok,
                                             const medusa_accept_params *params, const float *gumbel, int32_t *best,
                                             int32_t *accept_len, int32_t *next_root, int32_t *acc_nodes)
{
    TRY(check_ready(c, true, false));
    if (!logits || !tree_tok || !params || !best || !accept_len || !next_root || !acc_nodes)
        return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_evaluate_posterior: null pointer");
    if (!known_mode(params->mode))
        return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_evaluate_posterior: unknown mode %d", params->mode);
    if (params->mode == MEDUSA_REJECTION && (!gumbel || !(params->temperature > 0.f)))
        return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_evaluate_posterior: rejection sampling needs a noise row and a temperature above zero");
    MEDUSA_CUDA(c, cudaSetDevice(c->device));
    PosteriorArgs a{};
    a.logits = logits; a.tree_tok = tree_tok; a.retrieve = c->d_retrieve; a.parent = c->d_parent; a.gumbel = gumbel;
    a.uniform = params->mode == MEDUSA_REJECTION ? gumbel + c->m.vocab : nullptr;  // the noise row is gumbel[V], uniform[T]
    a.T = c->tree.T; a.V = c->m.vocab; a.P = c->tree.P; a.depth = c->tree.depth; a.mode = params->mode;
    a.temperature = params->temperature; a.eps = params->eps; a.delta = params->delta;
    a.node_argmax = c->node_argmax; a.node_lse = c->node_lse; a.node_ent = c->node_ent;
    a.node_part = c->node_part; a.stat_slices = NODE_STAT_SLICES;
    a.best = best; a.accept_len = accept_len; a.next_root = next_root; a.acc_nodes = acc_nodes;
    PROF(c, PC_POSTERIOR,2, launch_evaluate_posterior(a, c->stream));
    DEBUG_RANGE(c, acc_nodes, c->tree.depth + 1, -1, c->tree.T - 1);
    DEBUG_RANGE(c, best, 1, 0, c->tree.P - 1);
    DEBUG_RANGE(c, accept_len, 1, 0, c->tree.depth);
    DEBUG_RANGE(c, next_root, 1, 0, c->m.vocab - 1);
    MEDUSA_LAUNCH_CHECK(c);
    return MEDUSA_OK;
}

// ============================================================================ a8: commit

extern "C" int32_t medusa_accept_and_update_kv(medusa_ctx *c, const void *tree_k, const void *tree_v, void *k_cache,
                                               void *v_cache, const int32_t *acc_nodes, const int32_t *accept_len,
                                               int32_t max_commit, int32_t *cache_len, const float *hidden, float *h_last,
                                               const int32_t *tree_tok, int32_t *emitted, int32_t *n_emitted)
{
    TRY(check_ready(c, true, false));
    if (!tree_k || !tree_v || !k_cache || !v_cache || !acc_nodes || !accept_len || !cache_len || !hidden || !h_last ||
        !tree_tok || !emitted || !n_emitted)
        return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_accept_and_update_kv: null pointer");
    if (!aligned16(tree_k) || !aligned16(tree_v) || !aligned16(k_cache) || !aligned16(v_cache))
        return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_accept_and_update_kv: tensors must be 16-byte aligned");
    if (max_commit < 0) return fail(c, MEDUSA_ERR_INVALID_ARG, "max_commit < 0");
    MEDUSA_CUDA(c, cudaSetDevice(c->device));
    CommitArgs a{};
    a.tree_k = tree_k; a.tree_v = tree_v; a.k_cache = k_cache; a.v_cache = v_cache; a.acc_nodes = acc_nodes;
    a.accept_len = accept_len; a.max_commit = max_commit; a.cache_len = cache_len; a.hidden = hidden; a.h_last = h_last;
    a.tree_tok = tree_tok; a.emitted = emitted; a.n_emitted = n_emitted; a.status = c->d_state + ST_STATUS;
    a.next_root = nullptr; a.root_out = nullptr;
    a.tree_rows = c->rows; a.n_layers = c->m.n_layers; a.H = c->Hkv; a.D = c->m.head_dim; a.L_max = c->m.L_max; a.d = c->m.d;
    a.depth_plus1 = c->tree.depth + 1;
    PROF(c, PC_COMMIT,2, launch_commit(c->m.dtype, a, c->stream));
    MEDUSA_LAUNCH_CHECK(c);
    return MEDUSA_OK;
}

// ============================================================================ driver

extern "C" int32_t medusa_load_weights(medusa_ctx *c, const medusa_weights *w)
{
    if (!c || !w) return MEDUSA_ERR_INVALID_ARG;
    const medusa_model_desc &m = c->m;
    if (!w->embed || !w->final_norm || !w->lm_head || (m.n_layers > 0 && !w->layers_host) ||
        (m.n_medusa > 0 && (!w->medusa_w1 || !w->medusa_w2)))
        return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_load_weights: null pointer");
    drop_step_graphs(c);
    c->layers.assign(w->layers_host, w->layers_host + (size_t)m.n_layers * 9);
    for (const void *p : c->layers)
        if (!p || !aligned16(p)) return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_load_weights: layer pointer null or misaligned");
    c->w = *w;
    c->w.layers_host = nullptr;
    MEDUSA_CUDA(c, cudaSetDevice(c->device));
    if (!c->k_cache_all) {
        const size_t HkvD = (size_t)c->Hkv * m.head_dim;
        const size_t cache_bytes = (size_t)m.n_layers * HkvD * m.L_max * c->esz;
        const size_t tree_bytes = (size_t)m.n_layers * c->rows * HkvD * c->esz;
        c->cache_seq_bytes = cache_bytes;
        TRY(dev_alloc_bytes(c, (void **)&c->k_cache_all, cache_bytes * c->B));
        TRY(dev_alloc_bytes(c, (void **)&c->v_cache_all, cache_bytes * c->B));
        point_at(c, c->cur);
        TRY(dev_alloc_bytes(c, &c->tree_k, tree_bytes));
        TRY(dev_alloc_bytes(c, &c->tree_v, tree_bytes));
    }
    if (c->use_tc) {
        const int d = m.d, HD = m.n_heads * m.head_dim, HkvD = c->Hkv * m.head_dim, F = m.ffn;
        c->wmaps.resize((size_t)m.n_layers * 7);
        c->packed_on = c->pack_weights;
        if (!c->packed_copies.empty()) {  // weights loaded anew: the previous packed copies go
            MEDUSA_CUDA(c, cudaStreamSynchronize(c->stream));
            for (void *p : c->packed_copies) {
                cudaFree(p);
                c->allocs.erase(std::remove(c->allocs.begin(), c->allocs.end(), p), c->allocs.end());
            }
            c->packed_copies.clear();
        }
        bool ok = true;
        // one matrix: its map over the caller's tensor, or a packed copy of it (kept by the context) and that copy's map
        auto add = [&](TensorMap *tm, const void *W, int N, int K) -> int32_t {
            if (!c->packed_on) {
                ok = ok && make_weight_map(tm, W, N, K);
                return MEDUSA_OK;
            }
            void *Wp = nullptr;
            TRY(dev_alloc_bytes(c, &Wp, packed_weight_elems(N, K) * 2));
            c->packed_copies.push_back(Wp);
            launch_pack_weight(W, N, K, Wp, c->stream);
            ok = ok && make_packed_weight_map(tm, Wp, N, K);
            return MEDUSA_OK;
        };
        TRY(add(&c->map_lm, w->lm_head, m.vocab, d));
        for (int l = 0; l < m.n_layers && ok; ++l) {
            const void *const *lw = c->layers.data() + (size_t)l * 9;
            TensorMap *wm = c->wmaps.data() + (size_t)l * 7;
            TRY(add(wm + 0, lw[1], HD, d));
            TRY(add(wm + 1, lw[2], HkvD, d));
            TRY(add(wm + 2, lw[3], HkvD, d));
            TRY(add(wm + 3, lw[4], d, HD));
            TRY(add(wm + 4, lw[6], F, d));
            TRY(add(wm + 5, lw[7], F, d));
            TRY(add(wm + 6, lw[8], d, F));
        }
        MEDUSA_LAUNCH_CHECK(c);
        if (!ok) return fail(c, MEDUSA_ERR_CUDA, "cuTensorMapEncodeTiled failed for a weight matrix");
    }
    c->have_weights = true;
    return medusa_reset(c);
}

extern "C" int32_t medusa_reset(medusa_ctx *c)
{
    if (!c) return MEDUSA_ERR_INVALID_ARG;
    MEDUSA_CUDA(c, cudaSetDevice(c->device));
    MEDUSA_CUDA(c, cudaMemsetAsync(c->state_all, 0, (size_t)c->B * ST_WORDS * sizeof(int32_t), c->stream));
    c->L_upper_all.assign(c->B, 0);
    c->L_lower_all.assign(c->B, 0);
    c->L_upper = 0;
    c->L_lower = 0;
    return MEDUSA_OK;
}

// prompt: device pointer.  cache_len_host: what the host knows the cache length to be (prefill is only
// legal right after reset or another prefill, so the host can track it).
static int32_t prefill_dev(medusa_ctx *c, const int32_t *prompt, int32_t n, int32_t L0)
{
    const medusa_model_desc &m = c->m;
    if (L0 + n > m.L_max) return fail(c, MEDUSA_ERR_CACHE_FULL, "prompt of %d tokens does not fit the cache (L_max %d)", n, m.L_max);
    for (int off = 0; off < n; off += TREE_ROWS) {
        const int T = n - off < TREE_ROWS ? n - off : TREE_ROWS;
        TRY(tree_pass(c, prompt + off, T, c->d_chain_mask, c->d_chain_pos, T - 1, 1));
        PROF(c, PC_ELEMWISE, 1, (launch_pdl(set_i32_kernel, dim3(1), dim3(1), 0, c->stream, c->tmp_i32, T - 1)));  // "accept_len" of a chain: everything
        PROF(c, PC_POSTERIOR,1, launch_argmax_row(c->logits, m.vocab, T - 1, c->tmp_i32 + 1, c->stream));
        CommitArgs a{};
        a.tree_k = c->tree_k; a.tree_v = c->tree_v; a.k_cache = c->k_cache; a.v_cache = c->v_cache;
        a.acc_nodes = c->iota; a.accept_len = c->tmp_i32; a.max_commit = T; a.cache_len = c->d_state + ST_CACHE_LEN;
        a.hidden = c->hidden_f32; a.h_last = c->h_last; a.tree_tok = prompt + off; a.emitted = c->emitted;
        a.n_emitted = c->d_state + ST_N_EMITTED; a.status = c->d_state + ST_STATUS;
        a.next_root = c->tmp_i32 + 1; a.root_out = c->d_state + ST_ROOT;
        a.tree_rows = c->rows; a.n_layers = m.n_layers; a.H = c->Hkv; a.D = m.head_dim; a.L_max = m.L_max; a.d = m.d; a.depth_plus1 = T;
        PROF(c, PC_COMMIT,2, launch_commit(m.dtype, a, c->stream));
        MEDUSA_LAUNCH_CHECK(c);
        c->L_upper += T;
        c->L_lower += T;
    }
    return MEDUSA_OK;
}

extern "C" int32_t medusa_prefill(medusa_ctx *c, const int32_t *prompt, int32_t n)
{
    TRY(check_ready(c, false, true));
    if (!prompt || n < 1) return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_prefill: empty prompt");
    MEDUSA_CUDA(c, cudaSetDevice(c->device));
    int32_t L0 = 0;
    MEDUSA_CUDA(c, cudaMemcpyAsync(&L0, c->d_state + ST_CACHE_LEN, sizeof L0, cudaMemcpyDeviceToHost, c->stream));
    MEDUSA_CUDA(c, cudaStreamSynchronize(c->stream));
    c->L_upper = L0;
    c->L_lower = L0;
    return prefill_dev(c, prompt, n, L0);
}

extern "C" int32_t medusa_tree_pass(medusa_ctx *c, const int32_t *tokens)
{
    TRY(check_ready(c, true, true));
    if (!tokens) return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_tree_pass: null tokens");
    MEDUSA_CUDA(c, cudaSetDevice(c->device));
    return tree_pass(c, tokens, c->tree.T, c->d_mask, c->d_pos, 0, c->tree.mask_words);
}

// Everything one decode step enqueues on the context's stream (no host-side state is touched).
static int32_t decode_step_launches(medusa_ctx *c, const medusa_accept_params *params, const float *gumbel,
                                    int32_t max_commit, int32_t *emitted_host, int32_t *n_emitted_host)
{
    const medusa_model_desc &m = c->m;
    int32_t *st = c->d_state;
    // (1) candidates: heads on the last accepted hidden state, top-k, tree tokens
    TRY(heads_impl(c, c->h_last, 1, c->w.medusa_w1, c->w.medusa_w2, st + ST_ROOT, c->topk_idx, nullptr, nullptr, c->tree_tok));
    // (2) process them: one backbone pass with tree attention
    TRY(tree_pass(c, c->tree_tok, c->tree.T, c->d_mask, c->d_pos, 0, c->tree.mask_words));
    // (3) accept: longest accepted prefix, then commit its K/V
    TRY(medusa_evaluate_posterior(c, c->logits, c->tree_tok, params, gumbel, st + ST_BEST, st + ST_ACCEPT_LEN,
                                  st + ST_NEXT_ROOT, c->acc_nodes));
    CommitArgs a{};
    a.tree_k = c->tree_k; a.tree_v = c->tree_v; a.k_cache = c->k_cache; a.v_cache = c->v_cache;
    a.acc_nodes = c->acc_nodes; a.accept_len = st + ST_ACCEPT_LEN; a.max_commit = max_commit;
    a.cache_len = st + ST_CACHE_LEN; a.hidden = c->hidden_f32; a.h_last = c->h_last; a.tree_tok = c->tree_tok;
    a.emitted = c->emitted; a.n_emitted = st + ST_N_EMITTED; a.status = st + ST_STATUS;
    a.next_root = st + ST_NEXT_ROOT; a.root_out = st + ST_ROOT;
    a.tree_rows = c->rows; a.n_layers = m.n_layers; a.H = c->Hkv; a.D = m.head_dim; a.L_max = m.L_max; a.d = m.d;
    a.depth_plus1 = c->tree.depth + 1;
    PROF(c, PC_COMMIT,2, launch_commit(m.dtype, a, c->stream));
    MEDUSA_LAUNCH_CHECK(c);
    if (emitted_host)
        MEDUSA_CUDA(c, cudaMemcpyAsync(emitted_host, c->emitted, (c->tree.depth + 1) * sizeof(int32_t), cudaMemcpyDeviceToHost, c->stream));
    if (n_emitted_host)
        MEDUSA_CUDA(c, cudaMemcpyAsync(n_emitted_host, st + ST_N_EMITTED, sizeof(int32_t), cudaMemcpyDeviceToHost, c->stream));
    return MEDUSA_OK;
}

// A host pointer can be the target of a copy inside a captured graph only if it is page-locked.
static bool graph_safe_host_ptr(const void *p)
{
    if (!p) return true;
    cudaPointerAttributes at{};
    if (cudaPointerGetAttributes(&at, p) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return at.type != cudaMemoryTypeUnregistered;
}

constexpr size_t MAX_STEP_GRAPHS = 16;

// Captures one step with key `key` from the stream and instantiates it.  Nothing runs during the capture; on any
// failure the capture is closed, step graphs are switched off for this context and false is returned (the caller
// then enqueues the step directly).
static int32_t decode_step_batch_launches(medusa_ctx *c, const medusa_accept_params *params, const float *gumbel,
                                          int32_t max_commit, int32_t *emitted_host, int32_t *n_emitted_host);

static bool capture_step_graph(medusa_ctx *c, const medusa_ctx::StepKey &key, const medusa_accept_params *params,
                               const float *gumbel)
{
    int64_t before[MEDUSA_PROF_CATEGORIES];
    memcpy(before, c->launches, sizeof before);
    const std::string err_before = c->err;
    bool ok = cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeThreadLocal) == cudaSuccess;
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t exec = nullptr;
    if (ok) {
        const int32_t rc = key.seq < 0  // a batched step (all sequences) or the selected sequence's step
                               ? decode_step_batch_launches(c, params, gumbel, key.max_commit, key.emitted_host, key.n_emitted_host)
                               : decode_step_launches(c, params, gumbel, key.max_commit, key.emitted_host, key.n_emitted_host);
        const cudaError_t e = cudaStreamEndCapture(c->stream, &graph);
        ok = rc == MEDUSA_OK && e == cudaSuccess && graph != nullptr;
    }
    if (ok) ok = cudaGraphInstantiate(&exec, graph, 0) == cudaSuccess;
    if (graph) cudaGraphDestroy(graph);
    if (!ok) {
        cudaGetLastError();  // the failed capture leaves a non-sticky error behind
        memcpy(c->launches, before, sizeof before);
        c->err = err_before;
        c->step_graphs_on = false;
        return false;
    }
    if (c->step_graphs.size() >= MAX_STEP_GRAPHS) {  // make room: drop the graph that was used longest ago
        size_t old = 0;
        for (size_t i = 1; i < c->step_graphs.size(); ++i)
            if (c->step_graphs[i].used < c->step_graphs[old].used) old = i;
        cudaGraphExecDestroy(c->step_graphs[old].exec);
        c->step_graphs.erase(c->step_graphs.begin() + old);
    }
    medusa_ctx::StepGraph g{};
    g.key = key;
    g.exec = exec;
    for (int i = 0; i < MEDUSA_PROF_CATEGORIES; ++i) g.launches[i] = c->launches[i] - before[i];
    memcpy(c->launches, before, sizeof before);  // the replay below accounts for them
    g.used = 0;
    c->step_graphs.push_back(g);
    return true;
}

extern "C" int32_t medusa_decode_step(medusa_ctx *c, const medusa_accept_params *params, const float *gumbel,
                                      int32_t max_commit, int32_t *emitted_host, int32_t *n_emitted_host)
{
    TRY(check_ready(c, true, true));
    if (!params) return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_decode_step: null params");
    if (max_commit < 1) return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_decode_step: max_commit must be >= 1");
    if (!known_mode(params->mode))
        return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_decode_step: unknown mode %d", params->mode);
    if (params->mode == MEDUSA_REJECTION && (!gumbel || !(params->temperature > 0.f)))
        return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_decode_step: rejection sampling needs a noise row and a temperature above zero");
    const medusa_model_desc &m = c->m;
    const int32_t depth1 = c->tree.depth + 1;
    if (max_commit > depth1) max_commit = depth1;  // a step never commits more than one root-to-leaf path
    MEDUSA_CUDA(c, cudaSetDevice(c->device));

    // (a captured launch of the tcgen05 attention kernel freezes the grid it sized from the host's bound of the cache
    // length; the kernel copes with a cache that has grown past that bound -- its last grid row takes the remaining
    // tiles -- so replaying it stays correct, only less evenly split)
    bool graphed = false;
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    if (c->step_graphs_on && !c->prof && c->skip_mask == 0 && c->withhold == 0 &&
        cudaStreamIsCapturing(c->stream, &capturing) == cudaSuccess && capturing == cudaStreamCaptureStatusNone) {
        medusa_ctx::StepKey key;
        memset(&key, 0, sizeof key);
        key.max_commit = max_commit;
        key.seq = c->cur;
        key.long_cache = c->attn_mode == 0 && c->L_lower >= ATTN_TC_STEP_MIN_L ? 1 : 0;
        const bool noisy = gumbel && mode_reads_noise(params);  // the acceptance kernel's own condition
        key.has_gumbel = noisy ? 1 : 0;
        key.p = *params;
        key.emitted_host = emitted_host;
        key.n_emitted_host = n_emitted_host;
        medusa_ctx::StepGraph *g = nullptr;
        for (auto &cand : c->step_graphs)
            if (memcmp(&cand.key, &key, sizeof key) == 0) g = &cand;
        if (!g && c->have_last_key && memcmp(&c->last_key, &key, sizeof key) == 0 && graph_safe_host_ptr(emitted_host) &&
            graph_safe_host_ptr(n_emitted_host) &&
            capture_step_graph(c, key, params, noisy ? c->gumbel_dev : nullptr))
            g = &c->step_graphs.back();
        c->last_key = key;
        c->have_last_key = true;
        if (g) {
            // the graph reads the step's noise row from the context's own buffer
            if (noisy && gumbel != c->gumbel_dev)
                MEDUSA_CUDA(c, cudaMemcpyAsync(c->gumbel_dev, gumbel, noise_floats(c, params->mode) * sizeof(float), cudaMemcpyDeviceToDevice, c->stream));
            MEDUSA_CUDA(c, cudaGraphLaunch(g->exec, c->stream));
            for (int i = 0; i < MEDUSA_PROF_CATEGORIES; ++i) c->launches[i] += g->launches[i];
            g->used = ++c->step_clock;
            graphed = true;
        }
    }
    if (!graphed)
        TRY(decode_step_launches(c, params, gumbel, max_commit, emitted_host, n_emitted_host));
    c->L_upper += max_commit;
    if (c->L_upper > m.L_max) c->L_upper = m.L_max;
    if (c->L_lower < m.L_max) c->L_lower += 1;  // a step that is not refused for a full cache commits at least one token
    return MEDUSA_OK;
}

extern "C" int32_t medusa_select_sequence(medusa_ctx *c, int32_t b)
{
    if (!c) return MEDUSA_ERR_INVALID_ARG;
    if (b < 0 || b >= c->B) return fail(c, MEDUSA_ERR_INVALID_ARG, "sequence %d: the context holds %d sequence(s)", b, c->B);
    c->L_upper_all[c->cur] = c->L_upper;
    c->L_lower_all[c->cur] = c->L_lower;
    point_at(c, b);
    c->have_last_key = false;  // the next step belongs to another sequence: its graph is found by the key's sequence index
    return MEDUSA_OK;
}

// One step of ALL sequences of the context in one backbone pass (batch > 1): the heads and the integer stages run per
// sequence, the projections once over all sequences' token rows.
extern "C" int32_t medusa_decode_step_batch(medusa_ctx *c, const medusa_accept_params *params, const float *gumbel,
                                            int32_t max_commit, int32_t *emitted_host, int32_t *n_emitted_host)
{
    TRY(check_ready(c, true, true));
    if (!params) return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_decode_step_batch: null params");
    if (max_commit < 1) return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_decode_step_batch: max_commit must be >= 1");
    if (!known_mode(params->mode))
        return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_decode_step_batch: unknown mode %d", params->mode);
    if (params->mode == MEDUSA_REJECTION && (!gumbel || !(params->temperature > 0.f)))
        return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_decode_step_batch: rejection sampling needs noise rows and a temperature above zero");
    if (c->tree.T > TREE_ROWS)
        return fail(c, MEDUSA_ERR_SHAPE, "a batched step gives every sequence one tile of 64 token rows: the tree has %d nodes", c->tree.T);
    const medusa_model_desc &m = c->m;
    const int B = c->B, depth1 = c->tree.depth + 1;
    if (max_commit > depth1) max_commit = depth1;
    MEDUSA_CUDA(c, cudaSetDevice(c->device));
    const int keep = c->cur;
    c->L_upper_all[keep] = c->L_upper;
    c->L_lower_all[keep] = c->L_lower;

    // The launches of a batched step depend on the host through the same values as a single step's (acceptance parameters,
    // commit budget, presence of noise, the host result pointers): the second consecutive batched step with the same key
    // is captured into a graph (sequence index -1 in the key) and replayed afterwards.
    bool graphed = false;
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    if (c->step_graphs_on && !c->prof && c->skip_mask == 0 && c->withhold == 0 &&
        cudaStreamIsCapturing(c->stream, &capturing) == cudaSuccess && capturing == cudaStreamCaptureStatusNone) {
        medusa_ctx::StepKey key;
        memset(&key, 0, sizeof key);
        key.max_commit = max_commit;
        key.seq = -1;
        const bool noisy = gumbel && mode_reads_noise(params);
        key.has_gumbel = noisy ? 1 : 0;
        key.p = *params;
        key.emitted_host = emitted_host;
        key.n_emitted_host = n_emitted_host;
        medusa_ctx::StepGraph *g = nullptr;
        for (auto &cand : c->step_graphs)
            if (memcmp(&cand.key, &key, sizeof key) == 0) g = &cand;
        if (!g && c->have_last_key && memcmp(&c->last_key, &key, sizeof key) == 0 && graph_safe_host_ptr(emitted_host) &&
            graph_safe_host_ptr(n_emitted_host) && capture_step_graph(c, key, params, noisy ? c->gumbel_all : nullptr))
            g = &c->step_graphs.back();
        c->last_key = key;
        c->have_last_key = true;
        if (g) {
            // the graph reads the sequences' noise rows from the context's own buffer, packed [B][row]
            if (noisy && gumbel != c->gumbel_all)
                MEDUSA_CUDA(c, cudaMemcpyAsync(c->gumbel_all, gumbel, (size_t)B * noise_floats(c, params->mode) * sizeof(float),
                                               cudaMemcpyDeviceToDevice, c->stream));
            MEDUSA_CUDA(c, cudaGraphLaunch(g->exec, c->stream));
            for (int i = 0; i < MEDUSA_PROF_CATEGORIES; ++i) c->launches[i] += g->launches[i];
            g->used = ++c->step_clock;
            graphed = true;
        }
    }
    int32_t rc = MEDUSA_OK;
    if (!graphed) rc = decode_step_batch_launches(c, params, gumbel, max_commit, emitted_host, n_emitted_host);
    for (int b = 0; b < B; ++b) {
        const int up = c->L_upper_all[b] + max_commit;
        c->L_upper_all[b] = up > m.L_max ? m.L_max : up;
        if (c->L_lower_all[b] < m.L_max) c->L_lower_all[b] += 1;
    }
    point_at(c, keep);
    return rc;
}

// The launches of one batched step (also what a capture records).  Leaves the selected-sequence views on the last sequence.
static int32_t decode_step_batch_launches(medusa_ctx *c, const medusa_accept_params *params, const float *gumbel,
                                          int32_t max_commit, int32_t *emitted_host, int32_t *n_emitted_host)
{
    const medusa_model_desc &m = c->m;
    const int B = c->B, depth1 = c->tree.depth + 1, T = c->tree.T;
    int32_t rc = MEDUSA_OK;
    // (1) candidates of every sequence: the heads of all sequences in two launches (every head weight is read once),
    // then top-k and the sequence's tile of tree tokens per sequence
    {
        const int K = c->tree.depth;
        const size_t Ka = m.n_medusa ? m.n_medusa : 1;  // heads the per-sequence buffers are laid out for
        if (K > 0) {
            cudaError_t e = cudaSuccess;
            PROF(c, PC_HEADS, 1, e = launch_heads_resblock_batch(m.dtype, c->h_last_all, m.d, c->w.medusa_w1, c->head_x_all,
                                                                 (long long)(Ka * m.d), K, m.d, B, c->stream));
            if (e == cudaSuccess)
                PROF(c, PC_HEADS, 1, e = launch_heads_vocab_batch(m.dtype, c->head_x_all, (long long)(Ka * m.d), c->w.medusa_w2,
                                                                  c->head_logits_all, (long long)(Ka * m.vocab), K, m.d, m.vocab, B,
                                                                  c->stream));
            if (e != cudaSuccess) rc = fail(c, MEDUSA_ERR_CUDA, "batched heads launch failed: %s", cudaGetErrorString(e));
        }
        for (int b = 0; b < B && rc == MEDUSA_OK; ++b) {
            point_at(c, b);
            if (K > 0)
                PROF(c, PC_TOPK, c->tree.topk <= 8 ? 2 : 1,
                     launch_topk(c->head_logits, K, m.vocab, c->tree.topk, c->topk_idx, nullptr, c->topk_scratch, c->stream));
            PROF(c, PC_TOPK, 1, launch_expand(c->d_state + ST_ROOT, c->topk_idx, c->d_tree_idx, c->tree_tok + (size_t)b * TREE_ROWS,
                                              c->tree.T, c->stream));
            if (cudaGetLastError() != cudaSuccess) rc = fail(c, MEDUSA_ERR_CUDA, "top-k / expansion launch failed");
        }
    }
    // (2) one backbone pass over all sequences' tiles
    if (rc == MEDUSA_OK) rc = tree_pass(c, c->tree_tok, T, c->d_mask, c->d_pos, 0, c->tree.mask_words, B);
    // (3) acceptance and commit, sequence by sequence
    for (int b = 0; b < B && rc == MEDUSA_OK; ++b) {
        point_at(c, b);
        int32_t *st = c->d_state;
        const size_t ro = (size_t)b * TREE_ROWS;
        rc = medusa_evaluate_posterior(c, c->logits + ro * m.vocab, c->tree_tok + ro, params,
                                       gumbel ? gumbel + (size_t)b * noise_floats(c, params->mode) : nullptr, st + ST_BEST, st + ST_ACCEPT_LEN,
                                       st + ST_NEXT_ROOT, c->acc_nodes);
        if (rc != MEDUSA_OK) break;
        CommitArgs a{};
        const size_t HkvD = (size_t)c->Hkv * m.head_dim;
        a.tree_k = (const char *)c->tree_k + ro * HkvD * c->esz; a.tree_v = (const char *)c->tree_v + ro * HkvD * c->esz;
        a.k_cache = c->k_cache; a.v_cache = c->v_cache;
        a.acc_nodes = c->acc_nodes; a.accept_len = st + ST_ACCEPT_LEN; a.max_commit = max_commit;
        a.cache_len = st + ST_CACHE_LEN; a.hidden = c->hidden_f32 + ro * m.d; a.h_last = c->h_last; a.tree_tok = c->tree_tok + ro;
        a.emitted = c->emitted; a.n_emitted = st + ST_N_EMITTED; a.status = st + ST_STATUS;
        a.next_root = st + ST_NEXT_ROOT; a.root_out = st + ST_ROOT;
        a.tree_rows = c->rows; a.n_layers = m.n_layers; a.H = c->Hkv; a.D = m.head_dim; a.L_max = m.L_max; a.d = m.d;
        a.depth_plus1 = depth1;
        PROF(c, PC_COMMIT, 2, launch_commit(m.dtype, a, c->stream));
        if (cudaGetLastError() != cudaSuccess) { rc = fail(c, MEDUSA_ERR_CUDA, "commit launch failed"); break; }
        if (emitted_host &&
            cudaMemcpyAsync(emitted_host + (size_t)b * depth1, c->emitted, depth1 * sizeof(int32_t), cudaMemcpyDeviceToHost, c->stream) != cudaSuccess)
            rc = fail(c, MEDUSA_ERR_CUDA, "copy of the emitted tokens failed");
        if (n_emitted_host &&
            cudaMemcpyAsync(n_emitted_host + b, st + ST_N_EMITTED, sizeof(int32_t), cudaMemcpyDeviceToHost, c->stream) != cudaSuccess)
            rc = fail(c, MEDUSA_ERR_CUDA, "copy of the emitted count failed");
    }
    return rc;
}

// ============================================================================ training of the heads (Sec. 2.2.1, Eq. 1)

// Positions per chunk: the contraction length of the two gradient projections, whose results (V x d and d x d floats)
// are written once per chunk -- 1024 positions make them compute-bound instead of store-bound; a shorter batch takes
// the next multiple of 256 (four token tiles, one weight stream with a single plane).
static constexpr int TRAIN_ROWS_MAX = 1024;

// One projection over T token rows of a split activation (its map covers [2 * x_rows][K]) against a streamed operand of
// Nw rows: launches of up to 256 rows (one plane) or 128 rows (two planes), all with the same plan; every launch is
// fully serialised behind the kernel before it, because the streamed operand may have been written by that kernel.
static int32_t train_gemm(medusa_ctx *c, const TensorMap *mapX, int x_rows, const TensorMap *mapW, int Nw, int K, float *P,
                          size_t plane_stride, int ldy, int T, bool whole_tiles, int planes, PlaneDesc *pd, int out_t = 0)
{
    const int RT = gemm_tc_row_tiles(T, planes), rows_per_launch = RT * TREE_ROWS;
    *pd = gemm_tc_plan(1, Nw, K, whole_tiles, (long long)plane_stride, 0, RT, planes);
    if (!whole_tiles && (size_t)pd->n_max > c->train.part_planes)
        return fail(c, MEDUSA_ERR_SHAPE, "training projection needs %d partial planes, the workspace holds %zu", pd->n_max, c->train.part_planes);
    const TensorMap *maps[3] = {mapW, mapW, mapW};
    for (int r0 = 0; r0 < T; r0 += rows_per_launch) {
        const int Tt = T - r0 < rows_per_launch ? T - r0 : rows_per_launch;
        cudaError_t e = cudaSuccess;
        // out_t: the result goes transposed to P[n * ldy + token] (stored, or accumulated with out_t == 2)
        PROF(c, PC_GEMM, 1, e = launch_gemm_tc(mapX, maps, 1, Nw, K, *pd, out_t ? P + r0 : P + (size_t)r0 * ldy, ldy, Tt, 0,
                                               c->d_state + ST_STATUS, c->stream, 0, c->spin_limit, 0, r0, x_rows + r0, RT, planes, true,
                                               out_t, ldy));
        if (e != cudaSuccess) return fail(c, MEDUSA_ERR_CUDA, "training projection launch failed: %s", cudaGetErrorString(e));
    }
    return MEDUSA_OK;
}

static int32_t train_weight_maps(medusa_ctx *c)
{
    medusa_ctx::TrainWs &w = c->train;
    if (w.w1_of == c->w.medusa_w1 && w.w2_of == c->w.medusa_w2) return MEDUSA_OK;
    const size_t d = c->m.d, V = c->m.vocab, K = c->m.n_medusa;
    w.mW1.resize(K);
    w.mW2.resize(K);
    for (size_t k = 0; k < K; ++k)
        if (!make_weight_map(&w.mW1[k], (const char *)c->w.medusa_w1 + k * d * d * 2, (int)d, (int)d) ||
            !make_weight_map(&w.mW2[k], (const char *)c->w.medusa_w2 + k * V * d * 2, (int)V, (int)d))
            return fail(c, MEDUSA_ERR_CUDA, "training workspace: tensor map encoding failed");
    w.w1_of = c->w.medusa_w1;
    w.w2_of = c->w.medusa_w2;
    return MEDUSA_OK;
}

// maps of the chunk buffers for chunks of R positions (R is the K extent of the transposed buffers)
static int32_t train_chunk_maps(medusa_ctx *c, int R)
{
    medusa_ctx::TrainWs &w = c->train;
    if (w.R == R) return MEDUSA_OK;
    const int d = c->m.d, V = c->m.vocab;
    const bool ok = make_act_map(&w.mHp, w.Hp, d, R) && make_act_map(&w.mHT, w.HT, R, d) && make_act_map(&w.mH1p, w.H1p, d, R) &&
                    make_act_map(&w.mH1T, w.H1T, R, d) && make_act_map(&w.mdZp, w.dZp, V, R) && make_weight_map(&w.mdZT, w.dZT, V, R) &&
                    make_weight_map(&w.mW2T, w.W2T, d, V) && make_weight_map(&w.mdAT, w.dAT, d, R);
    if (!ok) return fail(c, MEDUSA_ERR_CUDA, "training workspace: tensor map encoding failed");
    w.R = R;
    return MEDUSA_OK;
}

static int32_t train_workspace(medusa_ctx *c)
{
    medusa_ctx::TrainWs &w = c->train;
    TRY(train_weight_maps(c));  // the heads' weights may have been registered anew since the last call
    if (w.ready) return MEDUSA_OK;
    const medusa_model_desc &m = c->m;
    const size_t d = m.d, V = m.vocab, R = TRAIN_ROWS_MAX, K = m.n_medusa;
    TRY(dev_alloc_bytes(c, &w.Hp, 2 * R * d * 2));
    TRY(dev_alloc_bytes(c, &w.HT, 2 * d * R * 2));
    TRY(dev_alloc_bytes(c, &w.H1p, 2 * R * d * 2));
    TRY(dev_alloc_bytes(c, &w.H1T, 2 * d * R * 2));
    TRY(dev_alloc(c, &w.A, R * d));
    TRY(dev_alloc(c, &w.Z, R * V));
    TRY(dev_alloc_bytes(c, &w.dZp, 2 * R * V * 2));
    TRY(dev_alloc_bytes(c, &w.dZT, V * R * 2));
    TRY(dev_alloc_bytes(c, &w.W2T, d * V * 2));
    TRY(dev_alloc_bytes(c, &w.dA, R * d * 2));
    TRY(dev_alloc_bytes(c, &w.dAT, d * R * 2));
    TRY(dev_alloc(c, &w.row_loss, R));
    TRY(dev_alloc(c, &w.n_valid, K));
    // the two projections whose output has only d columns (32 tiles at d = 4096) are cut stream-K over all CTAs
    const PlaneDesc p1 = gemm_tc_plan(1, (int)d, (int)d, false, (long long)(R * d), 0, 4, 1);
    const PlaneDesc p4 = gemm_tc_plan(1, (int)d, (int)V, false, (long long)(R * d), 0, 2, 2);
    w.part_planes = (size_t)(p1.n_max > p4.n_max ? p1.n_max : p4.n_max);
    TRY(dev_alloc(c, &w.part, w.part_planes * R * d));
    w.ready = true;
    return MEDUSA_OK;
}

extern "C" int32_t medusa_heads_loss_and_grads(medusa_ctx *c, const void *hidden, const int32_t *labels, int32_t N,
                                               const float *lambda_host, float *loss, float *grad_w1, float *grad_w2)
{
    TRY(check_ready(c, false, true));
    if (!hidden || !labels || !loss || !grad_w1 || !grad_w2 || N < 1)
        return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_heads_loss_and_grads: null pointer or no positions");
    const medusa_model_desc &m = c->m;
    const int d = m.d, V = m.vocab, K = m.n_medusa;
    const int R = N >= TRAIN_ROWS_MAX ? TRAIN_ROWS_MAX : ((N + 255) / 256) * 256;  // positions per chunk
    if (!c->use_tc || K < 1 || d % 256 != 0 || V % 128 != 0 || !c->w.medusa_w1 || !c->w.medusa_w2)
        return fail(c, MEDUSA_ERR_SHAPE, "medusa_heads_loss_and_grads: needs a bf16 context with heads, d a multiple of 256 and V a multiple of 128");
    if (!aligned16(hidden) || !aligned16(grad_w1) || !aligned16(grad_w2))
        return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_heads_loss_and_grads: tensors must be 16-byte aligned");
    MEDUSA_CUDA(c, cudaSetDevice(c->device));
    TRY(train_workspace(c));
    TRY(train_chunk_maps(c, R));
    medusa_ctx::TrainWs &w = c->train;
    cudaStream_t s = c->stream;
    const size_t dd = (size_t)d * d, Vd = (size_t)V * d, Rd = (size_t)R * d, RV = (size_t)R * V;
    MEDUSA_CUDA(c, cudaMemsetAsync(loss, 0, (size_t)(K + 1) * sizeof(float), s));
    PROF(c, PC_ELEMWISE, 1, launch_count_valid(labels, K, N, w.n_valid, s));
    for (int k = 0; k < K; ++k) {
        const float lambda = lambda_host ? lambda_host[k] : (float)pow(0.8, (double)(k + 1));
        // W2_k^T, the streamed operand of dh1 = dz W2_k
        PROF(c, PC_ELEMWISE, 1, launch_transpose_bf16((const char *)c->w.medusa_w2 + (size_t)k * Vd * 2, V, d, d, w.W2T, V, s));
        for (int n0 = 0; n0 < N; n0 += R) {
            const int rows = N - n0 < R ? N - n0 : R;
            // this chunk's hidden states (rows beyond the chunk are zero: they contribute nothing to any sum over positions)
            MEDUSA_CUDA(c, cudaMemcpyAsync(w.Hp, (const char *)hidden + (size_t)n0 * d * 2, (size_t)rows * d * 2, cudaMemcpyDeviceToDevice, s));
            if (rows < R)
                MEDUSA_CUDA(c, cudaMemsetAsync((char *)w.Hp + (size_t)rows * d * 2, 0, (size_t)(R - rows) * d * 2, s));
            PROF(c, PC_ELEMWISE, 1, launch_transpose_bf16(w.Hp, R, d, d, w.HT, R, s));
            PlaneDesc pd{};
            // a = W1_k h   (h is exactly bf16: one plane)
            TRY(train_gemm(c, &w.mHp, R, &w.mW1[k], d, d, w.part, Rd, d, R, false, 1, &pd));
            PROF(c, PC_ELEMWISE, 1, launch_head_hidden_fwd(w.part, pd, w.Hp, w.A, w.H1p, (char *)w.H1p + Rd * 2, R, d, s));
            PROF(c, PC_ELEMWISE, 1, launch_transpose_bf16(w.H1p, R, d, d, w.H1T, R, s));
            // z = W2_k h1   (every CTA owns whole tiles: one plane, written straight into the logits buffer)
            TRY(train_gemm(c, &w.mH1p, R, &w.mW2[k], V, d, w.Z, 0, V, R, true, 2, &pd));
            PROF(c, PC_ELEMWISE, 1, launch_ce_grad(w.Z, V, labels + (size_t)k * N + n0, R, rows, w.n_valid + k, lambda, w.row_loss, w.dZp,
                                                   (char *)w.dZp + RV * 2, s));
            PROF(c, PC_ELEMWISE, 1, launch_loss_accumulate(w.row_loss, R, w.n_valid + k, lambda, loss + k, loss + K, s));
            PROF(c, PC_ELEMWISE, 1, launch_transpose_bf16(w.dZp, R, V, V, w.dZT, R, s));
            // gW2_k^T [d][V] = h1^T (d token rows) x dz^T (V streamed rows, K = the chunk's positions)
            // (stored transposed by the projection's epilogue: straight into, or onto, gW2_k [V][d])
            TRY(train_gemm(c, &w.mH1T, d, &w.mdZT, V, R, grad_w2 + (size_t)k * Vd, 0, d, d, true, 1, &pd, n0 > 0 ? 2 : 1));
            // dh1 = dz W2_k
            TRY(train_gemm(c, &w.mdZp, R, &w.mW2T, d, V, w.part, Rd, d, R, false, 2, &pd));
            PROF(c, PC_ELEMWISE, 1, launch_head_hidden_bwd(w.part, pd, w.A, w.dA, R, d, s));
            PROF(c, PC_ELEMWISE, 1, launch_transpose_bf16(w.dA, R, d, d, w.dAT, R, s));
            // gW1_k^T [d][d] = h^T (d token rows) x da^T (d streamed rows)
            TRY(train_gemm(c, &w.mHT, d, &w.mdAT, d, R, grad_w1 + (size_t)k * dd, 0, d, d, true, 1, &pd, n0 > 0 ? 2 : 1));
        }
    }
    MEDUSA_LAUNCH_CHECK(c);
    return MEDUSA_OK;
}

extern "C" int32_t medusa_generate(medusa_ctx *c, const int32_t *prompt_host, int32_t n_prompt, int32_t G,
                                   const medusa_accept_params *params, const float *gumbel_host,
                                   int32_t *out_tokens_host, int32_t *emitted_per_step_host, int32_t *steps_host)
{
    TRY(check_ready(c, true, true));
    if (!prompt_host || n_prompt < 1 || G < 0 || !params || !out_tokens_host)
        return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_generate: bad arguments");
    const medusa_model_desc &m = c->m;
    MEDUSA_CUDA(c, cudaSetDevice(c->device));
    TRY(medusa_reset(c));
    int32_t *pd = nullptr;
    MEDUSA_CUDA(c, cudaMalloc((void **)&pd, (size_t)n_prompt * sizeof(int32_t)));
    cudaError_t e = cudaMemcpyAsync(pd, prompt_host, (size_t)n_prompt * sizeof(int32_t), cudaMemcpyHostToDevice, c->stream);
    int32_t rc = e == cudaSuccess ? prefill_dev(c, pd, n_prompt, 0) : MEDUSA_ERR_CUDA;
    cudaStreamSynchronize(c->stream);
    cudaFree(pd);
    if (rc != MEDUSA_OK) return rc;
    int32_t L = n_prompt, n_out = 0, steps = 0;
    if (!known_mode(params->mode) || (params->mode == MEDUSA_REJECTION && (!gumbel_host || !(params->temperature > 0.f))))
        return fail(c, MEDUSA_ERR_INVALID_ARG, "medusa_generate: unknown mode, or rejection sampling without noise rows or with temperature <= 0");
    const bool sample = gumbel_host && mode_reads_noise(params) && params->temperature > 0.f;
    const size_t nf = noise_floats(c, params->mode);
    while (n_out < G) {
        int32_t budget = G - n_out < m.L_max - L ? G - n_out : m.L_max - L;
        if (budget <= 0) break;
        if (sample)
            MEDUSA_CUDA(c, cudaMemcpyAsync(c->gumbel_dev, gumbel_host + (size_t)steps * nf, nf * sizeof(float),
                                           cudaMemcpyHostToDevice, c->stream));
        TRY(medusa_decode_step(c, params, sample ? c->gumbel_dev : nullptr, budget, c->pinned, c->pinned + TREE_ROWS));
        MEDUSA_CUDA(c, cudaStreamSynchronize(c->stream));
        const int32_t n = c->pinned[TREE_ROWS];
        if (n <= 0) return fail(c, MEDUSA_ERR_CACHE_FULL, "decode step emitted nothing (device status set)");
        for (int j = 0; j < n; ++j) out_tokens_host[n_out++] = c->pinned[j];
        if (emitted_per_step_host) emitted_per_step_host[steps] = n;
        L += n;
        c->L_upper = L;
        c->L_lower = L;
        ++steps;
    }
    if (steps_host) *steps_host = steps;
    return MEDUSA_OK;
}
