// Medusa heads (paper Sec. 2.1.1): x_k = h + SiLU(W1_k h), z_k = W2_k x_k, then the top-s_k tokens of every
// head and the candidate tokens of the static tree (Sec. 2.1.2).  At batch 1 both products are matrix-vector
// products that read each weight once (about 1 flop per byte), so they are pure HBM streaming: a warp owns
// four weight rows at a time, every lane issues independent 16-byte loads, the input vector sits in shared
// memory as float, and sums are formed in a fixed order (lane-strided, then an xor-shuffle tree).
#include "common.cuh"
#include "pdl.cuh"
#include "kernels.h"

namespace medusa {

constexpr int GV_WARPS = 8, GV_ROWS = 4;  // rows per warp pass; a block covers 32 consecutive rows

enum { GV_LOGITS = 0, GV_RESBLOCK = 1 };

// NR weight rows [row, row + NR) of one head against the input vector in shared memory: every lane issues NR
// independent 16-byte loads per step; sums in a fixed order (lane-strided, then an xor-shuffle tree), so a row's
// result does not depend on how rows are grouped.
template <typename WT, int EPI, int NR>
__device__ __forceinline__ void gemv_rows(const WT *__restrict__ Wh, const float *__restrict__ xs, float *__restrict__ out_h,
                                          int row, int d, int lane)
{
    constexpr int VN = Vec16<WT>::N;
    float acc[NR];
#pragma unroll
    for (int r = 0; r < NR; ++r)
        acc[r] = 0.f;
    const WT *w0 = Wh + (size_t)row * d;
    const int chunks = d / VN;
    for (int c = lane; c < chunks; c += 32) {
        float wv[NR][VN];
#pragma unroll
        for (int r = 0; r < NR; ++r)
            Vec16<WT>::load(w0 + (size_t)r * d + (size_t)c * VN, wv[r]);
        float xv[VN];
#pragma unroll
        for (int e = 0; e < VN; e += 4) {
            float4 t = *reinterpret_cast<const float4 *>(xs + c * VN + e);
            xv[e] = t.x; xv[e + 1] = t.y; xv[e + 2] = t.z; xv[e + 3] = t.w;
        }
#pragma unroll
        for (int r = 0; r < NR; ++r)
#pragma unroll
            for (int e = 0; e < VN; ++e)
                acc[r] = fmaf(wv[r][e], xv[e], acc[r]);
    }
#pragma unroll
    for (int r = 0; r < NR; ++r)
        acc[r] = warp_sum(acc[r]);
    if (lane < NR) {
        float y = acc[0];
#pragma unroll
        for (int r = 1; r < NR; ++r)
            if (lane == r)
                y = acc[r];
        out_h[row + lane] = EPI == GV_LOGITS ? y : xs[row + lane] + silu_f(y);
    }
}

// grid (blocks per head, heads).  The rows of a head are dealt out evenly to all the warps of the head's blocks
// (contiguous ranges that differ by at most one row), so that a grid sized to what is resident at once finishes
// together instead of in a last, partly filled wave; a warp walks its range four rows at a time, then two, then one.
// XT: type of the input vector (float inside the decode step, the model dtype at the public entry point)
template <typename WT, typename XT, int EPI>
__global__ void __launch_bounds__(GV_WARPS * 32)
gemv_kernel(const WT *__restrict__ W, const XT *__restrict__ x, int x_head_stride, float *__restrict__ out, int rows, int d)
{
    pdl_enter();
    extern __shared__ float xs[];  // [d]
    const int head = blockIdx.y;
    const XT *xh = x + (size_t)head * x_head_stride;
    for (int i = threadIdx.x; i < d; i += blockDim.x)
        xs[i] = to_f32(xh[i]);
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long w = (long long)blockIdx.x * GV_WARPS + warp, n_warps = (long long)gridDim.x * GV_WARPS;
    int row = (int)(w * rows / n_warps);
    const int row_end = (int)((w + 1) * rows / n_warps);
    const WT *Wh = W + (size_t)head * rows * d;
    float *out_h = out + (size_t)head * rows;
    for (; row + 4 <= row_end; row += 4)
        gemv_rows<WT, EPI, 4>(Wh, xs, out_h, row, d, lane);
    if (row + 2 <= row_end) {
        gemv_rows<WT, EPI, 2>(Wh, xs, out_h, row, d, lane);
        row += 2;
    }
    if (row < row_end)
        gemv_rows<WT, EPI, 1>(Wh, xs, out_h, row, d, lane);
}

// blocks per head: one per 32 rows, but no more than are resident at once over all heads
template <typename Kernel>
static int gemv_blocks_per_head(Kernel kernel, size_t smem, int rows, int K)
{
    int sms = 0, per_sm = 0, dev = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        sms = 148;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, GV_WARPS * 32, smem) != cudaSuccess || per_sm <= 0)
        per_sm = 4;
    const int want = (rows + GV_WARPS * GV_ROWS - 1) / (GV_WARPS * GV_ROWS);
    int cap = sms * per_sm / (K > 0 ? K : 1);
    if (cap < 1) cap = 1;
    return want < cap ? want : cap;
}

template <typename WT, typename XT, int EPI>
static void launch_gemv(const WT *W, const XT *x, int x_head_stride, float *out, int rows, int d, int K, cudaStream_t s)
{
    const size_t smem = (size_t)d * sizeof(float);
    static int blocks = 0, blocks_rows = -1, blocks_K = -1;  // (the occupancy query is not free: once per shape)
    static size_t blocks_smem = 0;
    if (rows != blocks_rows || K != blocks_K || smem != blocks_smem) {
        blocks = gemv_blocks_per_head(gemv_kernel<WT, XT, EPI>, smem, rows, K);
        blocks_rows = rows; blocks_K = K; blocks_smem = smem;
    }
    launch_pdl(gemv_kernel<WT, XT, EPI>, dim3(blocks, K), dim3(GV_WARPS * 32), smem, s, W, x, x_head_stride, out, rows, d);
}

// ---------------------------------------------------------------------------------------- batched GEMV (batch > 1)
// The same products for up to GVB_MAX sequences at once: every weight row is loaded once and multiplied with all the
// sequences' input vectors (held side by side in shared memory), so a batched step streams the head weights once.
// Sums per (row, sequence) are formed in the same order as in the single-sequence kernel.
constexpr int GVB_MAX = 4;

template <typename WT, int EPI, int NR>
__device__ __forceinline__ void gemv_rows_batch(const WT *__restrict__ Wh, const float *__restrict__ xs, float *__restrict__ out_h,
                                                long long out_batch_stride, int row, int d, int nb, int lane)
{
    constexpr int VN = Vec16<WT>::N;
    float acc[NR][GVB_MAX];
#pragma unroll
    for (int r = 0; r < NR; ++r)
#pragma unroll
        for (int b = 0; b < GVB_MAX; ++b)
            acc[r][b] = 0.f;
    const WT *w0 = Wh + (size_t)row * d;
    const int chunks = d / VN;
    for (int c = lane; c < chunks; c += 32) {
        float wv[NR][VN];
#pragma unroll
        for (int r = 0; r < NR; ++r)
            Vec16<WT>::load(w0 + (size_t)r * d + (size_t)c * VN, wv[r]);
#pragma unroll
        for (int b = 0; b < GVB_MAX; ++b) {
            if (b < nb) {
                float xv[VN];
#pragma unroll
                for (int e = 0; e < VN; e += 4) {
                    float4 t = *reinterpret_cast<const float4 *>(xs + (size_t)b * d + c * VN + e);
                    xv[e] = t.x; xv[e + 1] = t.y; xv[e + 2] = t.z; xv[e + 3] = t.w;
                }
#pragma unroll
                for (int r = 0; r < NR; ++r)
#pragma unroll
                    for (int e = 0; e < VN; ++e)
                        acc[r][b] = fmaf(wv[r][e], xv[e], acc[r][b]);
            }
        }
    }
#pragma unroll
    for (int b = 0; b < GVB_MAX; ++b) {
        if (b < nb) {
#pragma unroll
            for (int r = 0; r < NR; ++r)
                acc[r][b] = warp_sum(acc[r][b]);
            if (lane < NR) {
                float y = acc[0][b];
#pragma unroll
                for (int r = 1; r < NR; ++r)
                    if (lane == r)
                        y = acc[r][b];
                out_h[(size_t)b * out_batch_stride + row + lane] = EPI == GV_LOGITS ? y : xs[(size_t)b * d + row + lane] + silu_f(y);
            }
        }
    }
}

// x: float, sequence b's vector of head k at x + b * x_batch_stride + k * x_head_stride; out[b][k][rows] with
// out_batch_stride floats between sequences
template <typename WT, int EPI>
__global__ void __launch_bounds__(GV_WARPS * 32)
gemv_batch_kernel(const WT *__restrict__ W, const float *__restrict__ x, int x_head_stride, long long x_batch_stride,
                  float *__restrict__ out, long long out_batch_stride, int rows, int d, int nb)
{
    pdl_enter();
    extern __shared__ float xs[];  // [nb][d]
    const int head = blockIdx.y;
    for (int b = 0; b < nb; ++b) {
        const float *xh = x + (size_t)b * x_batch_stride + (size_t)head * x_head_stride;
        for (int i = threadIdx.x; i < d; i += blockDim.x)
            xs[(size_t)b * d + i] = xh[i];
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long w = (long long)blockIdx.x * GV_WARPS + warp, n_warps = (long long)gridDim.x * GV_WARPS;
    int row = (int)(w * rows / n_warps);
    const int row_end = (int)((w + 1) * rows / n_warps);
    const WT *Wh = W + (size_t)head * rows * d;
    float *out_h = out + (size_t)head * rows;
    for (; row + 2 <= row_end; row += 2)
        gemv_rows_batch<WT, EPI, 2>(Wh, xs, out_h, out_batch_stride, row, d, nb, lane);
    if (row < row_end)
        gemv_rows_batch<WT, EPI, 1>(Wh, xs, out_h, out_batch_stride, row, d, nb, lane);
}

template <typename WT, int EPI>
static cudaError_t launch_gemv_batch(const WT *W, const float *x, int x_head_stride, long long x_batch_stride, float *out,
                                     long long out_batch_stride, int rows, int d, int K, int nb, cudaStream_t s)
{
    const size_t smem = (size_t)nb * d * sizeof(float);
    static bool attr[64] = {};
    if (first_use_on_current_device(attr)) {
        cudaError_t e = cudaFuncSetAttribute(gemv_batch_kernel<WT, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess)
            return e;
    }
    const int blocks = gemv_blocks_per_head(gemv_batch_kernel<WT, EPI>, smem, rows, K);
    return launch_pdl(gemv_batch_kernel<WT, EPI>, dim3(blocks, K), dim3(GV_WARPS * 32), smem, s, W, x, x_head_stride, x_batch_stride,
                      out, out_batch_stride, rows, d, nb);
}

// h_all: float [nb][d] (h_stride floats apart); x_all: float out, sequence b's [K][d] block x_stride floats after b-1's
cudaError_t launch_heads_resblock_batch(int dtype, const float *h_all, long long h_stride, const void *W1, float *x_all,
                                        long long x_stride, int K, int d, int nb, cudaStream_t s)
{
    if (nb < 1 || nb > GVB_MAX)
        return cudaErrorInvalidValue;
    if (dtype == MEDUSA_BF16)
        return launch_gemv_batch<bf16, GV_RESBLOCK>((const bf16 *)W1, h_all, 0, h_stride, x_all, x_stride, d, d, K, nb, s);
    return launch_gemv_batch<float, GV_RESBLOCK>((const float *)W1, h_all, 0, h_stride, x_all, x_stride, d, d, K, nb, s);
}

// x_all as above; logits_all: float out, sequence b's [K][V] block z_stride floats after b-1's
cudaError_t launch_heads_vocab_batch(int dtype, const float *x_all, long long x_stride, const void *W2, float *logits_all,
                                     long long z_stride, int K, int d, int V, int nb, cudaStream_t s)
{
    if (nb < 1 || nb > GVB_MAX)
        return cudaErrorInvalidValue;
    if (dtype == MEDUSA_BF16)
        return launch_gemv_batch<bf16, GV_LOGITS>((const bf16 *)W2, x_all, d, x_stride, logits_all, z_stride, V, d, K, nb, s);
    return launch_gemv_batch<float, GV_LOGITS>((const float *)W2, x_all, d, x_stride, logits_all, z_stride, V, d, K, nb, s);
}

void launch_heads_resblock(int dtype, const void *h, int h_is_f32, const void *W1, float *x, int K, int d, cudaStream_t s)
{
    if (dtype == MEDUSA_BF16 && !h_is_f32)
        launch_gemv<bf16, bf16, GV_RESBLOCK>((const bf16 *)W1, (const bf16 *)h, 0, x, d, d, K, s);
    else if (dtype == MEDUSA_BF16)
        launch_gemv<bf16, float, GV_RESBLOCK>((const bf16 *)W1, (const float *)h, 0, x, d, d, K, s);
    else
        launch_gemv<float, float, GV_RESBLOCK>((const float *)W1, (const float *)h, 0, x, d, d, K, s);
}

void launch_heads_vocab(int dtype, const float *x, const void *W2, float *logits, int K, int d, int V, cudaStream_t s)
{
    if (dtype == MEDUSA_BF16)
        launch_gemv<bf16, float, GV_LOGITS>((const bf16 *)W2, x, d, logits, V, d, K, s);
    else
        launch_gemv<float, float, GV_LOGITS>((const float *)W2, x, d, logits, V, d, K, s);
}

// ---------------------------------------------------------------------------------------- top-k
// Order: value descending, then index ascending.  One block per head; pass r picks the best element not
// picked by passes 0..r-1.  Compares only, so the result is exact for any finite input.
__device__ __forceinline__ bool better(float v, int i, float bv, int bi)
{
    return v > bv || (v == bv && i < bi);
}

constexpr int TOPK_LOCAL = 8;    // per-thread candidate list of the single-pass kernel
constexpr int TOPK_SLICES = 16;  // blocks per row in the first of the two stages
constexpr int TOPK_NONE = 0x7fffffff;  // index of "no candidate": loses every comparison

// Single pass over elements [e0, e1) of row blockIdx.x: every thread keeps the best `topk` of its own elements
// (sorted), then the block pops the best `topk` times from the heads of those lists.
// Stage 1 (INDIRECT = false): grid (rows, slices); block (row, slice) scans its slice of the logits and writes its
// `topk` best as (value, index) candidates.  Stage 2 (INDIRECT = true): grid (rows); the block scans the row's
// slices * topk candidates, whose indices come from `src_idx`, and writes the final result, replacing "no
// candidate" (fewer than topk comparable values in the row: NaN logits) by the rank itself, a valid index.
template <bool INDIRECT>
__global__ void __launch_bounds__(256)
topk_stage_kernel(const float *__restrict__ vals, const int32_t *__restrict__ src_idx, int n, int topk,
                  int32_t *__restrict__ idx, float *__restrict__ val)
{
    pdl_enter();
    __shared__ float sv[8];
    __shared__ int si[8];
    __shared__ int s_win;
    const int slices = gridDim.y, slice = blockIdx.y;
    const int chunk = (((n + slices - 1) / slices) + 3) & ~3;  // multiple of 4: slices keep the row's alignment
    const int e0 = min(n, slice * chunk), e1 = min(n, e0 + chunk);
    const float *z = vals + (size_t)blockIdx.x * n;
    const int32_t *zi = INDIRECT ? src_idx + (size_t)blockIdx.x * n : nullptr;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float lv[TOPK_LOCAL];
    int li[TOPK_LOCAL];
#pragma unroll
    for (int k = 0; k < TOPK_LOCAL; ++k) {
        lv[k] = -INFINITY;
        li[k] = TOPK_NONE;
    }
    auto push = [&](float v, int i) {
        if (!better(v, i, lv[TOPK_LOCAL - 1], li[TOPK_LOCAL - 1]))
            return;
        lv[TOPK_LOCAL - 1] = v;
        li[TOPK_LOCAL - 1] = i;
#pragma unroll
        for (int k = TOPK_LOCAL - 1; k > 0; --k) {  // one bubble step per slot keeps the list sorted
            if (better(lv[k], li[k], lv[k - 1], li[k - 1])) {
                float tv = lv[k]; lv[k] = lv[k - 1]; lv[k - 1] = tv;
                int ti = li[k]; li[k] = li[k - 1]; li[k - 1] = ti;
            }
        }
    };
    if (!INDIRECT && (n & 3) == 0 && (reinterpret_cast<uintptr_t>(z) & 15u) == 0) {
        const float4 *z4 = reinterpret_cast<const float4 *>(z);
        const int c_end = e1 >> 2;
        for (int c = (e0 >> 2) + threadIdx.x; c < c_end; c += blockDim.x * 2) {
            const int c1 = c + blockDim.x;
            float4 a = z4[c], b = c1 < c_end ? z4[c1] : make_float4(0.f, 0.f, 0.f, 0.f);
            push(a.x, 4 * c); push(a.y, 4 * c + 1); push(a.z, 4 * c + 2); push(a.w, 4 * c + 3);
            if (c1 < c_end) { push(b.x, 4 * c1); push(b.y, 4 * c1 + 1); push(b.z, 4 * c1 + 2); push(b.w, 4 * c1 + 3); }
        }
    } else {
        for (int i = e0 + threadIdx.x; i < e1; i += blockDim.x)
            push(z[i], INDIRECT ? zi[i] : i);
    }
    const size_t out0 = ((size_t)blockIdx.x * slices + slice) * topk;
    int head = 0;  // next unpopped entry of this thread's list
    for (int r = 0; r < topk; ++r) {
        float bv = -INFINITY;
        int bi = TOPK_NONE;
#pragma unroll
        for (int k = 0; k < TOPK_LOCAL; ++k)
            if (k == head) { bv = lv[k]; bi = li[k]; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
        }
        if (lane == 0) { sv[warp] = bv; si[warp] = bi; }
        __syncthreads();
        if (warp == 0) {
            bv = lane < (blockDim.x >> 5) ? sv[lane] : -INFINITY;
            bi = lane < (blockDim.x >> 5) ? si[lane] : TOPK_NONE;
#pragma unroll
            for (int o = 4; o > 0; o >>= 1) {  // at most eight warps
                float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
            }
            if (lane == 0) {
                s_win = bi;
                if (INDIRECT && bi == TOPK_NONE) bi = r;
                idx[out0 + r] = bi;
                if (val)
                    val[out0 + r] = bv;
            }
        }
        __syncthreads();
        // the thread that owned the winner moves on to its next candidate
        bool mine = false;
#pragma unroll
        for (int k = 0; k < TOPK_LOCAL; ++k)
            if (k == head && li[k] == s_win && s_win != TOPK_NONE) mine = true;
        if (mine) ++head;
        __syncthreads();
    }
}

// General fallback (topk > TOPK_LOCAL): pass r picks the best element not picked by passes 0..r-1.
__global__ void __launch_bounds__(1024)
topk_multipass_kernel(const float *__restrict__ logits, int V, int topk, int32_t *__restrict__ idx, float *__restrict__ val)
{
    pdl_enter();
    __shared__ float sv[32];
    __shared__ int si[32];
    __shared__ int chosen[MAX_T];
    const float *z = logits + (size_t)blockIdx.x * V;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int r = 0; r < topk; ++r) {
        float bv = -INFINITY;
        int bi = 0x7fffffff;
        for (int i = threadIdx.x; i < V; i += blockDim.x) {
            bool taken = false;
            for (int c = 0; c < r; ++c)
                taken |= (chosen[c] == i);
            float v = z[i];
            if (!taken && better(v, i, bv, bi)) { bv = v; bi = i; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
        }
        if (lane == 0) { sv[warp] = bv; si[warp] = bi; }
        __syncthreads();
        if (warp == 0) {
            bv = lane < (blockDim.x >> 5) ? sv[lane] : -INFINITY;
            bi = lane < (blockDim.x >> 5) ? si[lane] : 0x7fffffff;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
            }
            if (lane == 0) {
                if (bi == 0x7fffffff) bi = r;
                chosen[r] = bi;
                idx[(size_t)blockIdx.x * topk + r] = bi;
                if (val)
                    val[(size_t)blockIdx.x * topk + r] = bv;
            }
        }
        __syncthreads();
    }
}

size_t topk_scratch_bytes(int K) { return (size_t)K * TOPK_SLICES * TOPK_LOCAL * (sizeof(float) + sizeof(int32_t)); }

void launch_topk(const float *logits, int K, int V, int topk, int32_t *idx, float *val, void *scratch, cudaStream_t s)
{
    if (K <= 0 || topk <= 0)
        return;
    if (topk <= TOPK_LOCAL && scratch) {
        // candidates of the row's slices: values [K][slices * topk], then their indices
        float *cv = (float *)scratch;
        int32_t *ci = (int32_t *)(cv + (size_t)K * TOPK_SLICES * TOPK_LOCAL);
        launch_pdl(topk_stage_kernel<false>, dim3(K, TOPK_SLICES), dim3(256), 0, s, logits, (const int32_t *)nullptr, V, topk, ci, cv);
        launch_pdl(topk_stage_kernel<true>, dim3(K, 1), dim3(128), 0, s, (const float *)cv, (const int32_t *)ci, TOPK_SLICES * topk, topk,
                   idx, val);
    } else {
        launch_pdl(topk_multipass_kernel, dim3(K), dim3(1024), 0, s, logits, V, topk, idx, val);
    }
}

// tree_tok[i] = pool[tree_idx[i]], pool = [root, head-1 top-k, head-2 top-k, ...]
__global__ void expand_kernel(const int32_t *root, const int32_t *topk_idx, const int32_t *tree_idx, int32_t *tree_tok,
                              int T)
{
    pdl_enter();
    int i = threadIdx.x;
    if (i < T) {
        int p = tree_idx[i];
        tree_tok[i] = p == 0 ? *root : topk_idx[p - 1];
    }
}

void launch_expand(const int32_t *root, const int32_t *topk_idx, const int32_t *tree_idx, int32_t *tree_tok, int T,
                   cudaStream_t s)
{
    launch_pdl(expand_kernel, dim3(1), dim3(MAX_T), 0, s, root, topk_idx, tree_idx, tree_tok, T);
}

}  // namespace medusa
