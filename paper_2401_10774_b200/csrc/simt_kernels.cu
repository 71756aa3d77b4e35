// CUDA-core kernels that work for any shape and both element types.  The fp32 model runs entirely on
// these (tensor cores have no true-fp32 mode); the bf16 model uses them for the element-wise stages.
// Every output element is produced by one thread with a fixed summation order, so results do not depend
// on how many token rows are processed together.
#include "common.cuh"
#include "pdl.cuh"
#include "kernels.h"

namespace medusa {

// ---------------------------------------------------------------------------------------- embedding
template <typename WT>
__global__ void embed_kernel(const int32_t *__restrict__ tok, const WT *__restrict__ embed, float *__restrict__ x, int d, int V)
{
    pdl_enter();
    int t = blockIdx.x;
    const int id = min(max(tok[t], 0), V - 1);  // an out-of-range id must never become an out-of-bounds read
    const WT *row = embed + (size_t)id * d;
    constexpr int VN = Vec16<WT>::N;  // d is a multiple of VN (checked at context creation)
    for (int i = threadIdx.x * VN; i < d; i += blockDim.x * VN) {
        float v[VN];
        Vec16<WT>::load(row + i, v);
#pragma unroll
        for (int e = 0; e < VN; e += 4)
            *reinterpret_cast<float4 *>(x + (size_t)t * d + i + e) = make_float4(v[e], v[e + 1], v[e + 2], v[e + 3]);
    }
}

void launch_embed(int dtype, const int32_t *tok, const void *embed, float *x, int T, int d, int V, cudaStream_t s)
{
    if (dtype == MEDUSA_BF16)
        launch_pdl(embed_kernel<bf16>, dim3(T), dim3(256), 0, s, tok, (const bf16 *)embed, x, d, V);
    else
        launch_pdl(embed_kernel<float>, dim3(T), dim3(256), 0, s, tok, (const float *)embed, x, d, V);
}

// ---------------------------------------------------------------------------------------- RMSNorm
// y_i = g_i * x_i / sqrt(mean(x^2) + eps); one block per token row; fixed-order block reduction.
// The result feeds a GEMM.  In the bf16 model it is stored as two bf16 planes, hi = bf16(y) and
// lo = bf16(y - hi), so that the tensor-core product W*hi + W*lo sees the activation to ~2^-17 relative
// instead of 2^-9: activations are tiny next to the weights, so this costs no HBM traffic.
template <typename WT> __device__ __forceinline__ void store_split(WT *hi, WT *lo, size_t i, float y);
template <> __device__ __forceinline__ void store_split<float>(float *hi, float *, size_t i, float y) { hi[i] = y; }
template <> __device__ __forceinline__ void store_split<bf16>(bf16 *hi, bf16 *lo, size_t i, float y)
{
    bf16 h = __float2bfloat16_rn(y);
    hi[i] = h;
    if (lo)
        lo[i] = __float2bfloat16_rn(y - __bfloat162float(h));
}

// If n_planes > 0 the residual stream is first advanced: x += planes[0] + planes[1] + ... (the k-split
// partial results of the preceding projection, added in plane order), and written back.
// One block per token row, 16-byte accesses, all plane loads of a chunk in flight together.
template <typename WT> __device__ __forceinline__ void store_split4(WT *hi, WT *lo, size_t i, const float *y);
template <> __device__ __forceinline__ void store_split4<float>(float *hi, float *, size_t i, const float *y)
{
    *reinterpret_cast<float4 *>(hi + i) = make_float4(y[0], y[1], y[2], y[3]);
}
template <> __device__ __forceinline__ void store_split4<bf16>(bf16 *hi, bf16 *lo, size_t i, const float *y)
{
    __nv_bfloat162 h0 = __floats2bfloat162_rn(y[0], y[1]), h1 = __floats2bfloat162_rn(y[2], y[3]);
    uint2 u;
    u.x = *reinterpret_cast<uint32_t *>(&h0);
    u.y = *reinterpret_cast<uint32_t *>(&h1);
    *reinterpret_cast<uint2 *>(hi + i) = u;
    if (lo) {
        __nv_bfloat162 l0 = __floats2bfloat162_rn(y[0] - __low2float(h0), y[1] - __high2float(h0));
        __nv_bfloat162 l1 = __floats2bfloat162_rn(y[2] - __low2float(h1), y[3] - __high2float(h1));
        u.x = *reinterpret_cast<uint32_t *>(&l0);
        u.y = *reinterpret_cast<uint32_t *>(&l1);
        *reinterpret_cast<uint2 *>(lo + i) = u;
    }
}
template <typename WT> __device__ __forceinline__ void load4(const WT *p, float *out);
template <> __device__ __forceinline__ void load4<float>(const float *p, float *out)
{
    float4 v = *reinterpret_cast<const float4 *>(p);
    out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
}
template <> __device__ __forceinline__ void load4<bf16>(const bf16 *p, float *out)
{
    uint2 u = *reinterpret_cast<const uint2 *>(p);
    out[0] = __uint_as_float(u.x << 16); out[1] = __uint_as_float(u.x & 0xffff0000u);
    out[2] = __uint_as_float(u.y << 16); out[3] = __uint_as_float(u.y & 0xffff0000u);
}

// x[i..i+4) plus the fp32 partial planes that cover column i, PLANES_IN_FLIGHT planes in flight per round and added in
// plane order; the sum is written back to x (the residual stream) and returned.
// PLANES_IN_FLIGHT: the output and the down projection of a 4096-wide model leave 9 to 10 pieces per tile (296 CTAs over
// 32 tiles); with ten loads in flight their sum takes one round trip to the L2 instead of two.
template <int PLANES_IN_FLIGHT>
__device__ __forceinline__ float4 add_planes(float *xr, const float *pr, const PlaneDesc &pd, int i)
{
    float4 v = *reinterpret_cast<const float4 *>(xr + i);
    if (pd.n_max > 0) {
        float4 add = make_float4(0.f, 0.f, 0.f, 0.f);
        const int n_planes = planes_of_col(pd, i);
        for (int p0 = 0; p0 < n_planes; p0 += PLANES_IN_FLIGHT) {
            float4 w[PLANES_IN_FLIGHT];
#pragma unroll
            for (int j = 0; j < PLANES_IN_FLIGHT; ++j)
                w[j] = *reinterpret_cast<const float4 *>(pr + (size_t)min(p0 + j, n_planes - 1) * pd.stride + i);
#pragma unroll
            for (int j = 0; j < PLANES_IN_FLIGHT; ++j)
                if (p0 + j < n_planes) {
                    add.x += w[j].x; add.y += w[j].y; add.z += w[j].z; add.w += w[j].w;
                }
        }
        v.x += add.x; v.y += add.y; v.z += add.z; v.w += add.w;
        *reinterpret_cast<float4 *>(xr + i) = v;
    }
    return v;
}

template <typename WT>
__device__ __forceinline__ void norm_store(const float4 &v, const float (&g)[4], float r, WT *out, WT *out_lo,
                                           float *out_f32, size_t at)
{
    float y[4] = {g[0] * (v.x * r), g[1] * (v.y * r), g[2] * (v.z * r), g[3] * (v.w * r)};
    store_split4<WT>(out, out_lo, at, y);
    if (out_f32)
        *reinterpret_cast<float4 *>(out_f32 + at) = make_float4(y[0], y[1], y[2], y[3]);
}

template <typename WT, int GROUPS, int MAXT>
__global__ void __launch_bounds__(MAXT)
rmsnorm_kernel(float *__restrict__ x, const float *__restrict__ planes, PlaneDesc pd,
               const WT *__restrict__ gain, float eps, WT *__restrict__ out, WT *__restrict__ out_lo,
               float *__restrict__ out_f32, int d)
{
    pdl_enter();
    __shared__ float red[32];
    const int t = blockIdx.x;
    float *xr = x + (size_t)t * d;
    const float *pr = planes + (size_t)t * d;
    float ss = 0.f;
    // Column group `it` of this thread is columns [tid*4 + it*step, +4).  The first GROUPS groups are handled by
    // fully unrolled code, so that the summed row stays in named registers for the second pass and the gains
    // are already on their way while the block reduces; wider rows fall through to the loop after them.
    const int step = blockDim.x * 4;
    float4 keep[GROUPS];
    float gn[GROUPS][4];
#pragma unroll
    for (int it = 0; it < GROUPS; ++it) {
        const int i = threadIdx.x * 4 + it * step;
        keep[it] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (i < d) {
            load4<WT>(gain + i, gn[it]);
            keep[it] = add_planes<GROUPS == 1 ? 10 : 8>(xr, pr, pd, i);
        }
        ss += keep[it].x * keep[it].x + keep[it].y * keep[it].y + keep[it].z * keep[it].z + keep[it].w * keep[it].w;
    }
    for (int i = threadIdx.x * 4 + GROUPS * step; i < d; i += step) {
        const float4 v = add_planes<GROUPS == 1 ? 10 : 8>(xr, pr, pd, i);
        ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0)
        red[threadIdx.x >> 5] = ss;
    __syncthreads();
    // every warp reduces the (at most 32) warp sums itself: one block barrier instead of two
    float tot = (threadIdx.x & 31) < (blockDim.x >> 5) ? red[threadIdx.x & 31] : 0.f;
    tot = warp_sum(tot);
    const float r = rsqrtf(tot / (float)d + eps);
#pragma unroll
    for (int it = 0; it < GROUPS; ++it) {
        const int i = threadIdx.x * 4 + it * step;
        if (i < d)
            norm_store<WT>(keep[it], gn[it], r, out, out_lo, out_f32, (size_t)t * d + i);
    }
    for (int i = threadIdx.x * 4 + GROUPS * step; i < d; i += step) {
        const float4 v = *reinterpret_cast<const float4 *>(xr + i);  // (written by this same thread above)
        float g[4];
        load4<WT>(gain + i, g);
        norm_store<WT>(v, g, r, out, out_lo, out_f32, (size_t)t * d + i);
    }
}

template <typename WT, int GROUPS, int MAXT>
static void launch_rmsnorm_as(float *x, const float *planes, const PlaneDesc &pd, const void *gain, float eps, void *out,
                              void *out_lo, float *out_f32, int T, int d, cudaStream_t s)
{
    int threads = ((d / (4 * GROUPS) + 31) / 32) * 32;
    if (threads > MAXT) threads = MAXT;
    launch_pdl(rmsnorm_kernel<WT, GROUPS, MAXT>, dim3(T), dim3(threads), 0, s, x, planes, pd, (const WT *)gain, eps,
               (WT *)out, (WT *)out_lo, out_f32, d);
}

void launch_add_rmsnorm(int dtype, float *x, const float *planes, const PlaneDesc &pd, const void *gain,
                        float eps, void *out, void *out_lo, float *out_f32, int T, int d, cudaStream_t s)
{
    // rows of up to 4096 columns: one column group per thread; wider rows: two groups per thread in blocks of at
    // most 768 threads, which leaves the compiler 80 registers for both groups' loads in flight
    if (dtype == MEDUSA_BF16) {
        if (d <= 4096) launch_rmsnorm_as<bf16, 1, 1024>(x, planes, pd, gain, eps, out, out_lo, out_f32, T, d, s);
        else launch_rmsnorm_as<bf16, 2, 768>(x, planes, pd, gain, eps, out, out_lo, out_f32, T, d, s);
    } else {
        if (d <= 4096) launch_rmsnorm_as<float, 1, 1024>(x, planes, pd, gain, eps, out, nullptr, out_f32, T, d, s);
        else launch_rmsnorm_as<float, 2, 768>(x, planes, pd, gain, eps, out, nullptr, out_f32, T, d, s);
    }
}

// ---------------------------------------------------------------------------------------- GEMM (CUDA cores)
// Y[t][col0+n] = sum_k X[t][k] W[n][k], T <= 64, X = X_hi (+ X_lo).  Block = 64 output columns x all rows,
// K staged in chunks of 32 through shared memory; thread (tx, ty) owns columns {tx, tx+32} and rows
// ty*8..ty*8+7.
constexpr int GS_BN = 64, GS_KC = 32;

template <typename WT, int MODE>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(const WT *__restrict__ X, const WT *__restrict__ Xlo, int ldx, const WT *__restrict__ W,
                 void *__restrict__ Yv, int ldy, int col0, int T, int N, int K)
{
    pdl_enter();
    __shared__ float Xs[TREE_ROWS][GS_KC + 1];
    __shared__ float Ws[GS_BN][GS_KC + 1];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int n0 = blockIdx.x * GS_BN;
    float acc[8][2];
#pragma unroll
    for (int r = 0; r < 8; ++r)
        acc[r][0] = acc[r][1] = 0.f;
    for (int k0 = 0; k0 < K; k0 += GS_KC) {
        for (int i = threadIdx.x; i < TREE_ROWS * GS_KC; i += 256) {
            int r = i / GS_KC, c = i % GS_KC;
            float v = 0.f;
            if (r < T && k0 + c < K) {
                v = to_f32(X[(size_t)r * ldx + k0 + c]);
                if (Xlo)
                    v += to_f32(Xlo[(size_t)r * ldx + k0 + c]);
            }
            Xs[r][c] = v;
        }
        for (int i = threadIdx.x; i < GS_BN * GS_KC; i += 256) {
            int r = i / GS_KC, c = i % GS_KC;
            Ws[r][c] = (n0 + r < N && k0 + c < K) ? to_f32(W[(size_t)(n0 + r) * K + k0 + c]) : 0.f;
        }
        __syncthreads();
#pragma unroll 8
        for (int k = 0; k < GS_KC; ++k) {
            float w0 = Ws[tx][k], w1 = Ws[tx + 32][k];
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                float xv = Xs[ty * 8 + r][k];
                acc[r][0] = fmaf(xv, w0, acc[r][0]);
                acc[r][1] = fmaf(xv, w1, acc[r][1]);
            }
        }
        __syncthreads();
    }
#pragma unroll
    for (int r = 0; r < 8; ++r) {
        int t = ty * 8 + r;
        if (t >= T)
            continue;
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            int n = n0 + tx + 32 * c;
            if (n >= N)
                continue;
            size_t o = (size_t)t * ldy + col0 + n;
            if (MODE == GEMM_STORE_F32)
                ((float *)Yv)[o] = acc[r][c];
            else
                ((float *)Yv)[o] += acc[r][c];
        }
    }
}

template <typename WT>
static void gemm_simt_dispatch(const void *X, const void *Xlo, int ldx, const void *W, void *Y, int ldy, int col0, int T,
                               int N, int K, GemmOut mode, cudaStream_t s)
{
    dim3 grid((N + GS_BN - 1) / GS_BN);
    if (mode == GEMM_STORE_F32)
        launch_pdl(gemm_simt_kernel<WT, GEMM_STORE_F32>, dim3(grid), dim3(256), 0, s, (const WT *)X, (const WT *)Xlo, ldx, (const WT *)W, Y, ldy, col0, T, N, K);
    else
        launch_pdl(gemm_simt_kernel<WT, GEMM_ADD_F32>, dim3(grid), dim3(256), 0, s, (const WT *)X, (const WT *)Xlo, ldx, (const WT *)W, Y, ldy, col0, T, N, K);
}

void launch_gemm_simt(int dtype, const void *X, const void *Xlo, int ldx, const void *W, void *Y, int ldy, int col0,
                      int T, int N, int K, GemmOut mode, cudaStream_t s)
{
    // the kernel covers 64 token rows: more rows run as one launch per tile of 64
    for (int r0 = 0; r0 < T; r0 += TREE_ROWS) {
        const int Tt = T - r0 < TREE_ROWS ? T - r0 : TREE_ROWS;
        if (dtype == MEDUSA_BF16)
            gemm_simt_dispatch<bf16>((const bf16 *)X + (size_t)r0 * ldx, Xlo ? (const bf16 *)Xlo + (size_t)r0 * ldx : nullptr, ldx, W,
                                     (float *)Y + (size_t)r0 * ldy, ldy, col0, Tt, N, K, mode, s);
        else
            gemm_simt_dispatch<float>((const float *)X + (size_t)r0 * ldx, nullptr, ldx, W, (float *)Y + (size_t)r0 * ldy, ldy, col0,
                                      Tt, N, K, mode, s);
    }
}

// ---------------------------------------------------------------------------------------- rotary embedding
// Angles are formed in double from the integer position so that long contexts lose no precision.
__global__ void rope_table_kernel(float2 *cs, const int32_t *cache_len, const int32_t *pos, int T, int D, float theta)
{
    pdl_enter();
    int half = D / 2;
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= T * half)
        return;
    int t = i / half, e = i % half;
    double p = (double)(*cache_len + pos[t]);
    double ang = p * pow((double)theta, -2.0 * (double)e / (double)D);
    double sn, c;
    sincos(ang, &sn, &c);
    cs[i] = make_float2((float)c, (float)sn);
}

void launch_rope_table(float2 *cs, const int32_t *cache_len, const int32_t *pos, int T, int D, float theta,
                       cudaStream_t s)
{
    int n = T * (D / 2);
    launch_pdl(rope_table_kernel, dim3((n + 127) / 128), dim3(128), 0, s, cs, cache_len, pos, T, D, theta);
}

// One thread handles four adjacent pairs (e..e+3, e+D/2..e+D/2+3) of one head of q, k or v (blockIdx.z): it adds the
// k-split planes of the QKV projection (both halves of a pair in flight together, four planes per round),
// rotates q and k, and stores.  A row of the projection's output is [q: H heads | k: Hkv heads | v: Hkv heads].
// With as many key/value heads as query heads one launch produced the whole row (pd_q == pd_kv, kv_col0 == 0);
// with fewer (grouped-query attention) q and [k | v] come from two launches with their own plane counts, and
// kv_col0 = H * D is the row column where the second launch's column 0 sits.
template <typename AT>
__global__ void __launch_bounds__(256)
rope_split_kernel(const float *__restrict__ qkv, PlaneDesc pd_q, PlaneDesc pd_kv, int kv_col0, const float2 *__restrict__ cs,
                  AT *__restrict__ q, AT *__restrict__ q_lo, AT *__restrict__ tk, AT *__restrict__ tv, int H, int Hkv, int D)
{
    pdl_enter();
    const int t = blockIdx.y, which = blockIdx.z, half = D / 2, per_head = half / 4;
    const int Hw = which == 0 ? H : Hkv, ld = (H + 2 * Hkv) * D;
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= Hw * per_head)
        return;
    const int h = idx / per_head, e = (idx % per_head) * 4;
    // column of the first half inside its launch's output, and inside the row
    const int col_l = which == 0 ? h * D + e : (H * D - kv_col0) + (which - 1) * Hkv * D + h * D + e;
    const int col = (which == 0 ? 0 : kv_col0) + col_l;
    const PlaneDesc &pd = which == 0 ? pd_q : pd_kv;
    const float *row = qkv + (size_t)t * ld + col;
    const int n_planes = planes_of_col(pd, col_l);  // a head never straddles two 128-column tiles' plane counts
    float4 a4 = make_float4(0.f, 0.f, 0.f, 0.f), b4 = a4;
    for (int p0 = 0; p0 < n_planes; p0 += 4) {
        float4 wa[4], wb[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int p = min(p0 + j, n_planes - 1);
            wa[j] = *reinterpret_cast<const float4 *>(row + (size_t)p * pd.stride);
            wb[j] = *reinterpret_cast<const float4 *>(row + (size_t)p * pd.stride + half);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (p0 + j < n_planes) {
                a4.x += wa[j].x; a4.y += wa[j].y; a4.z += wa[j].z; a4.w += wa[j].w;
                b4.x += wb[j].x; b4.y += wb[j].y; b4.z += wb[j].z; b4.w += wb[j].w;
            }
        }
    }
    const float xa[4] = {a4.x, a4.y, a4.z, a4.w}, xb[4] = {b4.x, b4.y, b4.z, b4.w};
    const size_t o = ((size_t)t * Hw + h) * D + e;
    if (which == 2) {
        store_split4<AT>(tv, nullptr, o, xa);
        store_split4<AT>(tv, nullptr, o + half, xb);
        return;
    }
    const float4 c01 = *reinterpret_cast<const float4 *>(cs + t * half + e);
    const float4 c23 = *reinterpret_cast<const float4 *>(cs + t * half + e + 2);
    const float cc[4] = {c01.x, c01.z, c23.x, c23.z}, sn[4] = {c01.y, c01.w, c23.y, c23.w};
    float y0[4], y1[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) { y0[i] = xa[i] * cc[i] - xb[i] * sn[i]; y1[i] = xb[i] * cc[i] + xa[i] * sn[i]; }
    // q may be kept as two planes (hi + lo), so that the scores do not carry q's rounding to one plane; keys are a
    // cache format (one plane by definition)
    AT *dst = which == 0 ? q : tk;
    AT *dst_lo = which == 0 ? q_lo : nullptr;
    store_split4<AT>(dst, dst_lo, o, y0);
    store_split4<AT>(dst, dst_lo, o + half, y1);
}

void launch_rope_split(int dtype, const float *qkv, const PlaneDesc &pd_q, const PlaneDesc &pd_kv, int kv_col0, const float2 *cs,
                       void *q, void *q_lo, void *tree_k, void *tree_v, int T, int H, int Hkv, int D, cudaStream_t s)
{
    const int n = H * (D / 8);
    dim3 grid((n + 255) / 256, T, 3);
    if (dtype == MEDUSA_BF16)
        launch_pdl(rope_split_kernel<bf16>, dim3(grid), dim3(256), 0, s, qkv, pd_q, pd_kv, kv_col0, cs, (bf16 *)q, (bf16 *)q_lo,
                   (bf16 *)tree_k, (bf16 *)tree_v, H, Hkv, D);
    else
        launch_pdl(rope_split_kernel<float>, dim3(grid), dim3(256), 0, s, qkv, pd_q, pd_kv, kv_col0, cs, (float *)q, (float *)nullptr,
                   (float *)tree_k, (float *)tree_v, H, Hkv, D);
}

template <typename AT>
__global__ void rope_apply_kernel(const AT *__restrict__ in, const float2 *__restrict__ cs, AT *__restrict__ out, int H,
                                  int D)
{
    pdl_enter();
    int t = blockIdx.x, h = blockIdx.y, half = D / 2;
    size_t o = ((size_t)t * H + h) * D;
    for (int e = threadIdx.x; e < half; e += blockDim.x) {
        float2 c = cs[t * half + e];
        float a = to_f32(in[o + e]), b = to_f32(in[o + e + half]);
        out[o + e] = from_f32<AT>(a * c.x - b * c.y);
        out[o + e + half] = from_f32<AT>(b * c.x + a * c.y);
    }
}

void launch_rope_apply(int dtype, const void *in, const float2 *cs, void *out, int T, int H, int D, cudaStream_t s)
{
    dim3 grid(T, H);
    if (dtype == MEDUSA_BF16)
        launch_pdl(rope_apply_kernel<bf16>, dim3(grid), dim3(64), 0, s, (const bf16 *)in, cs, (bf16 *)out, H, D);
    else
        launch_pdl(rope_apply_kernel<float>, dim3(grid), dim3(64), 0, s, (const float *)in, cs, (float *)out, H, D);
}

// ---------------------------------------------------------------------------------------- SwiGLU gate
// four elements per thread; the k-split planes of the fused gate/up projection are added on the fly
template <typename AT>
__global__ void __launch_bounds__(256)
silu_mul_kernel(const float *__restrict__ gu, PlaneDesc pd, AT *__restrict__ act, AT *__restrict__ act_lo,
                int F)
{
    pdl_enter();
    const int t = blockIdx.y;
    const int i = (blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (i >= F)
        return;
    float4 g = make_float4(0.f, 0.f, 0.f, 0.f), u = g;
    const float *row = gu + (size_t)t * 2 * F + i;
    const int ng = planes_of_col(pd, i), nu = planes_of_col(pd, F + i);  // gate and up live in different tiles
    for (int p0 = 0; p0 < max(ng, nu); p0 += 4) {  // four planes of each in flight per round, added in plane order
        float4 a[4], b[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            a[j] = *reinterpret_cast<const float4 *>(row + (size_t)min(p0 + j, ng - 1) * pd.stride);
            b[j] = *reinterpret_cast<const float4 *>(row + (size_t)min(p0 + j, nu - 1) * pd.stride + F);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (p0 + j < ng) { g.x += a[j].x; g.y += a[j].y; g.z += a[j].z; g.w += a[j].w; }
            if (p0 + j < nu) { u.x += b[j].x; u.y += b[j].y; u.z += b[j].z; u.w += b[j].w; }
        }
    }
    float y[4] = {silu_f(g.x) * u.x, silu_f(g.y) * u.y, silu_f(g.z) * u.z, silu_f(g.w) * u.w};
    store_split4<AT>(act, act_lo, (size_t)t * F + i, y);
}

void launch_silu_mul(int dtype, const float *gate_up, const PlaneDesc &pd, void *act, void *act_lo, int T,
                     int F, cudaStream_t s)
{
    dim3 grid((F / 4 + 255) / 256, T);
    if (dtype == MEDUSA_BF16)
        launch_pdl(silu_mul_kernel<bf16>, dim3(grid), dim3(256), 0, s, gate_up, pd, (bf16 *)act, (bf16 *)act_lo, F);
    else
        launch_pdl(silu_mul_kernel<float>, dim3(grid), dim3(256), 0, s, gate_up, pd, (float *)act, (float *)nullptr, F);
}

// ---------------------------------------------------------------------------------------- small helpers
__global__ void iota_kernel(int32_t *p, int n)
{
    pdl_enter();
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n)
        p[i] = i;
}
void launch_iota(int32_t *p, int n, cudaStream_t s) { launch_pdl(iota_kernel, dim3((n + 63) / 64), dim3(64), 0, s, p, n); }

// ---------------------------------------------------------------------------------------- read-only streaming probe
// Sums a buffer with 16-byte loads, eight in flight per thread, and writes one float per block: nothing but a DRAM
// read stream (the denominator for kernels that, like the projections and the attention, read far more than they write).
__global__ void __launch_bounds__(512) stream_read_kernel(const uint4 *__restrict__ p, long long n16, float *sink)
{
    const long long stride = (long long)gridDim.x * blockDim.x;
    long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    uint32_t acc = 0;
    for (; i + 7 * stride < n16; i += 8 * stride) {
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u)
            v[u] = __ldcs(p + i + u * stride);
#pragma unroll
        for (int u = 0; u < 8; ++u)
            acc += v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
    }
    for (; i < n16; i += stride) {
        const uint4 v = __ldcs(p + i);
        acc += v.x ^ v.y ^ v.z ^ v.w;
    }
    acc = __reduce_add_sync(0xffffffffu, acc);
    if ((threadIdx.x & 31) == 0 && acc == 0x9e3779b9u)  // practically never: keeps the loads alive
        sink[blockIdx.x] = 1.0f;
}
void launch_stream_read(const void *buf, long long bytes, float *sink, int blocks, cudaStream_t s)
{
    stream_read_kernel<<<blocks, 512, 0, s>>>((const uint4 *)buf, bytes / 16, sink);
}

}  // namespace medusa
