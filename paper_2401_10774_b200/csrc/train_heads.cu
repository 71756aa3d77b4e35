// Training of the Medusa heads with a frozen backbone (paper Sec. 2.2.1, Eq. 1): the element-wise and layout kernels
// around the five projections of one forward/backward pass of a head over up to 256 positions.  The projections
// themselves run on the tcgen05 GEMM of the decode path (gemm_tc.cu), whose streamed ("weight") operand is a
// row-major [rows][K] bf16 matrix and whose token operand is a split activation; the transposes below put the
// activations and gradients into those two forms.
//
//   a   = W1 h                      (projection)      h1 = h + SiLU(a)                      head_hidden_fwd_kernel
//   z   = W2 h1                     (projection)      loss, dz = lambda/n (softmax(z) - y)  ce_grad_kernel
//   gW2 = dz^T h1                   (projection of h1^T rows against dz^T; its epilogue stores or accumulates transposed)
//   dh1 = dz W2                     (projection against W2^T)
//   da  = dh1 * SiLU'(a)                                                                    head_hidden_bwd_kernel
//   gW1 = da^T h                    (projection of h^T rows against da^T, likewise)
#include "common.cuh"
#include "gemm_tc.h"
#include "kernels.h"

namespace medusa {

namespace {

__device__ __forceinline__ float plane_sum(const float *P, const PlaneDesc &pd, size_t off, int col)
{
    const int n = planes_of_col(pd, col);
    float acc = 0.f;
    for (int p = 0; p < n; ++p)  // plane order: the result does not depend on timing
        acc += P[(size_t)p * pd.stride + off];
    return acc;
}

__device__ __forceinline__ void split_store(bf16 *hi, bf16 *lo, size_t at, float y)
{
    const bf16 h = __float2bfloat16_rn(y);
    hi[at] = h;
    lo[at] = __float2bfloat16_rn(y - __bfloat162float(h));
}

// a[r][c] = sum of the projection's planes; h1 = h + SiLU(a) as a split activation; a is kept for the backward pass
__global__ void __launch_bounds__(256)
head_hidden_fwd_kernel(const float *__restrict__ A_planes, PlaneDesc pd, const bf16 *__restrict__ H, float *__restrict__ A,
                       bf16 *__restrict__ h1_hi, bf16 *__restrict__ h1_lo, int rows, int d)
{
    const size_t n = (size_t)rows * d;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const int col = (int)(i % d);
        const float a = plane_sum(A_planes, pd, i, col);
        A[i] = a;
        const float s = 1.f / (1.f + __expf(-a));
        split_store(h1_hi, h1_lo, i, __bfloat162float(H[i]) + a * s);
    }
}

// da = dh1 * SiLU'(a), SiLU'(a) = s (1 + a (1 - s)) with s = sigmoid(a); one bf16 plane (it becomes a streamed operand)
__global__ void __launch_bounds__(256)
head_hidden_bwd_kernel(const float *__restrict__ dH1_planes, PlaneDesc pd, const float *__restrict__ A, bf16 *__restrict__ dA,
                       int rows, int d)
{
    const size_t n = (size_t)rows * d;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const int col = (int)(i % d);
        const float g = plane_sum(dH1_planes, pd, i, col);
        const float a = A[i];
        const float s = 1.f / (1.f + __expf(-a));
        dA[i] = __float2bfloat16_rn(g * (s * (1.f + a * (1.f - s))));
    }
}

__device__ float block_max(float v, float *sh)
{
    for (int o = 16; o > 0; o >>= 1)
        v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = sh[0];
    for (int w = 1; w < (int)(blockDim.x >> 5); ++w)
        t = fmaxf(t, sh[w]);
    return t;
}
__device__ double block_sum(double v, double *sh)
{
    for (int o = 16; o > 0; o >>= 1)
        v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
    __syncthreads();
    double t = 0.0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w)  // same order in every thread
        t += sh[w];
    return t;
}

// One block per position: cross-entropy of the row's logits against its label (-1: the position has no label and
// contributes nothing) and the gradient of lambda * mean-over-labelled-positions of it with respect to the logits,
// as a split activation.  The normaliser is the head's number of labelled positions over the WHOLE batch (n_valid).
__global__ void __launch_bounds__(512)
ce_grad_kernel(const float *__restrict__ Z, int V, const int32_t *__restrict__ labels, int rows_valid,
               const int32_t *__restrict__ n_valid, float lambda, float *__restrict__ row_loss, bf16 *__restrict__ dz_hi,
               bf16 *__restrict__ dz_lo)
{
    __shared__ float shf[32];
    __shared__ double shd[32];
    const int row = blockIdx.x;
    const int y = row < rows_valid ? labels[row] : -1;
    const size_t base = (size_t)row * V;
    if (y < 0 || y >= V) {
        for (int v = threadIdx.x; v < V; v += blockDim.x) {
            dz_hi[base + v] = __float2bfloat16_rn(0.f);
            dz_lo[base + v] = __float2bfloat16_rn(0.f);
        }
        if (threadIdx.x == 0) row_loss[row] = 0.f;
        return;
    }
    const float *z = Z + base;
    float m = -INFINITY;
    for (int v = threadIdx.x; v < V; v += blockDim.x)
        m = fmaxf(m, z[v]);
    m = block_max(m, shf);
    double se = 0.0;
    for (int v = threadIdx.x; v < V; v += blockDim.x)
        se += (double)__expf(z[v] - m);
    se = block_sum(se, shd);
    const float lse = m + (float)log(se);
    const float scale = lambda / (float)max(*n_valid, 1);
    for (int v = threadIdx.x; v < V; v += blockDim.x) {
        const float p = __expf(z[v] - lse);
        split_store(dz_hi, dz_lo, base + v, scale * (p - (v == y ? 1.f : 0.f)));
    }
    if (threadIdx.x == 0) row_loss[row] = lse - z[y];
}

// loss[k] += sum(row_loss) / n_valid;  loss[K] += lambda * that   (one thread: a fixed order of additions)
__global__ void loss_accumulate_kernel(const float *__restrict__ row_loss, int rows, const int32_t *__restrict__ n_valid,
                                       float lambda, float *loss_k, float *loss_total)
{
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    double s = 0.0;
    for (int r = 0; r < rows; ++r)
        s += (double)row_loss[r];
    const float mean_part = (float)(s / (double)max(*n_valid, 1));
    *loss_k += mean_part;
    *loss_total += lambda * mean_part;
}

// n_valid[k] = number of labels >= 0 of head k
__global__ void __launch_bounds__(256) count_valid_kernel(const int32_t *__restrict__ labels, int N, int32_t *__restrict__ n_valid)
{
    __shared__ double shd[32];
    double c = 0.0;
    for (int n = threadIdx.x; n < N; n += blockDim.x)
        c += labels[(size_t)blockIdx.x * N + n] >= 0 ? 1.0 : 0.0;
    c = block_sum(c, shd);
    if (threadIdx.x == 0) n_valid[blockIdx.x] = (int32_t)c;
}

// out[c][r] = in[r][c] for a row-major [R][C] matrix (leading dimensions given), 32 x 32 tiles through shared memory
template <typename T>
__global__ void __launch_bounds__(256) transpose_kernel(const T *__restrict__ in, int R, int Cc, long long ld_in, T *__restrict__ out,
                                                        long long ld_out)
{
    __shared__ T tile[32][33];
    const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;  // 32 x 8
    for (int j = ty; j < 32; j += 8) {
        const int r = r0 + j, c = c0 + tx;
        if (r < R && c < Cc) tile[j][tx] = in[(size_t)r * ld_in + c];
    }
    __syncthreads();
    for (int j = ty; j < 32; j += 8) {
        const int c = c0 + j, r = r0 + tx;
        if (r < R && c < Cc)
            out[(size_t)c * ld_out + r] = tile[tx][j];
    }
}

}  // namespace

void launch_head_hidden_fwd(const float *A_planes, const PlaneDesc &pd, const void *H, float *A, void *h1_hi, void *h1_lo, int rows,
                            int d, cudaStream_t s)
{
    head_hidden_fwd_kernel<<<592, 256, 0, s>>>(A_planes, pd, (const bf16 *)H, A, (bf16 *)h1_hi, (bf16 *)h1_lo, rows, d);
}
void launch_head_hidden_bwd(const float *dH1_planes, const PlaneDesc &pd, const float *A, void *dA, int rows, int d, cudaStream_t s)
{
    head_hidden_bwd_kernel<<<592, 256, 0, s>>>(dH1_planes, pd, A, (bf16 *)dA, rows, d);
}
void launch_ce_grad(const float *Z, int V, const int32_t *labels, int rows, int rows_valid, const int32_t *n_valid, float lambda,
                    float *row_loss, void *dz_hi, void *dz_lo, cudaStream_t s)
{
    ce_grad_kernel<<<rows, 512, 0, s>>>(Z, V, labels, rows_valid, n_valid, lambda, row_loss, (bf16 *)dz_hi, (bf16 *)dz_lo);
}
void launch_loss_accumulate(const float *row_loss, int rows, const int32_t *n_valid, float lambda, float *loss_k, float *loss_total,
                            cudaStream_t s)
{
    loss_accumulate_kernel<<<1, 32, 0, s>>>(row_loss, rows, n_valid, lambda, loss_k, loss_total);
}
void launch_count_valid(const int32_t *labels, int K, int N, int32_t *n_valid, cudaStream_t s)
{
    count_valid_kernel<<<K, 256, 0, s>>>(labels, N, n_valid);
}
void launch_transpose_bf16(const void *in, int R, int Cc, long long ld_in, void *out, long long ld_out, cudaStream_t s)
{
    transpose_kernel<bf16><<<dim3((Cc + 31) / 32, (R + 31) / 32), 256, 0, s>>>((const bf16 *)in, R, Cc, ld_in, (bf16 *)out, ld_out);
}
}  // namespace medusa
