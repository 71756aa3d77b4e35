// Tree attention (paper Sec. 2.1.2, Fig. 2): every tree query attends to the whole KV cache and, inside the
// tree, only to itself and its ancestors.  This file holds the shape-generic CUDA-core kernel: one warp per
// (query, head), the lanes split the head dimension, scores reduced by warp shuffles, online softmax in
// float.  The key order (cache positions, then tree nodes in index order) is the same for every query, so a
// node's output does not depend on which other nodes share the launch.
#include "common.cuh"
#include "pdl.cuh"
#include "kernels.h"

namespace medusa {

template <typename AT, int D>
__global__ void __launch_bounds__(128)
tree_attention_simt_kernel(const AT *__restrict__ q, const AT *__restrict__ k_new, const AT *__restrict__ v_new,
                           const AT *__restrict__ k_cache, const AT *__restrict__ v_cache,
                           const int32_t *__restrict__ cache_len, const uint64_t *__restrict__ mask,
                           AT *__restrict__ out, AT *__restrict__ out_lo, float *__restrict__ lse, int T, int H,
                           int Hkv, int L_max, int mask_words)
{
    pdl_enter();
    constexpr int E = D / 32;  // elements per lane
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int i = blockIdx.x * 4 + warp, h = blockIdx.y;
    if (i >= T)
        return;
    const int hk = h / (H / Hkv);  // grouped-query attention: the key/value head this query head reads
    const int L = min(max(*cache_len, 0), L_max);  // a length outside [0, L_max] would index past the caches
    const float scale = rsqrtf((float)D);
    float qv[E], o[E];
#pragma unroll
    for (int e = 0; e < E; ++e) {
        qv[e] = to_f32(q[((size_t)i * H + h) * D + lane * E + e]) * scale;
        o[e] = 0.f;
    }
    float m = -INFINITY, l = 0.f;
    const uint64_t *mk = mask + (size_t)i * mask_words;  // the query's ancestor set, 64 tree nodes per word
    const int nk = L + T;
    for (int j = 0; j < nk; ++j) {
        const AT *kp, *vp;
        if (j < L) {
            kp = k_cache + ((size_t)hk * L_max + j) * D;
            vp = v_cache + ((size_t)hk * L_max + j) * D;
        } else {
            if (!((mk[(j - L) >> 6] >> ((j - L) & 63)) & 1ull))
                continue;
            kp = k_new + ((size_t)(j - L) * Hkv + hk) * D;
            vp = v_new + ((size_t)(j - L) * Hkv + hk) * D;
        }
        float s = 0.f;
#pragma unroll
        for (int e = 0; e < E; ++e)
            s = fmaf(qv[e], to_f32(kp[lane * E + e]), s);
        s = warp_sum(s);
        float mn = fmaxf(m, s);
        float corr = expf(m - mn), p = expf(s - mn);
        l = l * corr + p;
#pragma unroll
        for (int e = 0; e < E; ++e)
            o[e] = fmaf(p, to_f32(vp[lane * E + e]), o[e] * corr);
        m = mn;
    }
    float inv = 1.0f / l;
#pragma unroll
    for (int e = 0; e < E; ++e) {
        size_t idx = ((size_t)i * H + h) * D + lane * E + e;
        float y = o[e] * inv;
        AT hi = from_f32<AT>(y);
        out[idx] = hi;
        if (out_lo)  // second plane of a split activation: the rounding residual
            out_lo[idx] = from_f32<AT>(y - to_f32(hi));
    }
    if (lse && lane == 0)
        lse[(size_t)i * H + h] = m + logf(l);
}

void launch_tree_attention_simt(int dtype, const void *q, const void *k_new, const void *v_new, const void *k_cache,
                                const void *v_cache, const int32_t *cache_len, const uint64_t *mask, void *out,
                                void *out_lo, float *lse, int T, int H, int Hkv, int D, int L_max, cudaStream_t s,
                                int mask_words)
{
    dim3 grid((T + 3) / 4, H);
#define MEDUSA_ATT(AT, DD)                                                                                         \
    launch_pdl(tree_attention_simt_kernel<AT, DD>, dim3(grid), dim3(128), 0, s, (const AT *)q, (const AT *)k_new, (const AT *)v_new,  \
                                                            (const AT *)k_cache, (const AT *)v_cache, cache_len,  \
                                                            mask, (AT *)out, (AT *)out_lo, lse, T, H, Hkv, L_max, mask_words)
    if (dtype == MEDUSA_BF16) {
        if (D == 128) MEDUSA_ATT(bf16, 128); else MEDUSA_ATT(bf16, 64);
    } else {
        if (D == 128) MEDUSA_ATT(float, 128); else MEDUSA_ATT(float, 64);
    }
#undef MEDUSA_ATT
}

}  // namespace medusa
