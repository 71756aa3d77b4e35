// Shared device/host helpers of the Medusa B200 library: element-type traits, status words, launch checks.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <cstdlib>

#include "../../include/medusa.h"

namespace medusa {

constexpr int MAX_T = 256;      // tree nodes incl. root (one 64-bit mask word per query and 64 nodes)
constexpr int MAX_DEPTH = 8;
constexpr int TREE_ROWS = 64;   // token rows per tile: projections and attention work on tiles of 64 tree tokens; a
                                // context holds rows = 64 * ceil(max_tree_nodes / 64) of them (the row stride of its
                                // per-layer tree K/V scratch and of every activation buffer)

// indices into the int32 state block (MEDUSA_WS_STATE)
enum { ST_CACHE_LEN = 0, ST_ROOT = 1, ST_BEST = 2, ST_ACCEPT_LEN = 3, ST_NEXT_ROOT = 4, ST_N_EMITTED = 5,
       ST_STATUS = 6, ST_STEPS = 7, ST_WORDS = 8 };

using bf16 = __nv_bfloat16;

// Environment switches for comparison runs (MEDUSA_GEMM_STAGES, MEDUSA_NO_PDL, MEDUSA_DEBUG_SKIP, ...) exist only in a
// library built with -DMEDUSA_TIMING_AIDS; the default build reads nothing from its caller's environment.
inline const char *tuning_env(const char *name)
{
#ifdef MEDUSA_TIMING_AIDS
    return getenv(name);
#else
    (void)name;
    return nullptr;
#endif
}

// True the first time it is called with the calling thread's current device (function attributes such as the
// dynamic shared-memory limit are per device, so each device sets them once).
inline bool first_use_on_current_device(bool (&done)[64])
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64)
        return true;
    if (done[dev])
        return false;
    done[dev] = true;
    return true;
}

constexpr uint32_t DEFAULT_SPIN_LIMIT = 1u << 22;  // polls of a bounded device-side wait before it gives up

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<bf16>(bf16 v) { return __bfloat162float(v); }

template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f32<bf16>(float v) { return __float2bfloat16_rn(v); }

// 16-byte vector of elements, widened to float
template <typename T> struct Vec16;
template <> struct Vec16<float> {
    static constexpr int N = 4;
    __device__ __forceinline__ static void load(const float *p, float *out)
    {
        float4 v = *reinterpret_cast<const float4 *>(p);
        out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
    }
    __device__ __forceinline__ static void store(float *p, const float *in)
    {
        *reinterpret_cast<float4 *>(p) = make_float4(in[0], in[1], in[2], in[3]);
    }
};
template <> struct Vec16<bf16> {
    static constexpr int N = 8;
    __device__ __forceinline__ static void load(const bf16 *p, float *out)
    {
        uint4 v = *reinterpret_cast<const uint4 *>(p);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            out[2 * i] = __uint_as_float(w[i] << 16);
            out[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    __device__ __forceinline__ static void store(bf16 *p, const float *in)
    {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 t = __floats2bfloat162_rn(in[2 * i], in[2 * i + 1]);
            w[i] = *reinterpret_cast<uint32_t *>(&t);
        }
        *reinterpret_cast<uint4 *>(p) = make_uint4(w[0], w[1], w[2], w[3]);
    }
};

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
        v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
        v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

__device__ __forceinline__ float silu_f(float u) { return u / (1.0f + expf(-u)); }

}  // namespace medusa
