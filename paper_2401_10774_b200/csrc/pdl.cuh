// Programmatic dependent launch: every kernel of the decode path is launched with the stream-serialisation
// attribute relaxed, so that its blocks may be scheduled and run their prologue while the previous kernel in
// the stream is still finishing.  The protocol inside a kernel is: (1) `pdl_trigger()` as early as possible,
// which allows the NEXT kernel's blocks to start once all of this kernel's blocks have started;
// (2) `pdl_wait()` before the first access to anything an earlier kernel wrote (it returns once the previous
// kernel has completed and its writes are visible; completion is transitive along the stream);
// before the wait a kernel may only touch its own on-chip state and data that no kernel writes (weights).
#pragma once
#include <cuda_runtime.h>

#include <cstdlib>
#include <utility>

namespace medusa {

__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_enter()
{
    pdl_trigger();
    pdl_wait();
}

// MEDUSA_NO_PDL=1 launches every kernel fully serialised (comparison runs; builds with -DMEDUSA_TIMING_AIDS only)
inline bool pdl_enabled()
{
#ifdef MEDUSA_TIMING_AIDS
    static const bool on = getenv("MEDUSA_NO_PDL") == nullptr;
#else
    static const bool on = true;
#endif
    return on;
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pdl_enabled() ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

}  // namespace medusa
