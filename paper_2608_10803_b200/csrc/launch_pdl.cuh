// Programmatic dependent launch: every kernel of this library is launched with the
// programmatic-stream-serialization attribute and begins with pdl_enter().  A kernel then starts
// as soon as all CTAs of the kernel before it on the stream have started (they signal it first
// thing), runs its set-up (barrier init, TMEM allocation, tensor-map prefetch) while that kernel
// drains, and touches global memory only after griddepcontrol.wait has seen it complete and its
// writes flushed.  The data dependences between the launches of one call (copy -> GEMM -> reduce)
// and between calls that share a workspace are therefore kept; only the launch latency overlaps.
#pragma once

#include <cuda_runtime.h>
#include <utility>

namespace adapt {

// Allow the next kernel on the stream to be scheduled.  It is released once every CTA of this
// grid has executed this (or exited), so no CTA of this grid is left waiting for an SM.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
// Wait until the kernels this one depends on have completed and their memory is visible.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

inline bool& pdl_enabled()
{
    static bool on = true;      // ADAPT_NO_PDL=1 turns the launch attribute off (the device-side calls are then no-ops)
    return on;
}

// Fills the one attribute slot of a launch configuration.
inline void pdl_attribute(cudaLaunchAttribute* attr)
{
    attr->id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr->val.programmaticStreamSerializationAllowed = pdl_enabled() ? 1 : 0;
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args&&... args)
{
    cudaLaunchConfig_t cfg;
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    pdl_attribute(&attr[0]);
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

}  // namespace adapt
