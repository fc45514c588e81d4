// Programmatic dependent launch: every kernel of this library is launched with the
// programmatic-stream-serialization attribute and begins with pdl_enter().  A kernel then starts
// as soon as all CTAs of the kernel before it on the stream have started (they signal it first
// thing), runs its set-up (barrier init, TMEM allocation, tensor-map prefetch) while that kernel
// drains, and touches global memory only after griddepcontrol.wait has seen it complete and its
// writes flushed.  The data dependences between the launches of one call (copy -> GEMM -> reduce)
// and between calls that share a workspace are therefore kept; only the launch latency overlaps.
#pragma once

#include <cuda_runtime.h>
#include <cstring>
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

// Launch recorder (measurement support): while a thread has one armed, every launch it makes through
// launch_exc is also written down (configuration, attributes, kernel, a copy of the argument bytes), so that
// the same launches can be replayed bare and the host cost of a library call be compared with the cost of
// its launches alone.
struct LaunchRecord {
    static constexpr int kMax = 4;
    static constexpr size_t kArgBytes = 6144;
    int n = 0;
    struct One {
        cudaLaunchConfig_t cfg;
        cudaLaunchAttribute attrs[4];
        const void* func;
        int nargs;
        size_t off[8];
        alignas(64) unsigned char bytes[kArgBytes];
    } launch[kMax];
};
inline LaunchRecord*& launch_recorder()
{
    static thread_local LaunchRecord* r = nullptr;
    return r;
}

// Every launch of the library goes through here: cudaLaunchKernelExC with the arguments as an array of
// pointers (arg_bytes gives their sizes for the recorder).
inline cudaError_t launch_exc(const cudaLaunchConfig_t* cfg, const void* func, void** args, const size_t* arg_bytes, int nargs)
{
    LaunchRecord* rec = launch_recorder();
    if (rec && rec->n < LaunchRecord::kMax && nargs <= 8 && cfg->numAttrs <= 4) {
        LaunchRecord::One& o = rec->launch[rec->n];
        size_t off = 0;
        bool fits = true;
        for (int i = 0; i < nargs; ++i) {
            off = (off + 63) & ~(size_t)63;
            if (off + arg_bytes[i] > LaunchRecord::kArgBytes) { fits = false; break; }
            o.off[i] = off;
            memcpy(o.bytes + off, args[i], arg_bytes[i]);
            off += arg_bytes[i];
        }
        if (fits) {
            o.cfg = *cfg;
            for (unsigned i = 0; i < cfg->numAttrs; ++i) o.attrs[i] = cfg->attrs[i];
            o.cfg.attrs = o.attrs;
            o.func = func;
            o.nargs = nargs;
            ++rec->n;
        }
    }
    return cudaLaunchKernelExC(cfg, func, args);
}

inline cudaError_t launch_replay(LaunchRecord::One& o, cudaStream_t stream)
{
    void* args[8];
    for (int i = 0; i < o.nargs; ++i) args[i] = o.bytes + o.off[i];
    o.cfg.stream = stream;
    o.cfg.attrs = o.attrs;
    return cudaLaunchKernelExC(&o.cfg, o.func, args);
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args&&... args)
{
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    pdl_attribute(&attr[0]);
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    // the arguments converted to the kernel's parameter types, then passed by address
    return [&](KArgs... coerced) {
        void* argv[] = {(void*)&coerced...};
        const size_t sizes[] = {sizeof(KArgs)...};
        return launch_exc(&cfg, (const void*)kernel, argv, sizes, (int)sizeof...(KArgs));
    }(std::forward<Args>(args)...);
}

}  // namespace adapt
