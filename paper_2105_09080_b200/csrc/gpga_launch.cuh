// Launch helpers (host side).
#pragma once
#include <cuda_runtime.h>

namespace gpga {

// Raises a kernel's dynamic shared-memory limit once per device instead of on every
// launch (the attribute call costs about as much as a launch).  `done_mask` is a static
// of the call site, one bit per device; setting the attribute twice is harmless, so a
// race between host threads only repeats the call.
template <class Kernel>
inline cudaError_t ensure_smem_limit(Kernel kernel, int bytes, unsigned long long& done_mask)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const unsigned long long bit = 1ull << (dev & 63);
    if (done_mask & bit) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) done_mask |= bit;
    return e;
}

// Programmatic dependent launch.  A kernel launched with launch_after_trigger(..., true)
// may begin once every block of the kernel before it on the stream has called
// grid_launch_dependents() (or exited); whatever it does before grid_dependency_wait() runs
// beside that kernel and must touch nothing that kernel writes or still reads.
// grid_dependency_wait() returns when the earlier kernel has completed and its writes are
// visible; without an earlier kernel, or in a plain launch, it returns at once.
#ifdef __CUDACC__
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

template <class... KernelArgs, class... Args>
inline cudaError_t launch_after_trigger(void (*kernel)(KernelArgs...), dim3 grid, dim3 block, size_t smem,
                                        cudaStream_t s, bool early, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = early ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, KernelArgs(args)...);
}
#endif

}  // namespace gpga
