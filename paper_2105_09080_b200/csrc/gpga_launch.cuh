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

}  // namespace gpga
