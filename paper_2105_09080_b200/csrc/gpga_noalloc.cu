// gpga_logistic_gradient_noalloc: the per-node mini-batch logistic gradient for callers
// that cannot allocate device memory.
//
// Who this is for: code that runs where cudaMalloc is off the table -- inside a region
// that must not synchronise the device or touch the allocator (a latency-critical serving
// loop, a framework plug-in that is handed its tensors and nothing else, a library used
// under another runtime's memory pool with no hook into it).  Such a caller can hand over
// its inputs and the output buffer, but has nowhere to get the intermediate storage the
// gradient kernel needs for its per-chunk partial sums.  Here that storage is a fixed
// array inside the library image itself.
//
// The scratch array below lives in every GPU context that loads this library, from load
// until exit, whether or not this entry point is ever called.  It is 4 MiB.
//
// Things a user must know:
//  * The first call on each device looks up the array's device address (a symbol query,
//    not an allocation).  Make that first call outside any CUDA stream capture.
//  * Every call on a device uses the same array.  It holds whatever the previous call
//    left; each call overwrites every element before reading it, so nothing needs to be
//    cleared -- but two calls that overlap on the GPU (different streams, or different
//    host threads without ordering) race on it.  Order them on one stream.
//  * Problems whose partial sums do not fit are refused with GPGA_ERR_UNSUPPORTED, and the
//    number of bytes they would have needed is reported through needed_bytes_host.
#include <mutex>

#include "../../include/gpga.h"
#include "gpga_logreg.cuh"

using namespace gpga;

namespace {

constexpr long long kStaticScratchFloats = GPGA_NOALLOC_SCRATCH_BYTES / 4;

// In host code this name is only a handle for symbol queries, never a device address.
static __device__ __align__(256) float g_static_scratch[kStaticScratchFloats];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
float* g_scratch_addr[kMaxDevices] = {nullptr};

// Device address of the scratch array on the current device, looked up once per device.
cudaError_t static_scratch(float** out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[dev]) {
        float* ptr = nullptr;
        e = cudaGetSymbolAddress((void**)&ptr, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" {

int32_t gpga_logistic_gradient_noalloc(const float* A_dev, const float* y_dev, const float* x_dev,
                                       int64_t ldx, int64_t n, int64_t d, int64_t m, int64_t batch,
                                       float l2, uint64_t seed, int64_t k, float* G_dev, void* stream,
                                       int64_t* needed_bytes_host)
{
    if (needed_bytes_host) *needed_bytes_host = 0;
    if (!A_dev || !y_dev || !x_dev || !G_dev) return GPGA_ERR_INVALID_ARG;
    if (n < 1 || n > 65535 || d < 4 || (d % 4) != 0 || d > 48 * 1024 || ldx < d || (ldx % 4) != 0 ||
        m < 1 || m >= (int64_t(1) << 31) || batch < 1 || batch > (int64_t(1) << 20) || k < 0 ||
        k >= (int64_t(1) << 32) || !(l2 >= 0.f))
        return GPGA_ERR_INVALID_ARG;
    if (((uintptr_t)A_dev | (uintptr_t)x_dev | (uintptr_t)G_dev) & 15u) return GPGA_ERR_INVALID_ARG;
    // partial sums: ceil(batch / 32) * n * d floats
    const long long need = (long long)logreg_chunks(batch) * n * d;
    if (needed_bytes_host) *needed_bytes_host = need * 4;
    if (need > kStaticScratchFloats) return GPGA_ERR_UNSUPPORTED;   // larger than the built-in scratch
    float* scratch = nullptr;
    cudaError_t e = static_scratch(&scratch);
    if (e != cudaSuccess) return GPGA_ERR_CUDA;
    LogregParams p;
    p.A = A_dev;
    p.y = y_dev;
    p.x = x_dev;
    p.ldx = ldx;
    p.partial = scratch;
    p.G = G_dev;
    p.error_flag = nullptr;
    p.n = n; p.d = d; p.m = m; p.batch = batch;
    p.k = (uint32_t)k;
    p.l2 = l2;
    p.keys = make_philox_keys((uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32));
    e = launch_logreg_grad(p, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? GPGA_OK : GPGA_ERR_CUDA;
}

}  // extern "C"
