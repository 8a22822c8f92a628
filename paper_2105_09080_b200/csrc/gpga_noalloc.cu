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
//    not an allocation).  Under CUDA's lazy module loading that first query or launch is also
//    when the driver loads this library's device code and sets the array aside, and it may
//    synchronise the device.  Make that first call at start-up, outside any CUDA stream
//    capture and outside the region that must not stall.
//  * All four buffers must belong to the device that is current when the call is made; the
//    call checks this (a pointer query) and launches nothing otherwise.
//  * There is no handle and so no error word.  If a bounded wait inside the gradient kernel
//    gives up (an asynchronous row copy that does not complete within about a second), the
//    block writes NaN over its slice of the partial sums, so the affected rows of G come
//    out NaN rather than stale; the status, returned at launch time, is still GPGA_OK.
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

// Device address of the scratch array on device `dev` (the current one), looked up once per device.
cudaError_t static_scratch(int dev, float** out)
{
    cudaError_t e;
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

// The kernels run on the current device and use that device's copy of the scratch array, so every
// buffer must be memory that device owns (or managed memory).  A pointer query, not an allocation.
// A buffer of another GPU would be an illegal address there -- or, with peer access enabled, would
// quietly work while the partial sums land in the wrong device's array.
bool on_device(const void* p, int dev)
{
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, p) != cudaSuccess) {
        (void)cudaGetLastError();   // a pointer CUDA does not know: not an error of the context
        return false;
    }
    if (a.type == cudaMemoryTypeManaged) return true;
    return a.type == cudaMemoryTypeDevice && a.device == dev;
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
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return GPGA_ERR_CUDA;
    if (!on_device(A_dev, dev) || !on_device(y_dev, dev) || !on_device(x_dev, dev) || !on_device(G_dev, dev))
        return GPGA_ERR_INVALID_ARG;   // not this device's memory: nothing is launched
    float* scratch = nullptr;
    e = static_scratch(dev, &scratch);
    if (e != cudaSuccess) return GPGA_ERR_CUDA;
    LogregParams p;
    p.A = A_dev;
    p.y = y_dev;
    p.x = x_dev;
    p.ldx = ldx;
    p.partial = scratch;
    p.G = G_dev;
    p.error_flag = nullptr;   // no handle, no error word: a block whose bounded wait gives up writes NaN instead
    p.n = n; p.d = d; p.m = m; p.batch = batch;
    p.k = (uint32_t)k;
    p.l2 = l2;
    p.keys = make_philox_keys((uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32));
    e = launch_logreg_grad(p, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? GPGA_OK : GPGA_ERR_CUDA;
}

}  // extern "C"
