// Launchers for the per-node logistic-regression gradient and mini-batch loss.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "gpga_device.cuh"

namespace gpga {

constexpr int kChunkRows = 32;   // batch rows per block

struct LogregParams {
    const float* A;   // n x m x d
    const float* y;   // n x m, +-1
    const float* x;   // n x d, current state, row stride ldx
    long long ldx;
    float* partial;   // chunks x n x d
    float* G;         // n x d
    int* error_flag;  // set to 1 if a bounded wait inside a kernel gave up (may be NULL)
    long long n, d, m, batch;
    long long node0 = 0;   // global index of local node 0 (node sharding): keys the mini-batch draws
    uint32_t k;
    float l2;
    PhiloxKeys keys;
    // true only when the launch before this one on the stream is this library's own step kernel of
    // the previous iteration: the gradient kernel may then start drawing and copying rows of A
    // (which no kernel writes) while that step kernel is still running
    bool after_own_step = false;
};

int logreg_chunks(long long batch);
// One block waits (bounded) on a barrier nobody completes and must set *error_flag.
cudaError_t launch_bounded_wait_selftest(int* error_flag, cudaStream_t s);
// One launch: chunk partials only (the consumer adds them in index order).
cudaError_t launch_logreg_partial(const LogregParams& p, cudaStream_t s);
// Two launches: chunk partials, then the fixed-order sum into G (adds l2 x).
cudaError_t launch_logreg_grad(const LogregParams& p, cudaStream_t s);
// Two launches: per-node mini-batch loss (n doubles), then their mean into *result.
cudaError_t launch_logreg_loss(const LogregParams& p, double* node_loss, double* result, cudaStream_t s);

}  // namespace gpga
