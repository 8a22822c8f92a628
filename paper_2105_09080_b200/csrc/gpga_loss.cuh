// Global loss of problem (1), (1/n) sum_i f_i(xbar), evaluated at the node average xbar.
#pragma once
#include <cuda_runtime.h>

namespace gpga {

// Quadratic objective: (1/n) sum_i 1/2 ||xbar - b_i||^2.  partials: >= kMaxReduceBlocks doubles.
cudaError_t launch_quadratic_global_loss(const float* x, const float* b, long long n, long long d, long long ld,
                                         bool vec, double* partials, double* result, cudaStream_t s);

// Logistic objective over the full local data sets:
// (1/n) sum_i [ (1/m) sum_r ln(1 + exp(-y_ir a_ir^T xbar)) ] + (l2/2) ||xbar||^2.
// xbar: d floats of scratch; partials: `slots` doubles of scratch.
cudaError_t launch_logistic_global_loss(const float* A, const float* y, const float* x, long long ldx, long long n,
                                        long long d, long long m, float l2, float* xbar, double* partials,
                                        long long slots, double* result, cudaStream_t s);

}  // namespace gpga
