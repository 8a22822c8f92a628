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

// Node shards: the whole problem's diagnostics from the shards' parts.  sums: 4 ceil(d/4) doubles, the
// fp64 column sums of the shard's rows; gathered: `parts` such vectors in shard order.
cudaError_t launch_shard_state_sums(const float* x, long long n, long long d, long long ld, bool vec, double* sums,
                                    cudaStream_t s);
// sum over the local rows of ||x_i - xbar||^2, xbar = (sum of the parts) / n_total
cudaError_t launch_shard_consensus_part(const float* x, long long n, long long d, long long ld, bool vec,
                                        const double* gathered, int parts, long long n_total, double* partials,
                                        double* result, cudaStream_t s);
// (1 / n_total) sum over the local rows of f_i(xbar)
cudaError_t launch_shard_quadratic_loss_part(const float* b, long long n, long long d, long long ld, bool vec,
                                             const double* gathered, int parts, long long n_total, double* partials,
                                             double* result, cudaStream_t s);
cudaError_t launch_shard_logistic_loss_part(const float* A, const float* y, long long n, long long d, long long m, float l2,
                                            const double* gathered, int parts, long long n_total, float* xbar,
                                            double* partials, long long slots, double* result, cudaStream_t s);

}  // namespace gpga
