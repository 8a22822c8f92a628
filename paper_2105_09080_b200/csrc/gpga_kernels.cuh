// Kernel launchers of libgpga (host-callable; defined in gpga_kernels.cu).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "gpga_device.cuh"

namespace gpga {

// How the stochastic gradient G of Algorithm 1 is obtained inside the fused kernels.
enum GradMode {
    GRAD_QUAD = 0,        // g = x - b
    GRAD_QUAD_NOISE = 1,  // g = (x - b) + sigma * xi, xi generated in registers
    GRAD_BUFFER = 2,      // g read from an n x d buffer (written by the logistic kernel)
    GRAD_PARTIALS = 3     // g = (1/B) sum_c partial[c] + l2 x, partials from the logistic kernel (tile kernel only)
};

// Mixing selector of the tile kernel: a GPGA_TOPO_* value, or the global average.
enum { TILE_MIX_GLOBAL = 100 };

struct StepParams {
    const float* x;   // X^(k), n x d
    const float* b;   // quadratic: targets b; GRAD_BUFFER: gradient matrix G
    float* out;       // X^(k+1), n x d
    long long n, d;
    long long ld;     // row stride of x and out, in floats (>= d)
    long long ldb;    // row stride of b, in floats
    long long Q;      // column groups of four: ceil(d / 4)
    uint32_t q_base;  // global index of local group 0 (column offset / 4)
    uint32_t k;       // iteration index (third counter word)
    float gamma, sigma;
    int hop_log2;     // one-peer exponential: hop = 1 << hop_log2
    int len_log2;     // cycle length n / hop = 1 << len_log2
    int grid_cols;    // torus columns (grid topology)
    int chunks;       // GRAD_PARTIALS: number of chunk partials (b points at them, dense n x d each)
    float inv_batch;  // GRAD_PARTIALS: 1 / batch
    float l2;         // GRAD_PARTIALS: l2 coefficient
    PhiloxKeys keys;
};

// Fused local step + mix, one launch each.  mode is a GradMode; vec = 128-bit path usable.
cudaError_t launch_step_ring(const StepParams& p, int mode, bool vec, cudaStream_t s);
cudaError_t launch_step_exp(const StepParams& p, int mode, bool vec, cudaStream_t s);
cudaError_t launch_step_global(const StepParams& p, int mode, bool vec, cudaStream_t s);
// Generic neighbour-list mix through a shared-memory tile of Y (grid, static exponential, W = I).
cudaError_t launch_step_tile(const StepParams& p, int mode, bool vec, int mix, cudaStream_t s);
bool tile_supports(long long n);   // the n rows of one column group fit the shared-memory tile

// Consensus distance: partials (one double per block of 256 column groups) then a fixed-order final
// sum.  consensus_blocks(Q) is the number of partials it writes; the loss reductions use a
// grid-stride pass of at most kMaxReduceBlocks blocks (reduce_blocks).
constexpr int kMaxReduceBlocks = 148 * 8;
long long consensus_blocks(long long Q);
int reduce_blocks(long long Q);
cudaError_t launch_consensus(const float* x, long long n, long long d, long long ld, bool vec, double* partials,
                             double* result, cudaStream_t s);
// (1/n) sum_i 1/2 ||x_i - b_i||^2, same two-stage reduction.
cudaError_t launch_quadratic_loss(const float* x, const float* b, long long n, long long d, long long ld,
                                  bool vec, double* partials, double* result, cudaStream_t s);

// Seeded fills (quadratic objective); row0 = global index of local row 0 (node sharding).
cudaError_t launch_init_b(float* b, long long n, long long d, long long ld, uint32_t q_base, uint32_t row0, float shift,
                          bool vec, const PhiloxKeys& keys, cudaStream_t s);
cudaError_t launch_init_x0(float* x, long long n, long long d, long long ld, uint32_t q_base, uint32_t row0, int kind,
                           float std, bool vec, const PhiloxKeys& keys, cudaStream_t s);

// Generator surface.
cudaError_t launch_philox_words(const uint32_t* ctr, PhiloxKeys keys, long long count, uint32_t* out,
                                cudaStream_t s);
cudaError_t launch_box_muller_words(const uint32_t* a, const uint32_t* b, long long count, float* z,
                                    cudaStream_t s);
cudaError_t launch_normal_fill(PhiloxKeys keys, uint32_t stream_id, uint32_t k, uint32_t i,
                               uint32_t q0, long long count, float* out, cudaStream_t s);

}  // namespace gpga
