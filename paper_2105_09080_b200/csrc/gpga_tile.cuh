// Multi-iteration launcher of the shared-memory tile path (defined in gpga_tile.cu).
#pragma once
#include "gpga_kernels.cuh"

namespace gpga {

// A general sparse weight matrix W in CSR form on the device (row i: entries
// row_ptr[i] .. row_ptr[i+1]-1 give neighbour col[e] and weight w[e]).  All NULL = not used.
struct SparseW {
    const int* row_ptr = nullptr;
    const int* col = nullptr;
    const float* w = nullptr;
};

// Single-iteration tile launch with a CSR weight matrix (mix = GPGA_TOPO_SPARSE) or without.
cudaError_t launch_step_tile_w(const StepParams& p, int mode, bool vec, int mix, const SparseW& sw, cudaStream_t s);

// `steps` iterations starting at p.k in one launch, the strip of X, b, Y resident in shared
// memory (quadratic objective; bit-identical to `steps` single-iteration launches).
cudaError_t launch_run_tile(const StepParams& p, int mode, bool vec, int topology, long long H, int steps,
                            const SparseW& sw, cudaStream_t s);
bool run_tile_supports(long long n);

}  // namespace gpga
