// Multi-iteration launcher of the shared-memory tile path (defined in gpga_tile.cu).
#pragma once
#include "gpga_kernels.cuh"

namespace gpga {

// `steps` iterations starting at p.k in one launch, the strip of X, b, Y resident in shared
// memory (quadratic objective; bit-identical to `steps` single-iteration launches).
cudaError_t launch_run_tile(const StepParams& p, int mode, bool vec, int topology, long long H, int steps,
                            cudaStream_t s);
bool run_tile_supports(long long n);

}  // namespace gpga
