// Launchers of the node-sharded iteration (defined in gpga_shard.cu).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "gpga_device.cuh"

namespace gpga {

// How a shard kernel gets the stochastic gradient of a row.
enum ShardGrad { SHARD_GRAD_QUAD = 0, SHARD_GRAD_QUAD_NOISE = 1, SHARD_GRAD_BUFFER = 2 };

struct ShardParams {
    const float* x;      // X^(k), the shard's n x d rows, row stride ld
    const float* b;      // quadratic: targets b, row stride ldb = ld; BUFFER: the gradient matrix G, row stride ldb
    long long ldb;
    int grad;            // a ShardGrad
    float* out;          // X^(k+1), same layout (may be x: every kernel reads a row before it writes it)
    long long n;         // local rows (nodes of this shard)
    long long n_total;   // nodes of the whole problem
    long long row0;      // global index of local row 0 (second counter word of the generator)
    long long d, ld;
    long long Q;         // column groups of four: ceil(d / 4); exchange buffers have rows of 4 Q floats
    uint32_t q_base;     // global index of local group 0 (column offset / 4)
    uint32_t k;          // iteration index
    float gamma, sigma;
    PhiloxKeys keys;
};

// export: half-step rows first, first + stride, ... (rows of them) into the dense send buffer
cudaError_t launch_shard_export_rows(const ShardParams& p, bool vec, float* send, int first, int stride, int rows,
                                     cudaStream_t s);
// export: the shard's column sums of the half-step (4 Q doubles)
cudaError_t launch_shard_export_sums(const ShardParams& p, bool vec, double* sums, cudaStream_t s);
// export with the send fused in: row t to dst0 row t (t < split) or dst1 row t - split, and to
// `keep` when it is not null; dst0 / dst1 may be peer-mapped memory of another device
cudaError_t launch_shard_export_rows_to(const ShardParams& p, bool vec, float* keep, float* dst0, float* dst1, int split,
                                        int first, int stride, int rows, cudaStream_t s);
// export: the column sums into `count` gather areas (every shard's, possibly peer-mapped)
constexpr int kShardMaxDirect = 32;   // shards that one kernel can store its column sums to
struct ShardSumDests {
    double* dst[kShardMaxDirect];
    int count;
};
cudaError_t launch_shard_export_sums_to(const ShardParams& p, bool vec, const ShardSumDests& dl, cudaStream_t s);
// Which rows a gossip step kernel writes: all of them, only those whose neighbours are all local
// (so that they can be formed while the messages are still travelling), or only the others.
enum ShardPart { SHARD_ALL = 0, SHARD_INTERIOR = 1, SHARD_BOUNDARY = 2 };
// step: ring with recv = [row above local row 0 | row below the last local row]
cudaError_t launch_shard_ring(const ShardParams& p, bool vec, const float* recv, int part, cudaStream_t s);
// step: one-peer exponential graph, he = min(hop, local rows); recv = the partner shard's rows 0 .. he-1
cudaError_t launch_shard_exp(const ShardParams& p, bool vec, const float* recv, int he, int part, cudaStream_t s);
// step: the same when hop >= local rows and `own` still holds this shard's exported half-step rows
cudaError_t launch_shard_exp_exported(const ShardParams& p, bool vec, const float* own, const float* recv, cudaStream_t s);
// step: global average from `parts` vectors of column sums in shard order
cudaError_t launch_shard_global(const ShardParams& p, bool vec, const double* recv, int parts, cudaStream_t s);

}  // namespace gpga
