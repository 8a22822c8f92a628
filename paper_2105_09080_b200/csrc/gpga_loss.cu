// Global loss f(xbar) = (1/n) sum_i f_i(xbar) of problem (1) at the node average
// xbar = (1/n) sum_i x_i -- the quantity the paper's convergence plots track.
// Diagnostics, off the iteration's hot path; every sum is accumulated in fp64 and
// reduced in a fixed order.
#include "gpga_loss.cuh"

#include "gpga_kernels.cuh"
#include "gpga_launch.cuh"

namespace gpga {

constexpr int kLossBlock = 256;

// ---- quadratic: per column, the mean over rows of x, then sum_i (mean - b_i)^2 ----
template <bool VEC>
__global__ void __launch_bounds__(kLossBlock) quadratic_global_loss_kernel(const float* __restrict__ x,
                                                                           const float* __restrict__ b,
                                                                           long long n, long long d, long long ld,
                                                                           long long Q, double* __restrict__ partials)
{
    double acc = 0.0;
    for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < Q;
         q += (long long)gridDim.x * blockDim.x) {
        const long long j0 = q * 4;
        double m0 = 0.0, m1 = 0.0, m2 = 0.0, m3 = 0.0;
#pragma unroll 4
        for (long long i = 0; i < n; ++i) {
            const float4 v = load4<VEC>(x + i * ld, j0, d);
            m0 += (double)v.x;
            m1 += (double)v.y;
            m2 += (double)v.z;
            m3 += (double)v.w;
        }
        const double inv = 1.0 / (double)n;
        m0 *= inv; m1 *= inv; m2 *= inv; m3 *= inv;
        const bool in0 = j0 + 0 < d, in1 = j0 + 1 < d, in2 = j0 + 2 < d, in3 = j0 + 3 < d;
#pragma unroll 4
        for (long long i = 0; i < n; ++i) {
            const float4 v = load4<VEC>(b + i * ld, j0, d);
            const double r0 = m0 - (double)v.x, r1 = m1 - (double)v.y, r2 = m2 - (double)v.z, r3 = m3 - (double)v.w;
            if (in0) acc = fma(r0, r0, acc);
            if (in1) acc = fma(r1, r1, acc);
            if (in2) acc = fma(r2, r2, acc);
            if (in3) acc = fma(r3, r3, acc);
        }
    }
    acc = block_sum(acc);
    if (threadIdx.x == 0) partials[blockIdx.x] = acc;
}

__global__ void loss_final_kernel(const double* __restrict__ partials, int count, double scale,
                                  const float* __restrict__ xbar, int d, double half_l2, double* __restrict__ result)
{
    double v = 0.0;
    for (int t = threadIdx.x; t < count; t += 32) v += partials[t];
    v = warp_sum(v) * scale;
    double reg = 0.0;
    if (xbar) {
        for (int j = threadIdx.x; j < d; j += 32) reg = fma((double)xbar[j], (double)xbar[j], reg);
        reg = warp_sum(reg);
    }
    if (threadIdx.x == 0) *result = v + half_l2 * reg;
}

cudaError_t launch_quadratic_global_loss(const float* x, const float* b, long long n, long long d, long long ld,
                                         bool vec, double* partials, double* result, cudaStream_t s)
{
    const long long Q = (d + 3) / 4;
    const int blocks = reduce_blocks(Q);
    if (vec)
        quadratic_global_loss_kernel<true><<<blocks, kLossBlock, 0, s>>>(x, b, n, d, ld, Q, partials);
    else
        quadratic_global_loss_kernel<false><<<blocks, kLossBlock, 0, s>>>(x, b, n, d, ld, Q, partials);
    loss_final_kernel<<<1, 32, 0, s>>>(partials, blocks, 0.5 / (double)n, nullptr, 0, 0.0, result);
    return cudaGetLastError();
}

// ---- logistic ----
__global__ void __launch_bounds__(kLossBlock) column_mean_kernel(const float* __restrict__ x, long long ldx,
                                                                 long long n, long long d, float* __restrict__ xbar)
{
    const long long j = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= d) return;
    double s = 0.0;
    for (long long i = 0; i < n; ++i) s += (double)x[i * ldx + j];
    xbar[j] = (float)(s / (double)n);
}

// Block (i, c) sums ln(1 + exp(-y a^T xbar)) over rows [c * rows_per_block, ...) of node i:
// one warp per row, fp32 dot product against xbar in shared memory, fp64 loss sum.
__global__ void __launch_bounds__(kLossBlock) logistic_full_loss_kernel(const float* __restrict__ A,
                                                                        const float* __restrict__ y,
                                                                        const float* __restrict__ xbar, long long d,
                                                                        long long m, int rows_per_block,
                                                                        double* __restrict__ partials)
{
    extern __shared__ float xs[];
    const int i = blockIdx.x, c = blockIdx.y;
    for (int j = threadIdx.x; j < d; j += blockDim.x) xs[j] = xbar[j];
    __syncthreads();
    const float* Ai = A + (long long)i * m * d;
    const float* yi = y + (long long)i * m;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const long long r_begin = (long long)c * rows_per_block;
    long long r_end = r_begin + rows_per_block;
    if (r_end > m) r_end = m;
    const int d4 = (int)(d >> 2);
    double acc = 0.0;
    for (long long r = r_begin + warp; r < r_end; r += nwarps) {
        const float4* a4 = reinterpret_cast<const float4*>(Ai + r * d);
        float z = 0.f;
#pragma unroll 4
        for (int g = lane; g < d4; g += 32) {
            const float4 a = __ldg(a4 + g);
            const float4 xv = reinterpret_cast<const float4*>(xs)[g];
            z = fmaf(a.x, xv.x, z);
            z = fmaf(a.y, xv.y, z);
            z = fmaf(a.z, xv.z, z);
            z = fmaf(a.w, xv.w, z);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xFFFFFFFFu, z, o);
        if (lane == 0) {
            const double u = -(double)yi[r] * (double)z;
            acc += (u > 0.0) ? u + log1p(exp(-u)) : log1p(exp(u));
        }
    }
    acc = block_sum(acc);
    if (threadIdx.x == 0) partials[(long long)i * gridDim.y + c] = acc;
}

cudaError_t launch_logistic_global_loss(const float* A, const float* y, const float* x, long long ldx, long long n,
                                        long long d, long long m, float l2, float* xbar, double* partials,
                                        long long slots, double* result, cudaStream_t s)
{
    column_mean_kernel<<<(unsigned)((d + kLossBlock - 1) / kLossBlock), kLossBlock, 0, s>>>(x, ldx, n, d, xbar);
    long long chunks = slots / n;                       // partial slots available per node
    const long long want = (m + 63) / 64;                // at least 64 rows per block
    if (chunks > want) chunks = want;
    if (chunks < 1) chunks = 1;
    if (chunks > 65535) chunks = 65535;
    const int rows_per_block = (int)((m + chunks - 1) / chunks);
    chunks = (m + rows_per_block - 1) / rows_per_block;
    if ((size_t)d * sizeof(float) > 48 * 1024) {   // xbar in shared memory beyond the default limit
        static unsigned long long limit_set = 0;
        cudaError_t e = ensure_smem_limit(logistic_full_loss_kernel, 200 * 1024, limit_set);
        if (e != cudaSuccess) return e;
    }
    logistic_full_loss_kernel<<<dim3((unsigned)n, (unsigned)chunks), kLossBlock, (size_t)d * sizeof(float), s>>>(
        A, y, xbar, d, m, rows_per_block, partials);
    loss_final_kernel<<<1, 32, 0, s>>>(partials, (int)(n * chunks), 1.0 / ((double)n * (double)m), xbar, (int)d,
                                       0.5 * (double)l2, result);
    return cudaGetLastError();
}

// ---- node shards: diagnostics of the WHOLE problem from the shards' parts ---------------------
// The shards exchange the fp64 column sums of their rows (shard_state_sums_kernel, gathered in shard
// order like the column sums of a global average); with them every shard forms the mean over all
// nodes, xbar = (sum of the parts) / n_total, column by column, and its own part of
//   the consensus distance  sum_{i local} ||x_i - xbar||^2                     (Section 4)
//   the global loss         (1 / n_total) sum_{i local} f_i(xbar)              (problem (1))
// whose sums over the shards are the whole problem's values.
template <bool VEC>
__global__ void __launch_bounds__(kLossBlock) shard_state_sums_kernel(const float* __restrict__ x, long long n,
                                                                      long long d, long long ld, long long Q,
                                                                      double* __restrict__ sums)
{
    const long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= Q) return;
    double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
#pragma unroll 4
    for (long long i = 0; i < n; ++i) {
        const float4 v = load4<VEC>(x + i * ld, q * 4, d);
        s0 += (double)v.x; s1 += (double)v.y; s2 += (double)v.z; s3 += (double)v.w;
    }
    double* o = sums + 4 * q;
    o[0] = s0; o[1] = s1; o[2] = s2; o[3] = s3;
}

__device__ __forceinline__ void shard_mean4(const double* __restrict__ gathered, int parts, long long Q, long long q,
                                            double inv_n, double m[4])
{
    double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
    for (int t = 0; t < parts; ++t) {   // shard order
        const double* v = gathered + ((long long)t * Q + q) * 4;
        s0 += v[0]; s1 += v[1]; s2 += v[2]; s3 += v[3];
    }
    m[0] = s0 * inv_n; m[1] = s1 * inv_n; m[2] = s2 * inv_n; m[3] = s3 * inv_n;
}

// WHAT = 0: sum over the local rows of (x_ij - xbar_j)^2; WHAT = 1: of (xbar_j - b_ij)^2 (rows = b).
template <bool VEC, int WHAT>
__global__ void __launch_bounds__(kLossBlock) shard_square_part_kernel(const float* __restrict__ rows, long long n,
                                                                       long long d, long long ld, long long Q,
                                                                       const double* __restrict__ gathered, int parts,
                                                                       double inv_n, double* __restrict__ partials)
{
    double acc = 0.0;
    for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < Q;
         q += (long long)gridDim.x * blockDim.x) {
        const long long j0 = q * 4;
        double m[4];
        shard_mean4(gathered, parts, Q, q, inv_n, m);
        const bool in0 = j0 + 0 < d, in1 = j0 + 1 < d, in2 = j0 + 2 < d, in3 = j0 + 3 < d;
#pragma unroll 4
        for (long long i = 0; i < n; ++i) {
            const float4 v = load4<VEC>(rows + i * ld, j0, d);
            const double r0 = m[0] - (double)v.x, r1 = m[1] - (double)v.y, r2 = m[2] - (double)v.z, r3 = m[3] - (double)v.w;
            if (in0) acc = fma(r0, r0, acc);
            if (in1) acc = fma(r1, r1, acc);
            if (in2) acc = fma(r2, r2, acc);
            if (in3) acc = fma(r3, r3, acc);
        }
    }
    acc = block_sum(acc);
    if (threadIdx.x == 0) partials[blockIdx.x] = acc;
}

// xbar as fp32 (the logistic loss takes its margins in fp32, like the unsharded diagnostic)
__global__ void __launch_bounds__(kLossBlock) shard_xbar_kernel(const double* __restrict__ gathered, int parts, long long Q,
                                                                long long d, double inv_n, float* __restrict__ xbar)
{
    const long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= Q) return;
    double m[4];
    shard_mean4(gathered, parts, Q, q, inv_n, m);
    for (int t = 0; t < 4; ++t)
        if (q * 4 + t < d) xbar[q * 4 + t] = (float)m[t];
}

cudaError_t launch_shard_state_sums(const float* x, long long n, long long d, long long ld, bool vec, double* sums,
                                    cudaStream_t s)
{
    const long long Q = (d + 3) / 4;
    const unsigned grd = (unsigned)((Q + kLossBlock - 1) / kLossBlock);
    if (vec)
        shard_state_sums_kernel<true><<<grd, kLossBlock, 0, s>>>(x, n, d, ld, Q, sums);
    else
        shard_state_sums_kernel<false><<<grd, kLossBlock, 0, s>>>(x, n, d, ld, Q, sums);
    return cudaGetLastError();
}

cudaError_t launch_shard_consensus_part(const float* x, long long n, long long d, long long ld, bool vec,
                                        const double* gathered, int parts, long long n_total, double* partials,
                                        double* result, cudaStream_t s)
{
    const long long Q = (d + 3) / 4;
    const int blocks = reduce_blocks(Q);
    const double inv_n = 1.0 / (double)n_total;
    if (vec)
        shard_square_part_kernel<true, 0><<<blocks, kLossBlock, 0, s>>>(x, n, d, ld, Q, gathered, parts, inv_n, partials);
    else
        shard_square_part_kernel<false, 0><<<blocks, kLossBlock, 0, s>>>(x, n, d, ld, Q, gathered, parts, inv_n, partials);
    loss_final_kernel<<<1, 32, 0, s>>>(partials, blocks, 1.0, nullptr, 0, 0.0, result);
    return cudaGetLastError();
}

cudaError_t launch_shard_quadratic_loss_part(const float* b, long long n, long long d, long long ld, bool vec,
                                             const double* gathered, int parts, long long n_total, double* partials,
                                             double* result, cudaStream_t s)
{
    const long long Q = (d + 3) / 4;
    const int blocks = reduce_blocks(Q);
    const double inv_n = 1.0 / (double)n_total;
    if (vec)
        shard_square_part_kernel<true, 1><<<blocks, kLossBlock, 0, s>>>(b, n, d, ld, Q, gathered, parts, inv_n, partials);
    else
        shard_square_part_kernel<false, 1><<<blocks, kLossBlock, 0, s>>>(b, n, d, ld, Q, gathered, parts, inv_n, partials);
    loss_final_kernel<<<1, 32, 0, s>>>(partials, blocks, 0.5 * inv_n, nullptr, 0, 0.0, result);
    return cudaGetLastError();
}

cudaError_t launch_shard_logistic_loss_part(const float* A, const float* y, long long n, long long d, long long m, float l2,
                                            const double* gathered, int parts, long long n_total, float* xbar,
                                            double* partials, long long slots, double* result, cudaStream_t s)
{
    const long long Q = (d + 3) / 4;
    const double inv_n = 1.0 / (double)n_total;
    shard_xbar_kernel<<<(unsigned)((Q + kLossBlock - 1) / kLossBlock), kLossBlock, 0, s>>>(gathered, parts, Q, d, inv_n, xbar);
    long long chunks = slots / n;
    const long long want = (m + 63) / 64;
    if (chunks > want) chunks = want;
    if (chunks < 1) chunks = 1;
    if (chunks > 65535) chunks = 65535;
    const int rows_per_block = (int)((m + chunks - 1) / chunks);
    chunks = (m + rows_per_block - 1) / rows_per_block;
    if ((size_t)d * sizeof(float) > 48 * 1024) {
        static unsigned long long limit_set = 0;
        cudaError_t e = ensure_smem_limit(logistic_full_loss_kernel, 200 * 1024, limit_set);
        if (e != cudaSuccess) return e;
    }
    logistic_full_loss_kernel<<<dim3((unsigned)n, (unsigned)chunks), kLossBlock, (size_t)d * sizeof(float), s>>>(
        A, y, xbar, d, m, rows_per_block, partials);
    // the local nodes' share of (1 / n_total) sum_i f_i(xbar): their data terms and n / n_total of the regulariser
    loss_final_kernel<<<1, 32, 0, s>>>(partials, (int)(n * chunks), inv_n / (double)m, xbar, (int)d,
                                       0.5 * (double)l2 * (double)n * inv_n, result);
    return cudaGetLastError();
}

}  // namespace gpga
