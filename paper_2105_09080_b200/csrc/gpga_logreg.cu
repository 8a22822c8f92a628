// Per-node mini-batch logistic-regression gradient (Section 5.1 loss with an l2 term):
//   f_i(x) = (1/m) sum_r ln(1 + exp(-y_r a_r^T x)) + (l2/2) ||x||^2
//   g_i    = -(1/B) sum_{r in batch} y_r a_r / (1 + exp(y_r a_r^T x_i)) + l2 x_i
// The B rows of node i at iteration k are drawn with replacement from the generator
// (stream BATCH).  The batch is cut into chunks of kChunkRows rows; block (i, c) forms
// the margins of its rows (one warp per row, shuffle reduction) and then its partial
// sum over those rows; a second kernel adds the chunks in a fixed order, so the result
// does not depend on scheduling.
#include "gpga_logreg.cuh"

namespace gpga {

constexpr int kLrBlock = 256;

__device__ __forceinline__ uint32_t batch_row(uint32_t t, uint32_t i, uint32_t k, uint32_t m,
                                              const PhiloxKeys& ks)
{
    const uint4 w = philox4x32_10(t >> 2, i, k, 4u, ks);
    const uint32_t sel = t & 3u;
    const uint32_t word = sel == 0 ? w.x : sel == 1 ? w.y : sel == 2 ? w.z : w.w;
    return word % m;
}

__device__ __forceinline__ float warp_sum_f(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// partial[c][i][:] = sum over the chunk's rows of s_r a_r,  s_r = -y_r / (1 + exp(y_r z_r)).
__global__ void __launch_bounds__(kLrBlock) logreg_partial_kernel(const LogregParams p)
{
    extern __shared__ float smem[];
    float* xs = smem;                          // d floats: x_i
    float* coef = smem + p.d;                  // kChunkRows floats: s_r
    __shared__ uint32_t rows[kChunkRows];
    const int i = blockIdx.x, c = blockIdx.y;
    const int t0 = c * kChunkRows;
    const int nrows = min(kChunkRows, (int)p.batch - t0);
    const float* A = p.A + (long long)i * p.m * p.d;
    const float* y = p.y + (long long)i * p.m;
    const float* x = p.x + (long long)i * p.ldx;
    for (int j = threadIdx.x; j < p.d; j += blockDim.x) xs[j] = x[j];
    if (threadIdx.x < nrows)
        rows[threadIdx.x] = batch_row((uint32_t)(t0 + threadIdx.x), (uint32_t)i, p.k, (uint32_t)p.m, p.keys);
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int d4 = (int)(p.d >> 2);
    // margins: a warp takes two rows at a time so that both rows' loads are in flight together
    for (int t = warp; t < nrows; t += 2 * nwarps) {
        const int t2 = t + nwarps;
        const bool two = t2 < nrows;
        const float4* a4 = reinterpret_cast<const float4*>(A + (long long)rows[t] * p.d);
        const float4* b4 = reinterpret_cast<const float4*>(A + (long long)rows[two ? t2 : t] * p.d);
        float z = 0.f, z2 = 0.f;
#pragma unroll 4
        for (int g = lane; g < d4; g += 32) {
            const float4 a = __ldg(a4 + g);
            const float4 b = __ldg(b4 + g);
            const float4 xv = reinterpret_cast<const float4*>(xs)[g];
            z = fmaf(a.x, xv.x, z);
            z = fmaf(a.y, xv.y, z);
            z = fmaf(a.z, xv.z, z);
            z = fmaf(a.w, xv.w, z);
            z2 = fmaf(b.x, xv.x, z2);
            z2 = fmaf(b.y, xv.y, z2);
            z2 = fmaf(b.z, xv.z, z2);
            z2 = fmaf(b.w, xv.w, z2);
        }
        z = warp_sum_f(z);
        z2 = warp_sum_f(z2);
        if (lane == 0) {
            const float yr = y[rows[t]];
            coef[t] = -yr / (1.0f + expf(yr * z));
            if (two) {
                const float yr2 = y[rows[t2]];
                coef[t2] = -yr2 / (1.0f + expf(yr2 * z2));
            }
        }
    }
    __syncthreads();
    float4* out4 = reinterpret_cast<float4*>(p.partial + ((long long)c * p.n + i) * p.d);
    for (int g = threadIdx.x; g < d4; g += blockDim.x) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
        for (int t = 0; t < nrows; ++t) {
            const float4 a = __ldg(reinterpret_cast<const float4*>(A + (long long)rows[t] * p.d) + g);
            const float s = coef[t];
            acc.x = fmaf(s, a.x, acc.x);
            acc.y = fmaf(s, a.y, acc.y);
            acc.z = fmaf(s, a.z, acc.z);
            acc.w = fmaf(s, a.w, acc.w);
        }
        out4[g] = acc;
    }
}

// G[i][:] = (1/B) sum_c partial[c][i][:] + l2 x_i, chunks added in index order.
__global__ void __launch_bounds__(kLrBlock) logreg_reduce_kernel(const LogregParams p, int chunks)
{
    const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long d4 = p.d >> 2;
    const long long total4 = p.n * d4;
    if (e >= total4) return;
    const long long row = e / d4, g = e - row * d4;
    const float4* part = reinterpret_cast<const float4*>(p.partial);
    float4 acc = part[e];
    for (int c = 1; c < chunks; ++c) {
        const float4 v = part[(long long)c * total4 + e];
        acc.x += v.x;
        acc.y += v.y;
        acc.z += v.z;
        acc.w += v.w;
    }
    const float4 xv = reinterpret_cast<const float4*>(p.x + row * p.ldx)[g];
    const float inv = 1.0f / (float)p.batch;
    reinterpret_cast<float4*>(p.G)[e] =
        make_float4(fmaf(acc.x, inv, p.l2 * xv.x), fmaf(acc.y, inv, p.l2 * xv.y),
                    fmaf(acc.z, inv, p.l2 * xv.z), fmaf(acc.w, inv, p.l2 * xv.w));
}

// node_loss[i] = (1/B) sum_{r in batch} ln(1 + exp(-y_r a_r^T x_i)) + (l2/2)||x_i||^2 in fp64.
__global__ void __launch_bounds__(kLrBlock) logreg_loss_kernel(const LogregParams p, double* node_loss)
{
    const int i = blockIdx.x;
    const float* A = p.A + (long long)i * p.m * p.d;
    const float* y = p.y + (long long)i * p.m;
    const float* x = p.x + (long long)i * p.ldx;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    double acc = 0.0;
    for (int t = warp; t < (int)p.batch; t += nwarps) {
        const uint32_t r = batch_row((uint32_t)t, (uint32_t)i, p.k, (uint32_t)p.m, p.keys);
        double z = 0.0;
        for (int j = lane; j < (int)p.d; j += 32) z = fma((double)A[(long long)r * p.d + j], (double)x[j], z);
        z = warp_sum(z);
        if (lane == 0) {
            const double u = -(double)y[r] * z;
            acc += (u > 0.0) ? u + log1p(exp(-u)) : log1p(exp(u));
        }
    }
    double reg = 0.0;
    for (int j = threadIdx.x; j < (int)p.d; j += blockDim.x) reg = fma((double)x[j], (double)x[j], reg);
    const double total = block_sum(acc / (double)p.batch + 0.5 * (double)p.l2 * reg);
    if (threadIdx.x == 0) node_loss[i] = total;
}

__global__ void mean_kernel(const double* v, int count, double* result)
{
    double s = 0.0;
    for (int t = threadIdx.x; t < count; t += 32) s += v[t];
    s = warp_sum(s);
    if (threadIdx.x == 0) *result = s / (double)count;
}

int logreg_chunks(long long batch) { return (int)((batch + kChunkRows - 1) / kChunkRows); }

cudaError_t launch_logreg_partial(const LogregParams& p, cudaStream_t s)
{
    const int chunks = logreg_chunks(p.batch);
    const size_t smem = (size_t)(p.d + kChunkRows) * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(logreg_partial_kernel,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    logreg_partial_kernel<<<dim3((unsigned)p.n, (unsigned)chunks), kLrBlock, smem, s>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_logreg_grad(const LogregParams& p, cudaStream_t s)
{
    const int chunks = logreg_chunks(p.batch);
    cudaError_t e = launch_logreg_partial(p, s);
    if (e != cudaSuccess) return e;
    const long long total4 = p.n * (p.d >> 2);
    logreg_reduce_kernel<<<(unsigned)((total4 + kLrBlock - 1) / kLrBlock), kLrBlock, 0, s>>>(p, chunks);
    return cudaGetLastError();
}

cudaError_t launch_logreg_loss(const LogregParams& p, double* node_loss, double* result, cudaStream_t s)
{
    logreg_loss_kernel<<<(unsigned)p.n, kLrBlock, 0, s>>>(p, node_loss);
    mean_kernel<<<1, 32, 0, s>>>(node_loss, (int)p.n, result);
    return cudaGetLastError();
}

}  // namespace gpga
