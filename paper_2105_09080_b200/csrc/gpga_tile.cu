// Gossip step through a shared-memory tile of the half-step matrix Y.
//
// A block computes Y = X - gamma G (Algorithm 1's local update) for all n rows of a
// strip of column groups once -- each X, b element read once, each noise sample
// generated once -- parks it in shared memory, and then forms
// x_i^(k+1) = sum_{j in N_i} w_ij y_j (gossip step) or the column mean (global average)
// from the tile.  Threads are spread over (row, column group) cells, so the kernel has
// n times more parallelism than the row-streaming kernels.  It serves
//  - topologies whose neighbour sets are not a sliding window (torus grid, static
//    exponential graph) and W = I, at any width;
//  - every topology when d is so small that one thread per column group would leave
//    the GPU idle (the logistic workload: d = 1024).
#include "../../include/gpga.h"
#include "gpga_kernels.cuh"
#include "gpga_launch.cuh"

namespace gpga {

constexpr int kTileBlock = 256;
constexpr int kTileSmemBytes = 64 * 1024;

template <int MODE, bool VEC>
__device__ __forceinline__ float4 tile_half_step(const StepParams& p, int i, long long q)
{
    const long long j0 = q * 4;
    const float4 x = load4<VEC>(p.x + (long long)i * p.ld, j0, p.d);
    float4 g;
    if (MODE == GRAD_PARTIALS) {
        // g = (1/B) sum_c partial[c][i][:] + l2 x, chunks added in index order
        const long long stride = p.n * p.d;
        const float* part = p.b + (long long)i * p.d + j0;
        g = *reinterpret_cast<const float4*>(part);
        for (int c = 1; c < p.chunks; ++c) {
            const float4 v = *reinterpret_cast<const float4*>(part + c * stride);
            g.x += v.x;
            g.y += v.y;
            g.z += v.z;
            g.w += v.w;
        }
        g = make_float4(fmaf(g.x, p.inv_batch, p.l2 * x.x), fmaf(g.y, p.inv_batch, p.l2 * x.y),
                        fmaf(g.z, p.inv_batch, p.l2 * x.z), fmaf(g.w, p.inv_batch, p.l2 * x.w));
    } else {
        const float4 b = load4<VEC>(p.b + (long long)i * p.ldb, j0, p.d);
        if (MODE == GRAD_BUFFER) {
            g = b;
        } else {
            g = make_float4(x.x - b.x, x.y - b.y, x.z - b.z, x.w - b.w);
            if (MODE == GRAD_QUAD_NOISE) {
                const float4 z = normal4(p.q_base + (uint32_t)q, (uint32_t)i, p.k, 0u, p.keys);
                g.x = fmaf(p.sigma, z.x, g.x);
                g.y = fmaf(p.sigma, z.y, g.y);
                g.z = fmaf(p.sigma, z.z, g.z);
                g.w = fmaf(p.sigma, z.w, g.w);
            }
        }
    }
    return make_float4(fmaf(-p.gamma, g.x, x.x), fmaf(-p.gamma, g.y, x.y), fmaf(-p.gamma, g.z, x.z),
                       fmaf(-p.gamma, g.w, x.w));
}

__device__ __forceinline__ void acc4(float4& s, const float4 v)
{
    s.x += v.x;
    s.y += v.y;
    s.z += v.z;
    s.w += v.w;
}

template <int MODE, bool VEC>
__global__ void __launch_bounds__(kTileBlock) step_tile_kernel(const StepParams p, int mix, int tile_groups,
                                                               int log2n)
{
    extern __shared__ float4 ytile[];   // [n][tile_groups]
    const long long q_first = (long long)blockIdx.x * tile_groups;
    const int n = (int)p.n;
    const int cells = n * tile_groups;
    for (int c = threadIdx.x; c < cells; c += blockDim.x) {
        const int i = c / tile_groups, g = c - i * tile_groups;
        const long long q = q_first + g;
        if (q < p.Q) ytile[c] = tile_half_step<MODE, VEC>(p, i, q);
    }
    __syncthreads();
    for (int c = threadIdx.x; c < cells; c += blockDim.x) {
        const int i = c / tile_groups, g = c - i * tile_groups;
        const long long q = q_first + g;
        if (q >= p.Q) continue;
        float4 s = ytile[c];
        if (mix == TILE_MIX_GLOBAL) {
            // the same fp64 sum in the same order for every row: rows come out bit-identical
            double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
            for (int r = 0; r < n; ++r) {
                const float4 v = ytile[r * tile_groups + g];
                s0 += (double)v.x;
                s1 += (double)v.y;
                s2 += (double)v.z;
                s3 += (double)v.w;
            }
            const double dn = (double)n;
            s = make_float4((float)(s0 / dn), (float)(s1 / dn), (float)(s2 / dn), (float)(s3 / dn));
        } else if (mix == GPGA_TOPO_RING) {
            const float4 up = ytile[(i == 0 ? n - 1 : i - 1) * tile_groups + g];
            const float4 dn = ytile[(i == n - 1 ? 0 : i + 1) * tile_groups + g];
            const float third = 0.333333343f;
            s = make_float4((up.x + s.x + dn.x) * third, (up.y + s.y + dn.y) * third,
                            (up.z + s.z + dn.z) * third, (up.w + s.w + dn.w) * third);
        } else if (mix == GPGA_TOPO_EXP) {
            const float4 peer = ytile[((i + (1 << p.hop_log2)) & (n - 1)) * tile_groups + g];
            s = make_float4((s.x + peer.x) * 0.5f, (s.y + peer.y) * 0.5f, (s.z + peer.z) * 0.5f,
                            (s.w + peer.w) * 0.5f);
        } else if (mix == GPGA_TOPO_GRID) {
            const int cols = p.grid_cols, rows = n / cols;
            const int a = i / cols, b = i - a * cols;
            const int up = (a == 0 ? rows - 1 : a - 1) * cols + b;
            const int dn = (a == rows - 1 ? 0 : a + 1) * cols + b;
            const int lf = a * cols + (b == 0 ? cols - 1 : b - 1);
            const int rt = a * cols + (b == cols - 1 ? 0 : b + 1);
            acc4(s, ytile[up * tile_groups + g]);
            acc4(s, ytile[lf * tile_groups + g]);
            acc4(s, ytile[rt * tile_groups + g]);
            acc4(s, ytile[dn * tile_groups + g]);
            s = make_float4(s.x * 0.2f, s.y * 0.2f, s.z * 0.2f, s.w * 0.2f);
        } else if (mix == GPGA_TOPO_STATIC_EXP) {
            for (int t = 0; t < log2n; ++t) acc4(s, ytile[((i + (1 << t)) & (n - 1)) * tile_groups + g]);
            const float w = 1.0f / (float)(log2n + 1);
            s = make_float4(s.x * w, s.y * w, s.z * w, s.w * w);
        }   // GPGA_TOPO_NONE: W = I
        store4<VEC>(p.out + (long long)i * p.ld, q * 4, p.d, s);
    }
}

bool tile_supports(long long n) { return n * 16 <= kTileSmemBytes; }

cudaError_t launch_step_tile(const StepParams& p, int mode, bool vec, int mix, cudaStream_t s)
{
    if (!tile_supports(p.n)) return cudaErrorInvalidConfiguration;   // callers bound n
    // strip width: enough blocks to cover the SMs, at most 64 groups, at most 64 KB of tile
    long long tg = (p.Q + 2 * 148 - 1) / (2 * 148);
    if (tg < 2) tg = 2;
    if (tg > 64) tg = 64;
    if (tg > kTileSmemBytes / 16 / p.n) tg = kTileSmemBytes / 16 / p.n;
    if (tg > p.Q) tg = p.Q;
    const int tile_groups = (int)tg;
    int log2n = 0;
    while ((1LL << (log2n + 1)) <= p.n) ++log2n;
    const unsigned grd = (unsigned)((p.Q + tile_groups - 1) / tile_groups);
    const size_t smem = (size_t)p.n * tile_groups * 16;
    long long cells = p.n * tile_groups;
    const int blk = cells >= kTileBlock ? kTileBlock : (int)((cells + 31) / 32 * 32);
#define GPGA_TILE(M, V)                                                                          \
    do {                                                                                         \
        static unsigned long long limit_set = 0;                                                 \
        cudaError_t e = ensure_smem_limit(step_tile_kernel<M, V>, kTileSmemBytes, limit_set);    \
        if (e != cudaSuccess) return e;                                                          \
        step_tile_kernel<M, V><<<grd, blk, smem, s>>>(p, mix, tile_groups, log2n);               \
    } while (0)
    if (mode == GRAD_PARTIALS) {
        GPGA_TILE(GRAD_PARTIALS, true);   // logistic objective: d % 4 == 0 is required upstream
    } else if (vec) {
        if (mode == GRAD_QUAD) GPGA_TILE(GRAD_QUAD, true);
        else if (mode == GRAD_QUAD_NOISE) GPGA_TILE(GRAD_QUAD_NOISE, true);
        else GPGA_TILE(GRAD_BUFFER, true);
    } else {
        if (mode == GRAD_QUAD) GPGA_TILE(GRAD_QUAD, false);
        else if (mode == GRAD_QUAD_NOISE) GPGA_TILE(GRAD_QUAD_NOISE, false);
        else GPGA_TILE(GRAD_BUFFER, false);
    }
#undef GPGA_TILE
    return cudaGetLastError();
}

}  // namespace gpga
