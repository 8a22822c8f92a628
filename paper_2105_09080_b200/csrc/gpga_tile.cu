// Generic gossip step through a shared-memory tile of the half-step matrix Y.
//
// For topologies whose neighbour sets do not reduce to a sliding window (torus grid,
// static exponential graph) or that need no mixing at all (W = I), a block computes
// Y for all n rows of a strip of column groups once (each X, b element read once,
// each noise sample generated once), parks it in shared memory, and then forms
// x_i^(k+1) = sum_{j in N_i} w_ij y_j (Algorithm 1, gossip step) from the tile.
#include "../../include/gpga.h"
#include "gpga_kernels.cuh"

namespace gpga {

constexpr int kTileBlock = 256;
constexpr int kTileSmemBytes = 64 * 1024;

template <int MODE, bool VEC>
__device__ __forceinline__ float4 tile_half_step(const StepParams& p, long long i, long long q)
{
    const long long j0 = q * 4;
    const float4 x = load4<VEC>(p.x + i * p.ld, j0, p.d);
    const float4 b = load4<VEC>(p.b + i * p.ldb, j0, p.d);
    float4 g;
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
__global__ void __launch_bounds__(kTileBlock) step_tile_kernel(const StepParams p, int topology,
                                                               int tile_groups, int log2n)
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
        float w = 1.0f;
        if (topology == GPGA_TOPO_GRID) {
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
            w = 0.2f;
        } else if (topology == GPGA_TOPO_STATIC_EXP) {
            for (int t = 0; t < log2n; ++t)
                acc4(s, ytile[((i + (1 << t)) & (n - 1)) * tile_groups + g]);
            w = 1.0f / (float)(log2n + 1);
        }
        s.x *= w;
        s.y *= w;
        s.z *= w;
        s.w *= w;
        store4<VEC>(p.out + (long long)i * p.ld, q * 4, p.d, s);
    }
}

cudaError_t launch_step_tile(const StepParams& p, int mode, bool vec, int topology, cudaStream_t s)
{
    int tile_groups = kTileSmemBytes / 16 / (int)p.n;
    if (tile_groups < 1) return cudaErrorInvalidConfiguration;   // callers bound n
    if (tile_groups > 64) tile_groups = 64;
    if ((long long)tile_groups > p.Q) tile_groups = (int)p.Q;
    int log2n = 0;
    while ((1LL << (log2n + 1)) <= p.n) ++log2n;
    const unsigned grd = (unsigned)((p.Q + tile_groups - 1) / tile_groups);
    const size_t smem = (size_t)p.n * tile_groups * 16;
#define GPGA_TILE(M, V)                                                                          \
    do {                                                                                         \
        cudaError_t e = cudaFuncSetAttribute(step_tile_kernel<M, V>,                             \
                                             cudaFuncAttributeMaxDynamicSharedMemorySize,        \
                                             kTileSmemBytes);                                    \
        if (e != cudaSuccess) return e;                                                          \
        step_tile_kernel<M, V><<<grd, kTileBlock, smem, s>>>(p, topology, tile_groups, log2n);   \
    } while (0)
    if (vec) {
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
