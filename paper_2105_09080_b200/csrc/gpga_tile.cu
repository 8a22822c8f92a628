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
// A second kernel keeps the strip of X and b in shared memory across several
// iterations (columns evolve independently under the quadratic objective), for states
// so small that an iteration per launch is bound by launch latency, not by memory.
#include "../../include/gpga.h"
#include "gpga_kernels.cuh"
#include "gpga_launch.cuh"
#include "gpga_tile.cuh"

namespace gpga {

constexpr int kTileBlock = 256;
constexpr int kTileSmemBytes = 64 * 1024;

// y = x - gamma g for the quadratic objective (with or without noise) or a given gradient.
template <int MODE>
__device__ __forceinline__ float4 tile_finish(const StepParams& p, float4 x, float4 b, int i, long long q, uint32_t k)
{
    float4 g;
    if (MODE == GRAD_BUFFER) {
        g = b;
    } else {
        g = sub4(x, b);
        if (MODE == GRAD_QUAD_NOISE) g = fma4(p.sigma, normal4(p.q_base + (uint32_t)q, (uint32_t)i, k, 0u, p.keys), g);
    }
    return fma4(-p.gamma, g, x);
}

template <int MODE, bool VEC>
__device__ __forceinline__ float4 tile_half_step(const StepParams& p, int i, long long q)
{
    const long long j0 = q * 4;
    const float4 x = load4<VEC>(p.x + (long long)i * p.ld, j0, p.d);
    if (MODE == GRAD_PARTIALS) {
        // g = (1/B) sum_c partial[c][i][:] + l2 x, chunks added in index order
        const long long stride = p.n * p.d;
        const float* part = p.b + (long long)i * p.d + j0;
        float4 g = *reinterpret_cast<const float4*>(part);
        for (int c = 1; c < p.chunks; ++c) {
            const float4 v = *reinterpret_cast<const float4*>(part + c * stride);
            g.x += v.x;
            g.y += v.y;
            g.z += v.z;
            g.w += v.w;
        }
        g = make_float4(fmaf(g.x, p.inv_batch, p.l2 * x.x), fmaf(g.y, p.inv_batch, p.l2 * x.y),
                        fmaf(g.z, p.inv_batch, p.l2 * x.z), fmaf(g.w, p.inv_batch, p.l2 * x.w));
        return tile_finish<GRAD_BUFFER>(p, x, g, i, q, p.k);
    }
    const float4 b = load4<VEC>(p.b + (long long)i * p.ldb, j0, p.d);
    return tile_finish<MODE>(p, x, b, i, q, p.k);
}

__device__ __forceinline__ void acc4(float4& s, const float4 v) { s = add4(s, v); }

// x_i^(k+1) for cell (row i, group g) from the tile of Y.  `mix` is a GPGA_TOPO_* value or
// TILE_MIX_GLOBAL.
__device__ __forceinline__ float4 tile_mix(const float4* ytile, int i, int g, int n, int tile_groups, int mix,
                                           int hop_log2, int grid_cols, int log2n, const SparseW& sw)
{
    float4 s = ytile[i * tile_groups + g];
    if (mix == TILE_MIX_GLOBAL) {
        // the column mean exactly as the row-streaming kernel forms it: rows added pairwise in
        // fp32 in groups of four, group sums accumulated in fp64; the same sum in the same
        // order for every row, so the rows come out bit-identical
        double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
        int r = 0;
        for (; r + 4 <= n; r += 4) {
            float4 a = ytile[r * tile_groups + g], b = ytile[(r + 2) * tile_groups + g];
            acc4(a, ytile[(r + 1) * tile_groups + g]);
            acc4(b, ytile[(r + 3) * tile_groups + g]);
            acc4(a, b);
            s0 += (double)a.x;
            s1 += (double)a.y;
            s2 += (double)a.z;
            s3 += (double)a.w;
        }
        const int rest = n - r;
        if (rest >= 1) {
            float4 a = ytile[r * tile_groups + g];
            if (rest >= 2) acc4(a, ytile[(r + 1) * tile_groups + g]);
            s0 += (double)a.x;
            s1 += (double)a.y;
            s2 += (double)a.z;
            s3 += (double)a.w;
        }
        if (rest == 3) {
            const float4 b = ytile[(r + 2) * tile_groups + g];
            s0 += (double)b.x;
            s1 += (double)b.y;
            s2 += (double)b.z;
            s3 += (double)b.w;
        }
        if ((n & (n - 1)) == 0) {   // 1/n is exact: the product equals the quotient
            const double inv = 1.0 / (double)n;
            s = make_float4((float)(s0 * inv), (float)(s1 * inv), (float)(s2 * inv), (float)(s3 * inv));
        } else {
            const double dn = (double)n;
            s = make_float4((float)(s0 / dn), (float)(s1 / dn), (float)(s2 / dn), (float)(s3 / dn));
        }
    } else if (mix == GPGA_TOPO_RING) {
        const float4 up = ytile[(i == 0 ? n - 1 : i - 1) * tile_groups + g];
        const float4 dn = ytile[(i == n - 1 ? 0 : i + 1) * tile_groups + g];
        s = scale4(add4(add4(up, s), dn), 0.333333343f);
    } else if (mix == GPGA_TOPO_EXP) {
        const float4 peer = ytile[((i + (1 << hop_log2)) & (n - 1)) * tile_groups + g];
        s = scale4(add4(s, peer), 0.5f);
    } else if (mix == GPGA_TOPO_GRID) {
        const int cols = grid_cols, rows = n / cols;
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
    } else if (mix == GPGA_TOPO_SPARSE) {
        // x_i = sum_j w_ij y_j over the stored entries of row i, in storage order
        s = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int e = sw.row_ptr[i]; e < sw.row_ptr[i + 1]; ++e) {
            const float w = sw.w[e];
            const float4 v = ytile[sw.col[e] * tile_groups + g];
            s.x = fmaf(w, v.x, s.x);
            s.y = fmaf(w, v.y, s.y);
            s.z = fmaf(w, v.z, s.z);
            s.w = fmaf(w, v.w, s.w);
        }
    }   // GPGA_TOPO_NONE: W = I
    return s;
}

template <int MODE, bool VEC>
__global__ void __launch_bounds__(kTileBlock) step_tile_kernel(const StepParams p, int mix, int tile_groups,
                                                               int log2n, const SparseW sw)
{
    extern __shared__ float4 ytile[];   // [n][tile_groups]
    if (MODE == GRAD_PARTIALS) {
        // the next iteration's gradient kernel may start staging its rows of A beside this kernel;
        // this kernel itself may have been started before the gradient kernel it follows was done
        grid_launch_dependents();
        grid_dependency_wait();
    }
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
        const float4 s = tile_mix(ytile, i, g, n, tile_groups, mix, p.hop_log2, p.grid_cols, log2n, sw);
        store4<VEC>(p.out + (long long)i * p.ld, q * 4, p.d, s);
    }
}

// K iterations k0 .. k0+K-1 of Algorithm 1 on one strip of column groups, with the strip of
// X, b and Y resident in shared memory: X and b are read from global memory once and X written
// once for all K iterations.  Quadratic objective only (its columns are independent).  Each
// iteration does exactly what step_tile_kernel does, so the result is bit-identical to K
// single-iteration launches.
template <int MODE, bool VEC>
__global__ void __launch_bounds__(kTileBlock) run_tile_kernel(const StepParams p, int topology, long long H,
                                                              long long phase0, int hop0, int steps,
                                                              int tile_groups, int log2n, const SparseW sw)
{
    extern __shared__ float4 tile_smem[];   // X, b, Y: [n][tile_groups] each
    const int n = (int)p.n;
    const int cells = n * tile_groups;
    float4* xtile = tile_smem;
    float4* btile = tile_smem + cells;
    float4* ytile = tile_smem + 2 * cells;
    const long long q_first = (long long)blockIdx.x * tile_groups;
    for (int c = threadIdx.x; c < cells; c += blockDim.x) {
        const int i = c / tile_groups, g = c - i * tile_groups;
        const long long q = q_first + g;
        if (q < p.Q) {
            xtile[c] = load4<VEC>(p.x + (long long)i * p.ld, q * 4, p.d);
            btile[c] = load4<VEC>(p.b + (long long)i * p.ldb, q * 4, p.d);
        }
    }
    __syncthreads();
    // schedule counters kept incrementally (no division in the loop):
    // phase = (k + 1) mod H, global average when it is 0; hop_log2 = k mod log2(n)
    long long phase = phase0;
    int hop_log2 = hop0;
    // a thread's first cell, with its coordinates worked out once; further cells (strips with
    // more cells than threads) go through the generic loops
    const int c0 = threadIdx.x;
    const int i0 = c0 / tile_groups, g0 = c0 - i0 * tile_groups;
    const bool own0 = c0 < cells && q_first + g0 < p.Q;
    for (int t = 0; t < steps; ++t) {
        const uint32_t k = p.k + (uint32_t)t;
        const bool global = H > 0 && phase == 0;            // Algorithm 1's test mod(k + 1, H) = 0
        const int mix = global ? (int)TILE_MIX_GLOBAL : topology;
        if (own0) ytile[c0] = tile_finish<MODE>(p, xtile[c0], btile[c0], i0, q_first + g0, k);
        for (int c = c0 + blockDim.x; c < cells; c += blockDim.x) {
            const int i = c / tile_groups, g = c - i * tile_groups;
            const long long q = q_first + g;
            if (q < p.Q) ytile[c] = tile_finish<MODE>(p, xtile[c], btile[c], i, q, k);
        }
        __syncthreads();
        if (own0) xtile[c0] = tile_mix(ytile, i0, g0, n, tile_groups, mix, hop_log2, p.grid_cols, log2n, sw);
        for (int c = c0 + blockDim.x; c < cells; c += blockDim.x) {
            const int i = c / tile_groups, g = c - i * tile_groups;
            if (q_first + g < p.Q) xtile[c] = tile_mix(ytile, i, g, n, tile_groups, mix, hop_log2, p.grid_cols, log2n, sw);
        }
        __syncthreads();
        if (++phase >= H) phase = 0;
        if (++hop_log2 >= log2n) hop_log2 = 0;
    }
    for (int c = threadIdx.x; c < cells; c += blockDim.x) {
        const int i = c / tile_groups, g = c - i * tile_groups;
        const long long q = q_first + g;
        if (q < p.Q) store4<VEC>(p.out + (long long)i * p.ld, q * 4, p.d, xtile[c]);
    }
}

// The same K iterations for strips with at most one cell per thread (n * tile_groups <= block
// size): a thread keeps its cell's x and b in registers for the whole run, and only Y goes
// through shared memory, in two tiles used alternately so that one barrier per iteration is
// enough (a tile is rewritten two iterations later, and every thread passes the barrier in
// between only after its reads of it).  Same arithmetic per element as run_tile_kernel.
// TOPO: GPGA_TOPO_RING or GPGA_TOPO_EXP specialise the gossip mix (neighbour offsets formed once, the
// cell's own half-step taken from its register); -1 takes the general tile_mix.
template <int MODE, bool VEC, int TOPO>
__global__ void __launch_bounds__(kTileBlock) run_cell_kernel(const StepParams p, int topology, long long H,
                                                              long long phase0, int hop0, int steps,
                                                              int tile_groups, int log2n, const SparseW sw)
{
    extern __shared__ float4 tile_smem[];   // Y twice: [2][n][tile_groups], then the column-mean addends
    const int n = (int)p.n;
    const int cells = n * tile_groups;
    const long long q_first = (long long)blockIdx.x * tile_groups;
    const int c = threadIdx.x;
    const int i = c / tile_groups, g = c - i * tile_groups;
    const long long q = q_first + g;
    const bool own = c < cells && q < p.Q;
    float4 x = make_float4(0.f, 0.f, 0.f, 0.f), b = x;
    if (own) {
        x = load4<VEC>(p.x + (long long)i * p.ld, q * 4, p.d);
        b = load4<VEC>(p.b + (long long)i * p.ldb, q * 4, p.d);
    }
    // Iterations left until the next global average (phase0 = (k + 1) mod H of the first iteration, a
    // global average when it is 0), as 32-bit counters: a period beyond this launch's iterations is
    // cut to steps + 1, which the countdown cannot reach before the launch ends.
    const int period = H > 0 ? (int)(H < (long long)steps + 1 ? H : (long long)steps + 1) : steps + 1;
    int until = steps + 1;
    if (H > 0) until = phase0 == 0 ? 0 : (int)(H - phase0 < (long long)steps + 1 ? H - phase0 : (long long)steps + 1);
    int hop_log2 = hop0;        // k mod log2(n)
    float4* ycur = tile_smem;
    float4* ynext = tile_smem + cells;
    float4* gsum = tile_smem + 2 * cells;   // [n / 4 + 2][tile_groups]: the fp32 addends of the column mean
    float4* gmean = gsum + (n / 4 + 2) * tile_groups;   // [tile_groups]: the column means
    // ring: the cells above and below this one in the tile
    const int up_cell = (i == 0 ? n - 1 : i - 1) * tile_groups + g, dn_cell = (i == n - 1 ? 0 : i + 1) * tile_groups + g;
#pragma unroll 2
    for (int t = 0; t < steps; ++t) {
        const uint32_t k = p.k + (uint32_t)t;
        const bool global = until == 0;                     // Algorithm 1's test mod(k + 1, H) = 0
        const int mix = topology;
        float4 y = make_float4(0.f, 0.f, 0.f, 0.f);
        if (own) {
            y = tile_finish<MODE>(p, x, b, i, q, k);
            ycur[c] = y;
        }
        __syncthreads();
        if (global) {
            // The column mean, formed once per column group instead of once per cell: the first
            // row of every group of four adds its group in fp32, (y0 + y1) + (y2 + y3), as
            // tile_mix and the row-streaming kernel do; after a barrier one thread per column group
            // adds the group sums in fp64 in row order and hands the mean to the column's cells.
            // Same addends, same order, same result.
            const int full = n >> 2, rest = n & 3;
            if (own) {
                if ((i & 3) == 0 && i + 4 <= n) {
                    float4 a = ycur[c], b2 = ycur[(i + 2) * tile_groups + g];
                    acc4(a, ycur[(i + 1) * tile_groups + g]);
                    acc4(b2, ycur[(i + 3) * tile_groups + g]);
                    acc4(a, b2);
                    gsum[(i >> 2) * tile_groups + g] = a;
                } else if (i == 4 * full) {            // the unfinished last group: one or two addends
                    float4 a = ycur[c];
                    if (rest >= 2) acc4(a, ycur[(i + 1) * tile_groups + g]);
                    gsum[full * tile_groups + g] = a;
                    if (rest == 3) gsum[(full + 1) * tile_groups + g] = ycur[(i + 2) * tile_groups + g];
                }
            }
            __syncthreads();
            // thread c: component c & 3 of the mean of column group c >> 2 (four threads per group: the
            // fp64 chain of a component is what this step waits for, and the four are independent)
            for (int cc = c; cc < 4 * tile_groups; cc += blockDim.x) {   // (a block of n < 4 rows has fewer threads)
                const int gg = cc >> 2, comp = cc & 3;
                if (q_first + gg >= p.Q) continue;
                const int addends = full + (rest >= 1 ? 1 : 0) + (rest == 3 ? 1 : 0);
                const float* v = reinterpret_cast<const float*>(gsum + gg) + comp;
                double sum = 0.0;
                for (int j = 0; j < addends; ++j) sum += (double)v[(size_t)j * tile_groups * 4];
                float m;
                if ((n & (n - 1)) == 0)   // 1/n is exact: the product equals the quotient
                    m = (float)(sum * (1.0 / (double)n));
                else
                    m = (float)(sum / (double)n);
                reinterpret_cast<float*>(gmean + gg)[comp] = m;
            }
            __syncthreads();
            if (own) x = gmean[g];
        } else if (own) {
            if (TOPO == GPGA_TOPO_RING) {          // (up + self) + down, as tile_mix forms it
                x = scale4(add4(add4(ycur[up_cell], y), ycur[dn_cell]), 0.333333343f);
            } else if (TOPO == GPGA_TOPO_EXP) {
                x = scale4(add4(y, ycur[((i + (1 << hop_log2)) & (n - 1)) * tile_groups + g]), 0.5f);
            } else {
                x = tile_mix(ycur, i, g, n, tile_groups, mix, hop_log2, p.grid_cols, log2n, sw);
            }
        }
        float4* const swap = ycur;
        ycur = ynext;
        ynext = swap;
        until = global ? period - 1 : until - 1;
        if (++hop_log2 >= log2n) hop_log2 = 0;
    }
    if (own) store4<VEC>(p.out + (long long)i * p.ld, q * 4, p.d, x);
}

bool tile_supports(long long n) { return n * 16 <= kTileSmemBytes; }
bool run_tile_supports(long long n) { return n * 2 * 48 <= kTileSmemBytes; }   // X, b, Y strips of >= 2 groups

static int log2_floor(long long n)
{
    int t = 0;
    while ((1LL << (t + 1)) <= n) ++t;
    return t;
}

// Strip width: enough blocks to cover the SMs, at most 64 groups, within the shared-memory budget.
static int strip_groups(long long Q, long long n, int bytes_per_cell, int blocks_per_sm = 2)
{
    long long tg = (Q + blocks_per_sm * 148 - 1) / (blocks_per_sm * 148);
    if (tg < 2) tg = 2;
    if (tg > 64) tg = 64;
    if (tg > kTileSmemBytes / bytes_per_cell / n) tg = kTileSmemBytes / bytes_per_cell / n;
    if (tg > Q) tg = Q;
    // whole warps of cells where the strip can be narrowed to get them
    for (long long t = tg; t >= 2 && t * 2 > tg; --t)
        if ((n * t) % 32 == 0) { tg = t; break; }
    return (int)tg;
}

cudaError_t launch_step_tile(const StepParams& p, int mode, bool vec, int mix, cudaStream_t s)
{
    return launch_step_tile_w(p, mode, vec, mix, SparseW(), s);
}

cudaError_t launch_step_tile_w(const StepParams& p, int mode, bool vec, int mix, const SparseW& sw, cudaStream_t s)
{
    if (!tile_supports(p.n)) return cudaErrorInvalidConfiguration;   // callers bound n
    const int tile_groups = strip_groups(p.Q, p.n, 16);
    const int log2n = log2_floor(p.n);
    const unsigned grd = (unsigned)((p.Q + tile_groups - 1) / tile_groups);
    const size_t smem = (size_t)p.n * tile_groups * 16;
    const long long cells = p.n * tile_groups;
    const int blk = cells >= kTileBlock ? kTileBlock : (int)((cells + 31) / 32 * 32);
#define GPGA_TILE(M, V)                                                                          \
    do {                                                                                         \
        static unsigned long long limit_set = 0;                                                 \
        cudaError_t e = ensure_smem_limit(step_tile_kernel<M, V>, kTileSmemBytes, limit_set);    \
        if (e != cudaSuccess) return e;                                                          \
        step_tile_kernel<M, V><<<grd, blk, smem, s>>>(p, mix, tile_groups, log2n, sw);           \
    } while (0)
    if (mode == GRAD_PARTIALS) {   // logistic objective: d % 4 == 0 is required upstream
        // always follows the gradient kernel on the stream and waits for it first thing, so it may
        // be made resident while that kernel drains
        static unsigned long long limit_set = 0;
        cudaError_t e = ensure_smem_limit(step_tile_kernel<GRAD_PARTIALS, true>, kTileSmemBytes, limit_set);
        if (e != cudaSuccess) return e;
        return launch_after_trigger(step_tile_kernel<GRAD_PARTIALS, true>, dim3(grd), dim3(blk), smem, s, true, p,
                                    mix, tile_groups, log2n, sw);
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

cudaError_t launch_run_tile(const StepParams& p, int mode, bool vec, int topology, long long H, int steps,
                            const SparseW& sw, cudaStream_t s)
{
    if (!run_tile_supports(p.n) || (mode != GRAD_QUAD && mode != GRAD_QUAD_NOISE))
        return cudaErrorInvalidConfiguration;   // callers check
    const int log2n = log2_floor(p.n);
    const long long phase0 = H > 0 ? ((long long)p.k + 1) % H : 1;
    const int hop0 = log2n > 0 ? (int)(p.k % (uint32_t)log2n) : 0;
    if (p.n <= kTileBlock) {
        // one cell per thread: the narrowest strip that fills whole warps (small blocks balance
        // best over the SMs and wait least at their barrier); up to four warps' worth when there
        // are more blocks than fit on the GPU at once (the column means of a global-average
        // iteration are formed by one thread per column group: wider strips fill that warp)
        long long tg = kTileBlock / p.n;
        for (long long t = 1; t * p.n <= kTileBlock; ++t)
            if ((t * p.n) % 32 == 0) { tg = t; break; }
        while ((p.Q + tg - 1) / tg > 148 * 32 && 2 * tg * p.n <= kTileBlock / 2) tg *= 2;
        if (tg > p.Q) tg = p.Q;
        const int tile_groups = (int)tg;
        const unsigned grd = (unsigned)((p.Q + tile_groups - 1) / tile_groups);
        const long long cells = p.n * tile_groups;
        const int blk = (int)((cells + 31) / 32 * 32);
        const size_t smem = (size_t)cells * 32 + (size_t)(p.n / 4 + 3) * tile_groups * 16;
#define GPGA_RUN_CELL(M, V)                                                                                         \
    do {                                                                                                            \
        if (topology == GPGA_TOPO_RING)                                                                             \
            run_cell_kernel<M, V, GPGA_TOPO_RING><<<grd, blk, smem, s>>>(p, topology, H, phase0, hop0, steps, tile_groups, log2n, sw); \
        else if (topology == GPGA_TOPO_EXP)                                                                         \
            run_cell_kernel<M, V, GPGA_TOPO_EXP><<<grd, blk, smem, s>>>(p, topology, H, phase0, hop0, steps, tile_groups, log2n, sw);  \
        else                                                                                                        \
            run_cell_kernel<M, V, -1><<<grd, blk, smem, s>>>(p, topology, H, phase0, hop0, steps, tile_groups, log2n, sw);             \
    } while (0)
        if (vec) {
            if (mode == GRAD_QUAD) GPGA_RUN_CELL(GRAD_QUAD, true);
            else GPGA_RUN_CELL(GRAD_QUAD_NOISE, true);
        } else {
            if (mode == GRAD_QUAD) GPGA_RUN_CELL(GRAD_QUAD, false);
            else GPGA_RUN_CELL(GRAD_QUAD_NOISE, false);
        }
#undef GPGA_RUN_CELL
        return cudaGetLastError();
    }
    const int tile_groups = strip_groups(p.Q, p.n, 48, 8);   // compute-bound: fill every SM with warps
    const unsigned grd = (unsigned)((p.Q + tile_groups - 1) / tile_groups);
    const size_t smem = (size_t)p.n * tile_groups * 48;
    const long long cells = p.n * tile_groups;
    const int blk = cells >= kTileBlock ? kTileBlock : (int)((cells + 31) / 32 * 32);
#define GPGA_RUN_TILE(M, V)                                                                      \
    do {                                                                                         \
        static unsigned long long limit_set = 0;                                                 \
        cudaError_t e = ensure_smem_limit(run_tile_kernel<M, V>, kTileSmemBytes, limit_set);     \
        if (e != cudaSuccess) return e;                                                          \
        run_tile_kernel<M, V><<<grd, blk, smem, s>>>(p, topology, H, phase0, hop0, steps, tile_groups, log2n, sw); \
    } while (0)
    if (vec) {
        if (mode == GRAD_QUAD) GPGA_RUN_TILE(GRAD_QUAD, true);
        else GPGA_RUN_TILE(GRAD_QUAD_NOISE, true);
    } else {
        if (mode == GRAD_QUAD) GPGA_RUN_TILE(GRAD_QUAD, false);
        else GPGA_RUN_TILE(GRAD_QUAD_NOISE, false);
    }
#undef GPGA_RUN_TILE
    return cudaGetLastError();
}

}  // namespace gpga
