// Per-node mini-batch logistic-regression gradient (Section 5.1 loss with an l2 term):
//   f_i(x) = (1/m) sum_r ln(1 + exp(-y_r a_r^T x)) + (l2/2) ||x||^2
//   g_i    = -(1/B) sum_{r in batch} y_r a_r / (1 + exp(y_r a_r^T x_i)) + l2 x_i
// The B rows of node i at iteration k are drawn with replacement from the generator
// (stream BATCH).  The batch is cut into chunks of kChunkRows rows; block (i, c) forms
// the margins of its rows (one warp per row, shuffle reduction) and then its partial
// sum over those rows; a second kernel adds the chunks in a fixed order, so the result
// does not depend on scheduling.
#include "gpga_logreg.cuh"
#include "gpga_launch.cuh"
#include "gpga_tma.cuh"

namespace gpga {

constexpr int kLrBlock = 256;

// partial[c][i][:] = sum over the chunk's rows of s_r a_r,  s_r = -y_r / (1 + exp(y_r z_r)).
__global__ void __launch_bounds__(kLrBlock) logreg_partial_kernel(const LogregParams p)
{
    extern __shared__ float smem[];
    float* xs = smem;                          // d floats: x_i
    float* coef = smem + p.d;                  // kChunkRows floats: s_r
    __shared__ uint32_t rows[kChunkRows];
    __shared__ float ys[kChunkRows];
    const int i = blockIdx.x, c = blockIdx.y;
    const int t0 = c * kChunkRows;
    const int nrows = min(kChunkRows, (int)p.batch - t0);
    const float* A = p.A + (long long)i * p.m * p.d;
    const float* y = p.y + (long long)i * p.m;
    const float* x = p.x + (long long)i * p.ldx;
    for (int j = threadIdx.x; j < p.d; j += blockDim.x) xs[j] = x[j];
    if (threadIdx.x < nrows)
        rows[threadIdx.x] = batch_row((uint32_t)(t0 + threadIdx.x), (uint32_t)(i + p.node0), p.k, (uint32_t)p.m, p.keys);
    if (threadIdx.x < nrows) ys[threadIdx.x] = y[rows[threadIdx.x]];
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
            const float yr = ys[t];
            coef[t] = -yr / (1.0f + expf(yr * z));
            if (two) {
                const float yr2 = ys[t2];
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

// Polls of an mbarrier before a kernel gives up on a bulk copy.  A poll of a phase that is not
// complete blocks for about 4 microseconds (measured: 2000 polls of a barrier nobody completes take
// 8.2 ms), so this is about one second: far beyond any copy's latency, and finite.
constexpr uint32_t kTmaMaxTries = 1u << 18;

// A block whose bounded wait gave up and that was given no error word to raise writes NaN over its
// slice of the chunk partials (whole block calls): the sum over chunks, and so the gradient row of
// node i, is then NaN instead of whatever an earlier call left in that slice.
__device__ __forceinline__ void poison_partial(const LogregParams& p, int i, int c)
{
    float4* out4 = reinterpret_cast<float4*>(p.partial + ((long long)c * p.n + i) * p.d);
    const float q = __int_as_float(0x7FC00000);
    for (int g = threadIdx.x; g < (int)(p.d >> 2); g += blockDim.x) out4[g] = make_float4(q, q, q, q);
}

// Narrow rows (d <= kRegMaxD): the batch rows are staged in shared memory by bulk asynchronous
// copies (one 16-byte-aligned row of d floats per copy, completion counted on an mbarrier) and
// every warp runs its own pipeline -- it draws the indices of its rows (rows warp, warp + 8, ...
// of the chunk), copies each into one of its `slots` row buffers, and takes a staged row through
// registers once: the margin a^T x against x held in registers, then s * a added to per-lane
// accumulators.  A row is read from shared memory once, x not at all, and no block-wide
// barrier stands between rows; A is fetched from HBM exactly once.  The per-warp accumulators are added in warp
// order at the end (fixed order: the result does not depend on scheduling).
constexpr int kRegMaxD = 1024;
constexpr int kRegGroups = kRegMaxD / 4 / 32;   // float4 per lane
constexpr int kRegWarps = kLrBlock / 32;
constexpr int kRegMaxSlots = 4;                 // kChunkRows / kRegWarps rows per warp at most
constexpr int kRegSmemBytes = 96 * 1024;
static_assert(kRegWarps * kRegMaxSlots >= kChunkRows, "a warp must be able to hold all its rows");

__global__ void __launch_bounds__(kLrBlock, 2) logreg_partial_tma_reg_kernel(const LogregParams p, int slots)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t bars[kRegWarps * kRegMaxSlots];
    const int i = blockIdx.x, c = blockIdx.y;
    const int t0 = c * kChunkRows;
    const int nrows = min(kChunkRows, (int)p.batch - t0);
    const float* A = p.A + (long long)i * p.m * p.d;
    const float* y = p.y + (long long)i * p.m;
    const float4* x4 = reinterpret_cast<const float4*>(p.x + (long long)i * p.ldx);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int d4 = (int)(p.d >> 2);
    const uint32_t row_bytes = (uint32_t)p.d * 4u;
    float* mine = reinterpret_cast<float*>(smem_raw) + (size_t)warp * slots * p.d;   // this warp's row buffers
    uint64_t* bar = bars + warp * kRegMaxSlots;
    const int my_rows = warp < nrows ? (nrows - warp + kRegWarps - 1) / kRegWarps : 0;
    // lane r holds the index and the label of this warp's r-th row
    uint32_t my_idx = 0u;
    float my_y = 0.f;
    if (lane < my_rows) {
        my_idx = batch_row((uint32_t)(t0 + warp + lane * kRegWarps), (uint32_t)(i + p.node0), p.k, (uint32_t)p.m, p.keys);
        my_y = y[my_idx];
    }
    if (lane == 0) {
        for (int s = 0; s < slots; ++s) mbar_init(&bar[s], 1);
        mbar_init_fence();
    }
    __syncwarp();
    auto issue = [&](int r) {   // whole warp calls; lane 0 starts the copy of row r into slot r % slots
        const uint32_t idx = __shfl_sync(0xFFFFFFFFu, my_idx, r);
        if (lane == 0) {
            const int s = r % slots;
            mbar_arrive_expect_tx(&bar[s], row_bytes);
            bulk_copy_g2s(mine + (size_t)s * p.d, A + (long long)idx * p.d, row_bytes, &bar[s]);
        }
    };
    const int first = min(slots, my_rows);
    for (int r = 0; r < first; ++r) issue(r);
    // everything above reads only A, y and the iteration index; x is the previous step's output and
    // the partial sums may still be read by it
    grid_dependency_wait();
    // x_i and the running sums as packed pairs: one instruction does two fused multiply-adds, each
    // half rounded exactly as a scalar fmaf
    ulonglong2 xr[kRegGroups], acc[kRegGroups];
    const ulonglong2 zero2 = make_ulonglong2(0ull, 0ull);
#pragma unroll
    for (int j = 0; j < kRegGroups; ++j) {
        const int g = lane + 32 * j;
        xr[j] = g < d4 ? reinterpret_cast<const ulonglong2*>(x4)[g] : zero2;
        acc[j] = zero2;
    }
    bool failed = false;
    for (int r = 0; r < my_rows; ++r) {
        const int s = r % slots;
        const uint32_t parity = (uint32_t)(r / slots) & 1u;
        if (!__all_sync(0xFFFFFFFFu, mbar_wait_bounded(&bar[s], parity, kTmaMaxTries))) {   // warp-uniform
            // give the copies still in flight (this one and the later slots') one more bounded chance to land
            for (int q = r; q < min(my_rows, r + slots); ++q)
                mbar_wait_bounded(&bar[q % slots], (uint32_t)(q / slots) & 1u, kTmaMaxTries);
            failed = true;
            break;
        }
        const ulonglong2* a4 = reinterpret_cast<const ulonglong2*>(mine + (size_t)s * p.d);
        ulonglong2 a[kRegGroups];
        f32x2_t z01 = 0ull, z23 = 0ull;   // four running sums z0 .. z3
#pragma unroll
        for (int j = 0; j < kRegGroups; ++j) {
            const int g = lane + 32 * j;
            a[j] = g < d4 ? a4[g] : zero2;
            z01 = fma2(a[j].x, xr[j].x, z01);
            z23 = fma2(a[j].y, xr[j].y, z23);
        }
        const float2 za = unpack2(z01), zb = unpack2(z23);
        const float z = warp_sum_f((za.x + za.y) + (zb.x + zb.y));   // every lane holds the sum
        // the sum needed every lane's loads, so the slot is free: refill it before the arithmetic
        if (r + slots < my_rows) issue(r + slots);
        const float yr = __shfl_sync(0xFFFFFFFFu, my_y, r);
        const float sc = -yr / (1.0f + expf(yr * z));
        const f32x2_t sc2 = pack2(sc, sc);
#pragma unroll
        for (int j = 0; j < kRegGroups; ++j) {
            acc[j].x = fma2(sc2, a[j].x, acc[j].x);
            acc[j].y = fma2(sc2, a[j].y, acc[j].y);
        }
    }
    grid_launch_dependents();   // the step kernel may take its place; it waits for this grid before reading
    if (__syncthreads_or(failed)) {
        if (p.error_flag) {
            if (threadIdx.x == 0) atomicExch(p.error_flag, 1);
        } else {
            poison_partial(p, i, c);   // no error word to raise: make the result visibly invalid, never stale
        }
        return;
    }
    // every copy has landed and been read: park the per-warp sums in each warp's first slot
    float4* red = reinterpret_cast<float4*>(smem_raw);
    const int wstride = slots * d4;
#pragma unroll
    for (int j = 0; j < kRegGroups; ++j) {
        const int g = lane + 32 * j;
        if (g < d4) reinterpret_cast<ulonglong2*>(red)[warp * wstride + g] = acc[j];
    }
    __syncthreads();
    float4* out4 = reinterpret_cast<float4*>(p.partial + ((long long)c * p.n + i) * p.d);
    for (int g = threadIdx.x; g < d4; g += blockDim.x) {
        float4 sum = red[g];
        for (int w = 1; w < kRegWarps; ++w) {
            const float4 v = red[w * wstride + g];
            sum.x += v.x;
            sum.y += v.y;
            sum.z += v.z;
            sum.w += v.w;
        }
        out4[g] = sum;
    }
}

// Wider rows (kRegMaxD < d <= kTmaMaxD): the batch rows are staged in shared memory by bulk
// asynchronous copies (one 16-byte-aligned row of d floats per copy, completion counted on an
// mbarrier), two tiles of rows alternating: while one is consumed the next is in flight.  A
// thread owns J groups of four columns (group t + 256 u): x_i of those columns and its slice of
// the tile's rows sit in registers, so a staged row is read from shared memory once; the
// margins of the tile's rows are reduced over the block (lanes by shuffle, warps in index
// order through shared memory), and s * a is added to the thread's accumulators from the
// registers.  One block barrier per tile; A is fetched from HBM exactly once.
constexpr int kTmaMaxD = 8192;
constexpr int kColsCells = 8;            // (rows per tile) x (groups per thread), in registers

template <int J>
__global__ void __launch_bounds__(kLrBlock, 2) logreg_partial_tma_cols_kernel(const LogregParams p)
{
    constexpr int T = kColsCells / J;   // rows per tile
    constexpr int kWarps = kLrBlock / 32;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    float* tiles = reinterpret_cast<float*>(smem_raw);         // 2 x T x d
    __shared__ uint32_t rows[kChunkRows];
    __shared__ float ys[kChunkRows];
    __shared__ float wsum[2][T][kWarps];                       // per-warp margin sums, by tile parity
    __shared__ __align__(8) uint64_t bar[2];
    const int i = blockIdx.x, c = blockIdx.y;
    const int t0 = c * kChunkRows;
    const int nrows = min(kChunkRows, (int)p.batch - t0);
    const int ntiles = (nrows + T - 1) / T;
    const float* A = p.A + (long long)i * p.m * p.d;
    const float* y = p.y + (long long)i * p.m;
    const float4* x4 = reinterpret_cast<const float4*>(p.x + (long long)i * p.ldx);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int d4 = (int)(p.d >> 2);
    const uint32_t row_bytes = (uint32_t)p.d * 4u;
    if (threadIdx.x < nrows)
        rows[threadIdx.x] = batch_row((uint32_t)(t0 + threadIdx.x), (uint32_t)(i + p.node0), p.k, (uint32_t)p.m, p.keys);
    if (threadIdx.x == 0) {
        mbar_init(&bar[0], 1);
        mbar_init(&bar[1], 1);
        mbar_init_fence();
    }
    __syncthreads();
    // warp 0 starts the copies of tile s into buffer s & 1
    auto issue = [&](int s) {
        const int r0 = s * T;
        const int rr = min(T, nrows - r0);
        float* dst = tiles + (size_t)(s & 1) * T * p.d;
        if (lane == 0) mbar_arrive_expect_tx(&bar[s & 1], (uint32_t)rr * row_bytes);
        __syncwarp();
        if (lane < rr) bulk_copy_g2s(dst + (size_t)lane * p.d, A + (long long)rows[r0 + lane] * p.d, row_bytes, &bar[s & 1]);
    };
    if (warp == 0) {
        issue(0);
        if (ntiles > 1) issue(1);
    }
    if (threadIdx.x < nrows) ys[threadIdx.x] = y[rows[threadIdx.x]];
    // everything above reads only A, y and the iteration index; x is the previous step's output and
    // the partial sums may still be read by it
    grid_dependency_wait();
    float4 xr[J], acc[J];
#pragma unroll
    for (int u = 0; u < J; ++u) {
        const int g = threadIdx.x + u * kLrBlock;
        xr[u] = g < d4 ? x4[g] : make_float4(0.f, 0.f, 0.f, 0.f);
        acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    __syncthreads();   // ys
    uint32_t parity0 = 0u, parity1 = 0u;
    bool failed = false;
    for (int s = 0; s < ntiles; ++s) {
        const int buf = s & 1;
        const int r0 = s * T;
        const int rr = min(T, nrows - r0);
        const float* tile = tiles + (size_t)buf * T * p.d;
        const uint32_t par = buf ? parity1 : parity0;
        const bool ok = mbar_wait_bounded(&bar[buf], par, kTmaMaxTries);
        if (__syncthreads_or(!ok)) {
            // a copy did not report in time: flag it, give the copies in flight (they target
            // this block's shared memory) one more bounded chance to land, and leave
            if (!ok) mbar_wait_bounded(&bar[buf], par, kTmaMaxTries);
            if (s + 1 < ntiles) mbar_wait_bounded(&bar[buf ^ 1], buf ? parity0 : parity1, kTmaMaxTries);
            if (threadIdx.x == 0 && p.error_flag) atomicExch(p.error_flag, 1);
            failed = true;
            break;
        }
        if (buf) parity1 ^= 1u; else parity0 ^= 1u;
        // this thread's slice of the tile, and its part of every row's margin
        float4 a[T][J];
#pragma unroll
        for (int t = 0; t < T; ++t) {
            float z = 0.f;
#pragma unroll
            for (int u = 0; u < J; ++u) {
                const int g = threadIdx.x + u * kLrBlock;
                a[t][u] = (t < rr && g < d4) ? reinterpret_cast<const float4*>(tile + (size_t)t * p.d)[g]
                                             : make_float4(0.f, 0.f, 0.f, 0.f);
                z = fmaf(a[t][u].x, xr[u].x, z);
                z = fmaf(a[t][u].y, xr[u].y, z);
                z = fmaf(a[t][u].z, xr[u].z, z);
                z = fmaf(a[t][u].w, xr[u].w, z);
            }
            z = warp_sum_f(z);
            if (lane == 0) wsum[buf][t][warp] = z;
        }
        __syncthreads();   // margins complete; every thread holds its slice, so the buffer is free
        if (warp == 0 && s + 2 < ntiles) issue(s + 2);
#pragma unroll
        for (int t = 0; t < T; ++t) {
            if (t < rr) {
                float z = wsum[buf][t][0];
#pragma unroll
                for (int w = 1; w < kWarps; ++w) z += wsum[buf][t][w];
                const float yr = ys[r0 + t];
                const float sc = -yr / (1.0f + expf(yr * z));
#pragma unroll
                for (int u = 0; u < J; ++u) {
                    acc[u].x = fmaf(sc, a[t][u].x, acc[u].x);
                    acc[u].y = fmaf(sc, a[t][u].y, acc[u].y);
                    acc[u].z = fmaf(sc, a[t][u].z, acc[u].z);
                    acc[u].w = fmaf(sc, a[t][u].w, acc[u].w);
                }
            }
        }
    }
    grid_launch_dependents();   // the step kernel may take its place; it waits for this grid before reading
    if (failed) {   // block-uniform
        if (!p.error_flag) poison_partial(p, i, c);
        return;
    }
    float4* out4 = reinterpret_cast<float4*>(p.partial + ((long long)c * p.n + i) * p.d);
#pragma unroll
    for (int u = 0; u < J; ++u) {
        const int g = threadIdx.x + u * kLrBlock;
        if (g < d4) out4[g] = acc[u];
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
        const uint32_t r = batch_row((uint32_t)t, (uint32_t)(i + p.node0), p.k, (uint32_t)p.m, p.keys);
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

// A wait that cannot succeed: the barrier expects one arrival that never comes.  Exercises the
// give-up path of mbar_wait_bounded and the error word without any copy in flight.
__global__ void bounded_wait_selftest_kernel(int* error_flag, uint32_t tries)
{
    __shared__ __align__(8) uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        mbar_init_fence();
    }
    __syncthreads();
    const bool ok = mbar_wait_bounded(&bar, 0u, tries);
    if (!ok && threadIdx.x == 0) atomicExch(error_flag, 1);
}

cudaError_t launch_bounded_wait_selftest(int* error_flag, cudaStream_t s)
{
    bounded_wait_selftest_kernel<<<1, 32, 0, s>>>(error_flag, 2000u);
    return cudaGetLastError();
}

int logreg_chunks(long long batch) { return (int)((batch + kChunkRows - 1) / kChunkRows); }

cudaError_t launch_logreg_partial(const LogregParams& p, cudaStream_t s)
{
    const int chunks = logreg_chunks(p.batch);
    if (p.d <= kRegMaxD) {
        int slots = kRegSmemBytes / (kRegWarps * (int)p.d * 4);   // row buffers per warp
        if (slots > kRegMaxSlots) slots = kRegMaxSlots;
        const size_t smem_reg = (size_t)kRegWarps * slots * p.d * sizeof(float);
        static unsigned long long reg_limit_set = 0;
        cudaError_t e = ensure_smem_limit(logreg_partial_tma_reg_kernel, kRegSmemBytes, reg_limit_set);
        if (e != cudaSuccess) return e;
        return launch_after_trigger(logreg_partial_tma_reg_kernel, dim3((unsigned)p.n, (unsigned)chunks),
                                    dim3(kLrBlock), smem_reg, s, p.after_own_step, p, slots);
    }
    if (p.d <= kTmaMaxD) {
        const int groups = (int)((p.d / 4 + kLrBlock - 1) / kLrBlock);   // groups of four columns per thread
        const dim3 grid((unsigned)p.n, (unsigned)chunks);
        const size_t smem_cols = 2 * (size_t)kColsCells * p.d * sizeof(float);   // before / J below
#define GPGA_COLS(J)                                                                                   \
    do {                                                                                               \
        static unsigned long long limit_set = 0;                                                       \
        cudaError_t e = ensure_smem_limit(logreg_partial_tma_cols_kernel<J>, 64 * 1024, limit_set);    \
        if (e != cudaSuccess) return e;                                                                \
        return launch_after_trigger(logreg_partial_tma_cols_kernel<J>, grid, dim3(kLrBlock), smem_cols / J, s, \
                                    p.after_own_step, p);                                              \
    } while (0)
        if (groups <= 2) GPGA_COLS(2);
        else if (groups <= 4) GPGA_COLS(4);
        else GPGA_COLS(8);
#undef GPGA_COLS
    }
    const size_t smem = (size_t)(p.d + kChunkRows) * sizeof(float);
    static unsigned long long plain_limit_set = 0;
    cudaError_t e = ensure_smem_limit(logreg_partial_kernel, 200 * 1024, plain_limit_set);
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
