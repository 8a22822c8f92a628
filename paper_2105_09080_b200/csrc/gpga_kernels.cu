// Fused Gossip-PGA kernels for sm_100a.
//
// Every step kernel gives one thread a group of four adjacent columns and streams
// it down the n rows (nodes): each element of X and of b is read once, the
// half-step Y = X - gamma G (Algorithm 1's local update) lives only in registers,
// the noise is generated in registers, and each element of X^(k+1) is written once:
// 12 bytes of HBM traffic per node-parameter update.  The mixing of Algorithm 1
// (gossip step or global average) acts along the rows of one column group, so no
// thread ever needs another thread's data.
#include "gpga_kernels.cuh"

namespace gpga {

constexpr int kBlock = 256;

// One row's inputs for one column group, and x^(k+1/2) formed from them
// (Algorithm 1: gradient, then the local update).  Loading and finishing are split
// so that a thread can have the loads of several rows in flight before it needs any.
struct RowIn {
    float4 x, b;
};

// What one thread needs to address its group of four columns in any row.  Row indices
// are 32-bit (n < 2^31); the element offset row * ld is formed in 64 bits.
struct ColGroup {
    const float* x;    // p.x + j0 (128-bit path) or p.x
    const float* b;
    float* out;
    long long j0;      // first local column of the group
    uint32_t qg;       // global group index = first counter word of the generator
};

template <bool VEC>
__device__ __forceinline__ ColGroup col_group(const StepParams& p, long long q)
{
    ColGroup c;
    c.j0 = q * 4;
    c.x = VEC ? p.x + c.j0 : p.x;
    c.b = VEC ? p.b + c.j0 : p.b;
    c.out = VEC ? p.out + c.j0 : p.out;
    c.qg = p.q_base + (uint32_t)q;
    return c;
}

template <bool VEC>
__device__ __forceinline__ RowIn load_row(const StepParams& p, const ColGroup& c, int i)
{
    RowIn r;
    if (VEC) {
        r.x = ld_stream4(c.x + (long long)i * p.ld);
        r.b = ld_stream4(c.b + (long long)i * p.ldb);
    } else {
        r.x = load4<false>(c.x + (long long)i * p.ld, c.j0, p.d);
        r.b = load4<false>(c.b + (long long)i * p.ldb, c.j0, p.d);
    }
    return r;
}

template <bool VEC>
__device__ __forceinline__ void store_row(const StepParams& p, const ColGroup& c, int i, float4 v)
{
    if (VEC)
        st_stream4(c.out + (long long)i * p.ld, v);
    else
        store4<false>(c.out + (long long)i * p.ld, c.j0, p.d, v);
}

template <int MODE>
__device__ __forceinline__ float4 finish_row(const StepParams& p, const ColGroup& c, const RowIn& r, int i)
{
    float4 g;
    if (MODE == GRAD_BUFFER) {
        g = r.b;
    } else {
        g = sub4(r.x, r.b);
        if (MODE == GRAD_QUAD_NOISE) g = fma4(p.sigma, normal4(c.qg, (uint32_t)i, p.k, 0u, p.keys), g);
    }
    return fma4(-p.gamma, g, r.x);
}

template <int MODE, bool VEC>
__device__ __forceinline__ float4 half_step(const StepParams& p, const ColGroup& c, int i)
{
    return finish_row<MODE>(p, c, load_row<VEC>(p, c, i), i);
}

// Visit steps t = t0 .. n-1 of a walk over the rows: row_of(t) is the row read at step
// t, visit(t, row, y) consumes its half-step value.  Steps are visited in order.
// A thread issues the loads of U rows before it needs any of them; with PIPE the
// loads of the next batch are issued before the arithmetic of the current one
// (software pipeline in registers), so the memory system never waits for the noise
// arithmetic.  U and PIPE are tuned per kernel.
template <int MODE, bool VEC, int U, bool PIPE, class RowOf, class Visit>
__device__ __forceinline__ void stream_rows(const StepParams& p, const ColGroup& c, int t0, RowOf row_of,
                                            Visit visit)
{
    const int n = (int)p.n;
    int t = t0;
    RowIn cur[U], nxt[U];
    if (t + U <= n) {
#pragma unroll
        for (int u = 0; u < U; ++u) cur[u] = load_row<VEC>(p, c, row_of(t + u));
    }
    while (t + U <= n) {
        const bool more = (t + 2 * U <= n);
        if (PIPE && more) {
#pragma unroll
            for (int u = 0; u < U; ++u) nxt[u] = load_row<VEC>(p, c, row_of(t + U + u));
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int row = row_of(t + u);
            visit(t + u, row, finish_row<MODE>(p, c, cur[u], row));
        }
        t += U;
        if (PIPE) {
#pragma unroll
            for (int u = 0; u < U; ++u) cur[u] = nxt[u];
        } else if (more) {
#pragma unroll
            for (int u = 0; u < U; ++u) cur[u] = load_row<VEC>(p, c, row_of(t + u));
        }
    }
    for (; t < n; ++t) {
        const int row = row_of(t);
        visit(t, row, half_step<MODE, VEC>(p, c, row));
    }
}

// ---------------------------------------------------------------------------
// Ring: x_i^(k+1) = (y_{i-1} + y_i + y_{i+1}) / 3, indices mod n.  A three-row
// window slides down the rows; rows 0 and 1 are kept for the wrap-around.
// ---------------------------------------------------------------------------
__device__ __forceinline__ float4 mix3(float4 a, float4 b, float4 c)
{
    return scale4(add4(add4(a, b), c), 0.333333343f);
}

template <int MODE, bool VEC, int U, bool PIPE>
__device__ __forceinline__ void ring_columns(const StepParams& p, long long q)
{
    const ColGroup c = col_group<VEC>(p, q);
    const int n = (int)p.n;
    if (n <= 2) {
        const float4 y0 = half_step<MODE, VEC>(p, c, 0);
        if (n == 1) {
            store_row<VEC>(p, c, 0, mix3(y0, y0, y0));
            return;
        }
        const float4 y1 = half_step<MODE, VEC>(p, c, 1);
        store_row<VEC>(p, c, 0, mix3(y1, y0, y1));
        store_row<VEC>(p, c, 1, mix3(y0, y1, y0));
        return;
    }
    const RowIn r0 = load_row<VEC>(p, c, 0), r1 = load_row<VEC>(p, c, 1);
    const float4 y0 = finish_row<MODE>(p, c, r0, 0);
    const float4 y1 = finish_row<MODE>(p, c, r1, 1);
    float4 a = y0, b = y1;
    stream_rows<MODE, VEC, U, PIPE>(
        p, c, 2, [](int t) { return t; },
        [&](int, int i, float4 v) {
            store_row<VEC>(p, c, i - 1, mix3(a, b, v));
            a = b;
            b = v;
        });
    store_row<VEC>(p, c, n - 1, mix3(a, b, y0));
    store_row<VEC>(p, c, 0, mix3(b, y0, y1));
}

// The grid holds one thread per column group.  (Cutting the grid of a state of a few waves to one
// resident wave, every thread taking several groups a grid apart, measured slower: n = 32,
// d = 2^20: 75.8 against 70.7 us per launch; n = 32, d = 2^21: 150 against 132 us.)
template <int MODE, bool VEC, int U, bool PIPE, int BLOCK, int MINB>
__global__ void __launch_bounds__(BLOCK, MINB) step_ring_kernel(const StepParams p)
{
    const long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (q < p.Q) ring_columns<MODE, VEC, U, PIPE>(p, q);
}

// ---------------------------------------------------------------------------
// One-peer exponential graph: x_i^(k+1) = (y_i + y_{(i+h) mod n}) / 2, h = 2^t.
// i -> i + h splits the nodes into h cycles of length n/h; walking a cycle needs
// only the previous row and the cycle's first row, so each row is read (and its
// noise generated) once.  Step t of the flattened walk visits row
// (t / L) + (t mod L) * h with L = n / h.
// ---------------------------------------------------------------------------
template <int MODE, bool VEC, int U, bool PIPE>
__device__ __forceinline__ void exp_columns(const StepParams& p, long long q)
{
    const ColGroup c = col_group<VEC>(p, q);
    const int len_log2 = p.len_log2, hop_log2 = p.hop_log2;
    const int hop = 1 << hop_log2;
    const int lmask = (1 << len_log2) - 1;
    float4 first = make_float4(0.f, 0.f, 0.f, 0.f), prev = first;
    const int n = (int)p.n;
    if (U == 4 && n >= 4) {
        // Batches of four consecutive steps of the walk (n and the cycle length L are powers of two).
        // With L >= 4 a batch lies inside one cycle: rows row0 + u h, addressed from one base by
        // multiples of h rows; with L = 2 it is two whole cycles: rows c, c + h, c + 1, c + 1 + h.
        // Only the batch start is tracked (position in the cycle, first row), not every row.
        const int L = 1 << len_log2;
        const long long hop_ld = (long long)p.ld << hop_log2, hop_ldb = (long long)p.ldb << hop_log2;
        const long long j0 = VEC ? 0 : c.j0;
        auto load_at = [&](long long ox, long long ob) {
            RowIn r;
            r.x = load4<VEC>(c.x + ox, j0, p.d);
            r.b = load4<VEC>(c.b + ob, j0, p.d);
            return r;
        };
        auto store_at = [&](long long o, float4 v) { store4<VEC>(c.out + o, j0, p.d, v); };
        auto half = [](float4 a, float4 b) { return scale4(add4(a, b), 0.5f); };
        if (L >= 4) {
            int s0 = 0, row0 = 0;
            for (int t = 0; t < n; t += 4) {
                const long long ox = (long long)row0 * p.ld, ob = (long long)row0 * p.ldb;
                RowIn r[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) r[u] = load_at(ox + u * hop_ld, ob + u * hop_ldb);
                float4 y = finish_row<MODE>(p, c, r[0], row0);
                if (s0 == 0)
                    first = y;
                else
                    store_at(ox - hop_ld, half(prev, y));
                prev = y;
#pragma unroll
                for (int u = 1; u < 4; ++u) {
                    y = finish_row<MODE>(p, c, r[u], row0 + (u << hop_log2));
                    store_at(ox + (u - 1) * hop_ld, half(prev, y));
                    prev = y;
                }
                s0 += 4;
                if (s0 == L) {   // the cycle closes: its last row mixes with its first
                    store_at(ox + 3 * hop_ld, half(prev, first));
                    s0 = 0;
                    row0 = (t + 4) >> len_log2;
                } else {
                    row0 += 4 << hop_log2;
                }
            }
        } else {   // L == 2
            for (int cyc = 0; cyc < hop; cyc += 2) {
                const long long ox = (long long)cyc * p.ld, ob = (long long)cyc * p.ldb;
                RowIn r[4];
                r[0] = load_at(ox, ob);
                r[1] = load_at(ox + hop_ld, ob + hop_ldb);
                r[2] = load_at(ox + p.ld, ob + p.ldb);
                r[3] = load_at(ox + p.ld + hop_ld, ob + p.ldb + hop_ldb);
                const float4 y0 = finish_row<MODE>(p, c, r[0], cyc);
                const float4 y1 = finish_row<MODE>(p, c, r[1], cyc + hop);
                store_at(ox, half(y0, y1));
                store_at(ox + hop_ld, half(y1, y0));
                const float4 y2 = finish_row<MODE>(p, c, r[2], cyc + 1);
                const float4 y3 = finish_row<MODE>(p, c, r[3], cyc + 1 + hop);
                store_at(ox + p.ld, half(y2, y3));
                store_at(ox + p.ld + hop_ld, half(y3, y2));
            }
        }
        return;
    }
    stream_rows<MODE, VEC, U, PIPE>(
        p, c, 0, [=](int t) { return (t >> len_log2) + ((t & lmask) << hop_log2); },
        [&](int t, int row, float4 cur) {
            const int s = t & lmask;
            if (s == 0)
                first = cur;
            else
                store_row<VEC>(p, c, row - hop, scale4(add4(prev, cur), 0.5f));
            if (s == lmask) store_row<VEC>(p, c, row, scale4(add4(cur, first), 0.5f));
            prev = cur;
        });
}

template <int MODE, bool VEC, int U, bool PIPE, int BLOCK, int MINB>
__global__ void __launch_bounds__(BLOCK, MINB) step_exp_kernel(const StepParams p)
{
    const long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (q < p.Q) exp_columns<MODE, VEC, U, PIPE>(p, q);
}

// ---------------------------------------------------------------------------
// Global average: m_j = (1/n) sum_i y_ij, written to every row.  Rows are added
// pairwise in fp32 in groups of four, (y0 + y1) + (y2 + y3), and the group sums are
// accumulated in fp64 and rounded once.  A group sum carries at most three fp32
// roundings, so the mean is within a few 1e-8 (1 + |y|) of the exact one; and when all
// rows are equal every group sum (v, 2v or 4v) is exact, so the mean is exactly v.
// ---------------------------------------------------------------------------
template <int MODE, bool VEC, int U, bool PIPE>
__device__ __forceinline__ void global_columns(const StepParams& p, long long q)
{
    const ColGroup c = col_group<VEC>(p, q);
    double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
    stream_rows<MODE, VEC, U, PIPE>(
        p, c, 0, [](int t) { return t; },
        [&](int t, int, float4 y) {
            const int phase = t & 3;
            if (phase == 0) {
                a = y;
            } else if (phase == 1) {
                a = add4(a, y);
            } else if (phase == 2) {
                b = y;
            } else {
                b = add4(b, y);
                const float4 g = add4(a, b);
                s0 += (double)g.x;
                s1 += (double)g.y;
                s2 += (double)g.z;
                s3 += (double)g.w;
            }
        });
    const int n = (int)p.n, rest = n & 3;   // rows of an unfinished last group
    if (rest >= 1) {
        s0 += (double)a.x;
        s1 += (double)a.y;
        s2 += (double)a.z;
        s3 += (double)a.w;
    }
    if (rest == 3) {
        s0 += (double)b.x;
        s1 += (double)b.y;
        s2 += (double)b.z;
        s3 += (double)b.w;
    }
    const double inv = (double)p.n;
    const float4 m = make_float4((float)(s0 / inv), (float)(s1 / inv), (float)(s2 / inv),
                                 (float)(s3 / inv));
#pragma unroll 4
    for (int i = 0; i < n; ++i) store_row<VEC>(p, c, i, m);
}

template <int MODE, bool VEC, int U, bool PIPE, int BLOCK, int MINB>
__global__ void __launch_bounds__(BLOCK, MINB) step_global_kernel(const StepParams p)
{
    const long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (q < p.Q) global_columns<MODE, VEC, U, PIPE>(p, q);
}

static inline unsigned grid_for(long long Q, int block) { return (unsigned)((Q + block - 1) / block); }

// Launch shape per kernel: rows in flight per thread (U), register pipeline (PIPE),
// threads per block and minimum resident blocks (the register cap), chosen by timing
// on B200 at the ResNet-50- and BERT-Large-sized states.
// (ring: four rows in flight need ~85 registers; 768 threads per SM with four rows each keep more
// bytes in flight than 1024 threads with two, worth 2.5 % in the seconds-long loop under the power
// cap: 2.96 against 3.03 ms per launch at n = 64, d = 25,557,032.  The exponential and the
// global-average kernel already have four rows in flight at 64 registers; 128-thread blocks, six or
// eight rows in flight or a looser register cap measured equal or slower for them.)
struct RingTune { static constexpr int U = 4; static constexpr bool PIPE = false; static constexpr int BLOCK = 128; static constexpr int MINB = 6; };
struct ExpTune { static constexpr int U = 4; static constexpr bool PIPE = false; static constexpr int BLOCK = 256; static constexpr int MINB = 4; };
struct GlobalTune { static constexpr int U = 4; static constexpr bool PIPE = false; static constexpr int BLOCK = 256; static constexpr int MINB = 4; };
constexpr int kSmallBlock = 64;   // small problems: narrow blocks spread the column groups over more SMs

#define GPGA_DISPATCH(kernel, T, p, mode, vec, s)                                                      \
    do {                                                                                               \
        const bool small = (p).Q < 148LL * 4 * T::BLOCK;                                               \
        const int blk = small ? kSmallBlock : T::BLOCK;                                                \
        const unsigned grd = grid_for((p).Q, blk);                                                     \
        if (vec) {                                                                                     \
            if (mode == GRAD_QUAD) kernel<GRAD_QUAD, true, T::U, T::PIPE, T::BLOCK, T::MINB><<<grd, blk, 0, s>>>(p);             \
            else if (mode == GRAD_QUAD_NOISE) kernel<GRAD_QUAD_NOISE, true, T::U, T::PIPE, T::BLOCK, T::MINB><<<grd, blk, 0, s>>>(p); \
            else kernel<GRAD_BUFFER, true, T::U, T::PIPE, T::BLOCK, T::MINB><<<grd, blk, 0, s>>>(p);                             \
        } else {                                                                                       \
            if (mode == GRAD_QUAD) kernel<GRAD_QUAD, false, 2, false, T::BLOCK, 1><<<grd, blk, 0, s>>>(p);                       \
            else if (mode == GRAD_QUAD_NOISE) kernel<GRAD_QUAD_NOISE, false, 2, false, T::BLOCK, 1><<<grd, blk, 0, s>>>(p);      \
            else kernel<GRAD_BUFFER, false, 2, false, T::BLOCK, 1><<<grd, blk, 0, s>>>(p);                                       \
        }                                                                                              \
        return cudaGetLastError();                                                                     \
    } while (0)

cudaError_t launch_step_ring(const StepParams& p, int mode, bool vec, cudaStream_t s)
{
    GPGA_DISPATCH(step_ring_kernel, RingTune, p, mode, vec, s);
}
cudaError_t launch_step_exp(const StepParams& p, int mode, bool vec, cudaStream_t s)
{
    GPGA_DISPATCH(step_exp_kernel, ExpTune, p, mode, vec, s);
}
cudaError_t launch_step_global(const StepParams& p, int mode, bool vec, cudaStream_t s)
{
    GPGA_DISPATCH(step_global_kernel, GlobalTune, p, mode, vec, s);
}

// ---------------------------------------------------------------------------
// Consensus distance sum_j sum_i (x_ij - xbar_j)^2.  One pass over X: with
// e_i = x_i - x_0, sum_i (x_i - xbar)^2 = sum e_i^2 - (sum e_i)^2 / n; shifting by row 0 keeps
// the subtraction benign when the rows are nearly equal.  e_i is formed in fp32: exact when x_i
// and x_0 are within a factor of two of each other (the nearly-consensual case, where it matters),
// one rounding of 2^-24 relative otherwise.  Rows are taken in groups of four: e and e^2 are added
// pairwise in fp32 inside a group, (e0 + e1) + (e2 + e3), and the group sums are accumulated in
// fp64 -- a quarter of the conversions and fp64 additions of an all-fp64 pass, at a relative error of
// a few 1e-7.  Like the step kernels, one thread owns a group of four columns and keeps the loads
// of four rows in flight; one block covers 256 adjacent column groups (a contiguous window in
// every row), writes one partial, and a second kernel adds the partials in a fixed order.
// ---------------------------------------------------------------------------
constexpr int kReduceBlock = 256;

long long consensus_blocks(long long Q)
{
    const long long b = (Q + kReduceBlock - 1) / kReduceBlock;
    return b < 1 ? 1 : b;
}

int reduce_blocks(long long Q)
{
    long long b = (Q + kReduceBlock - 1) / kReduceBlock;
    if (b > kMaxReduceBlocks) b = kMaxReduceBlocks;
    if (b < 1) b = 1;
    return (int)b;
}

__device__ __forceinline__ float4 mul4(float4 a, float4 b)
{
    return join4(mul2(pack2(a.x, a.y), pack2(b.x, b.y)), mul2(pack2(a.z, a.w), pack2(b.z, b.w)));
}
// a * a + c, component-wise
__device__ __forceinline__ float4 sqadd4(float4 a, float4 c)
{
    return join4(fma2(pack2(a.x, a.y), pack2(a.x, a.y), pack2(c.x, c.y)),
                 fma2(pack2(a.z, a.w), pack2(a.z, a.w), pack2(c.z, c.w)));
}

template <bool VEC>
__global__ void __launch_bounds__(kReduceBlock, 4) consensus_kernel(const float* __restrict__ x,
                                                                 long long n, long long d,
                                                                 long long ld, long long Q, int slabs,
                                                                 double* __restrict__ partials)
{
    double acc = 0.0;
    // a block covers `slabs` adjacent slabs of 256 column groups (more than one when n is small, so
    // that a block lives long enough to amortise its start and its reduction)
    for (int sl = 0; sl < slabs; ++sl) {
        const long long q = ((long long)blockIdx.x * slabs + sl) * blockDim.x + threadIdx.x;
        if (q >= Q) break;
        const long long j0 = q * 4;
        const float* col = VEC ? x + j0 : x;       // load4<true> ignores j0 and d
        const long long jv = VEC ? 0 : j0;
        const float4 r0 = load4<VEC>(col, jv, d);
        double s1[4] = {0, 0, 0, 0}, s2[4] = {0, 0, 0, 0};
        long long i = 1;
        for (; i + 4 <= n; i += 4) {
            float4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) v[u] = load4<VEC>(col + (i + u) * ld, jv, d);
            const float4 e0 = sub4(v[0], r0), e1 = sub4(v[1], r0), e2 = sub4(v[2], r0), e3 = sub4(v[3], r0);
            const float4 sum = add4(add4(e0, e1), add4(e2, e3));
            const float4 sq = add4(sqadd4(e1, mul4(e0, e0)), sqadd4(e3, mul4(e2, e2)));
            s1[0] += (double)sum.x; s1[1] += (double)sum.y; s1[2] += (double)sum.z; s1[3] += (double)sum.w;
            s2[0] += (double)sq.x; s2[1] += (double)sq.y; s2[2] += (double)sq.z; s2[3] += (double)sq.w;
        }
        for (; i < n; ++i) {   // at most three rows left
            const float4 e = sub4(load4<VEC>(col + i * ld, jv, d), r0);
            const double e0 = (double)e.x, e1 = (double)e.y, e2 = (double)e.z, e3 = (double)e.w;
            s1[0] += e0; s2[0] = fma(e0, e0, s2[0]);
            s1[1] += e1; s2[1] = fma(e1, e1, s2[1]);
            s1[2] += e2; s2[2] = fma(e2, e2, s2[2]);
            s1[3] += e3; s2[3] = fma(e3, e3, s2[3]);
        }
        const double inv_n = 1.0 / (double)n;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            // columns past d loaded as zeros in every row: they contribute exactly 0
            const double v = s2[e] - s1[e] * s1[e] * inv_n;
            acc += v > 0.0 ? v : 0.0;
        }
    }
    acc = block_sum(acc);
    if (threadIdx.x == 0) partials[blockIdx.x] = acc;
}

__global__ void final_sum_kernel(const double* __restrict__ partials, int count, double scale,
                                 double* __restrict__ result)
{
    // one warp, fixed order: lane l adds partials l, l+32, ...; then a shuffle tree
    double v = 0.0;
    for (int t = threadIdx.x; t < count; t += 32) v += partials[t];
    v = warp_sum(v);
    if (threadIdx.x == 0) *result = v * scale;
}

// The same for many partials: thread t of one 1024-thread block adds partials t, t + 1024, ... in
// that order, then the block's fixed shuffle / shared-memory tree.  Independent of scheduling.
__global__ void __launch_bounds__(1024) final_sum_wide_kernel(const double* __restrict__ partials, long long count,
                                                              double* __restrict__ result)
{
    double v = 0.0;
    for (long long t = threadIdx.x; t < count; t += 1024) v += partials[t];
    v = block_sum(v);
    if (threadIdx.x == 0) *result = v;
}

cudaError_t launch_consensus(const float* x, long long n, long long d, long long ld, bool vec, double* partials,
                             double* result, cudaStream_t s)
{
    const long long Q = (d + 3) / 4;
    // about 64 rows' worth of loads per thread: n >= 64 one slab, n = 16 four, at most 8
    int slabs = (int)(64 / (n < 1 ? 1 : n));
    slabs = slabs < 1 ? 1 : (slabs > 8 ? 8 : slabs);
    if (consensus_blocks(Q) < 148 * 16) slabs = 1;   // small states: keep every SM busy
    const long long blocks = (consensus_blocks(Q) + slabs - 1) / slabs;
    if (vec)
        consensus_kernel<true><<<(unsigned)blocks, kReduceBlock, 0, s>>>(x, n, d, ld, Q, slabs, partials);
    else
        consensus_kernel<false><<<(unsigned)blocks, kReduceBlock, 0, s>>>(x, n, d, ld, Q, slabs, partials);
    if (blocks <= 4096)
        final_sum_kernel<<<1, 32, 0, s>>>(partials, (int)blocks, 1.0, result);
    else
        final_sum_wide_kernel<<<1, 1024, 0, s>>>(partials, blocks, result);
    return cudaGetLastError();
}

// (1/n) sum_i 1/2 ||x_i - b_i||^2 over all elements.
template <bool VEC>
__global__ void __launch_bounds__(kReduceBlock, 3) quadratic_loss_kernel(const float* __restrict__ x,
                                                                      const float* __restrict__ b,
                                                                      long long n, long long d,
                                                                      long long ld, long long Q,
                                                                      double* __restrict__ partials)
{
    double acc = 0.0;
    for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < Q;
         q += (long long)gridDim.x * blockDim.x) {
        const long long j0 = q * 4;
#pragma unroll 4
        for (long long i = 0; i < n; ++i) {
            const float4 xv = load4<VEC>(x + i * ld, j0, d);   // columns past d load as zeros
            const float4 bv = load4<VEC>(b + i * ld, j0, d);
            const double r0 = (double)xv.x - (double)bv.x, r1 = (double)xv.y - (double)bv.y;
            const double r2 = (double)xv.z - (double)bv.z, r3 = (double)xv.w - (double)bv.w;
            acc = fma(r0, r0, acc);
            acc = fma(r1, r1, acc);
            acc = fma(r2, r2, acc);
            acc = fma(r3, r3, acc);
        }
    }
    acc = block_sum(acc);
    if (threadIdx.x == 0) partials[blockIdx.x] = acc;
}

cudaError_t launch_quadratic_loss(const float* x, const float* b, long long n, long long d, long long ld,
                                  bool vec, double* partials, double* result, cudaStream_t s)
{
    const long long Q = (d + 3) / 4;
    const int blocks = reduce_blocks(Q);
    if (vec)
        quadratic_loss_kernel<true><<<blocks, kReduceBlock, 0, s>>>(x, b, n, d, ld, Q, partials);
    else
        quadratic_loss_kernel<false><<<blocks, kReduceBlock, 0, s>>>(x, b, n, d, ld, Q, partials);
    final_sum_kernel<<<1, 32, 0, s>>>(partials, blocks, 0.5 / (double)n, result);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Seeded fills
// ---------------------------------------------------------------------------
template <bool VEC>
__global__ void __launch_bounds__(kBlock) init_b_kernel(float* __restrict__ b, long long n,
                                                        long long d, long long ld, long long Q, uint32_t q_base,
                                                        uint32_t row0, float shift, const PhiloxKeys keys)
{
    const long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= Q) return;
    for (long long i = 0; i < n; ++i) {   // local row i is node row0 + i of the whole problem
        float4 z = normal4(q_base + (uint32_t)q, row0 + (uint32_t)i, 0u, 1u, keys);
        if (shift != 0.0f) {
            const float s = normal4(0u, row0 + (uint32_t)i, 0u, 3u, keys).x;
            z.x = fmaf(shift, s, z.x);
            z.y = fmaf(shift, s, z.y);
            z.z = fmaf(shift, s, z.z);
            z.w = fmaf(shift, s, z.w);
        }
        store4<VEC>(b + i * ld, q * 4, d, z);
    }
}

template <bool VEC>
__global__ void __launch_bounds__(kBlock) init_x0_kernel(float* __restrict__ x, long long n,
                                                         long long d, long long ld, long long Q, uint32_t q_base,
                                                         uint32_t row0, int kind, float std, const PhiloxKeys keys)
{
    const long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= Q) return;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (kind == 1) v = scale4(normal4(q_base + (uint32_t)q, 0u, 0u, 2u, keys), std);
    for (long long i = 0; i < n; ++i) {
        if (kind == 2) v = scale4(normal4(q_base + (uint32_t)q, row0 + (uint32_t)i, 0u, 2u, keys), std);
        store4<VEC>(x + i * ld, q * 4, d, v);
    }
}

cudaError_t launch_init_b(float* b, long long n, long long d, long long ld, uint32_t q_base, uint32_t row0, float shift,
                          bool vec, const PhiloxKeys& keys, cudaStream_t s)
{
    const long long Q = (d + 3) / 4;
    if (vec)
        init_b_kernel<true><<<grid_for(Q, kBlock), kBlock, 0, s>>>(b, n, d, ld, Q, q_base, row0, shift, keys);
    else
        init_b_kernel<false><<<grid_for(Q, kBlock), kBlock, 0, s>>>(b, n, d, ld, Q, q_base, row0, shift, keys);
    return cudaGetLastError();
}

cudaError_t launch_init_x0(float* x, long long n, long long d, long long ld, uint32_t q_base, uint32_t row0, int kind,
                           float std, bool vec, const PhiloxKeys& keys, cudaStream_t s)
{
    const long long Q = (d + 3) / 4;
    if (vec)
        init_x0_kernel<true><<<grid_for(Q, kBlock), kBlock, 0, s>>>(x, n, d, ld, Q, q_base, row0, kind, std, keys);
    else
        init_x0_kernel<false><<<grid_for(Q, kBlock), kBlock, 0, s>>>(x, n, d, ld, Q, q_base, row0, kind, std, keys);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Generator surface
// ---------------------------------------------------------------------------
__global__ void philox_words_kernel(const uint32_t* __restrict__ ctr, const PhiloxKeys keys,
                                    long long count, uint32_t* __restrict__ out)
{
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= count) return;
    const uint4 w = philox4x32_10(ctr[4 * t], ctr[4 * t + 1], ctr[4 * t + 2], ctr[4 * t + 3], keys);
    out[4 * t] = w.x;
    out[4 * t + 1] = w.y;
    out[4 * t + 2] = w.z;
    out[4 * t + 3] = w.w;
}

__global__ void box_muller_words_kernel(const uint32_t* __restrict__ a, const uint32_t* __restrict__ b,
                                        long long count, float* __restrict__ z)
{
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= count) return;
    const float2 v = box_muller(a[t], b[t]);
    z[2 * t] = v.x;
    z[2 * t + 1] = v.y;
}

__global__ void normal_fill_kernel(const PhiloxKeys keys, uint32_t stream_id, uint32_t k, uint32_t i,
                                   uint32_t q0, long long count, float* __restrict__ out)
{
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= count) return;
    const float4 z = normal4(q0 + (uint32_t)t, i, k, stream_id, keys);
    out[4 * t] = z.x;
    out[4 * t + 1] = z.y;
    out[4 * t + 2] = z.z;
    out[4 * t + 3] = z.w;
}

cudaError_t launch_philox_words(const uint32_t* ctr, PhiloxKeys keys, long long count, uint32_t* out,
                                cudaStream_t s)
{
    if (count > 0) philox_words_kernel<<<grid_for(count, kBlock), kBlock, 0, s>>>(ctr, keys, count, out);
    return cudaGetLastError();
}
cudaError_t launch_box_muller_words(const uint32_t* a, const uint32_t* b, long long count, float* z,
                                    cudaStream_t s)
{
    if (count > 0) box_muller_words_kernel<<<grid_for(count, kBlock), kBlock, 0, s>>>(a, b, count, z);
    return cudaGetLastError();
}
cudaError_t launch_normal_fill(PhiloxKeys keys, uint32_t stream_id, uint32_t k, uint32_t i,
                               uint32_t q0, long long count, float* out, cudaStream_t s)
{
    if (count > 0)
        normal_fill_kernel<<<grid_for(count, kBlock), kBlock, 0, s>>>(keys, stream_id, k, i, q0, count, out);
    return cudaGetLastError();
}

}  // namespace gpga
