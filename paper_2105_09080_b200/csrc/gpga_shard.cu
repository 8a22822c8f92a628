// Node-sharded Gossip-PGA: the n nodes (rows of X) are split over several devices, each
// holding n_l = n / shards consecutive nodes and all d columns -- the deployment of Section 3,
// where a gossip step exchanges half-step parameter vectors x^(k+1/2) between neighbouring nodes
// and the global average is an All-Reduce.  One iteration of Algorithm 1 on a shard is two
// kernels with an exchange between them:
//
//   export : form the half-step rows y = x - gamma g that OTHER shards need (ring: the first and
//            the last local row; one-peer exponential graph with hop h: the first min(h, n_l)
//            local rows; global average: the shard's column sums over its rows) -> send buffer
//   -- the caller moves send buffers into the peers' receive buffers (a copy, or NCCL) --
//   step   : the fused local update + mix over the local rows, reading what was received where
//            a neighbour is not local (ring: the row above the first and below the last local
//            row; exponential graph: the partner rows; global average: all shards' column sums)
//
// Every result is formed by the operations, in the order, of the unsharded kernels (ring:
// (up + self) + down; exponential graph: (y_i + y_partner) / 2; column mean: rows added pairwise
// in fp32 in groups of four, group sums accumulated in fp64 in row order -- shard boundaries
// fall on multiples of four rows -- and the shards' fp64 sums added in shard order), so a
// sharded run agrees with the unsharded one bit for bit whenever the fp64 accumulation of a
// column is exact (always, unless magnitudes inside one column differ by more than 2^29), and to
// one fp64 rounding otherwise.  Remote rows are only ever read from this device's own memory.
#include "gpga_shard.cuh"

namespace gpga {

namespace {

constexpr int kShardBlock = 256;

struct Group {
    long long j0;   // first local column
    uint32_t qg;    // global group index (first counter word of the generator)
};

__device__ __forceinline__ Group group_of(const ShardParams& p, long long q)
{
    Group g;
    g.j0 = q * 4;
    g.qg = p.q_base + (uint32_t)q;
    return g;
}

// One local row's inputs for one column group, and the half-step formed from them (Algorithm 1:
// gradient, local update).  Loading and finishing are split so that a thread can issue the loads of
// several rows before it stores anything: the output may alias the input (in-place update), so the
// compiler cannot move a load above a store by itself.
struct RowIn {
    float4 x, b;
};
template <bool VEC>
__device__ __forceinline__ RowIn load_row(const ShardParams& p, const Group& g, int i)
{
    RowIn r;
    r.x = load4<VEC>(p.x + (long long)i * p.ld, g.j0, p.d);
    r.b = load4<VEC>(p.b + (long long)i * p.ldb, g.j0, p.d);
    return r;
}
template <int NOISE>   // a ShardGrad
__device__ __forceinline__ float4 finish_row(const ShardParams& p, const Group& g, const RowIn& r, int i)
{
    float4 gr;
    if (NOISE == SHARD_GRAD_BUFFER) {
        gr = r.b;   // the gradient was formed by another kernel (logistic objective)
    } else {
        gr = sub4(r.x, r.b);
        if (NOISE == SHARD_GRAD_QUAD_NOISE) gr = fma4(p.sigma, normal4(g.qg, (uint32_t)(p.row0 + i), p.k, 0u, p.keys), gr);
    }
    return fma4(-p.gamma, gr, r.x);
}
template <int NOISE, bool VEC>
__device__ __forceinline__ float4 half_step_row(const ShardParams& p, const Group& g, int i)
{
    return finish_row<NOISE>(p, g, load_row<VEC>(p, g, i), i);
}

constexpr int kRowsInFlight = 4;

template <bool VEC>
__device__ __forceinline__ float4 load_dense(const float* buf, long long row, const ShardParams& p, const Group& g)
{
    // exchange buffers are dense: row stride d4 * 4 floats (d rounded up to a whole group)
    const long long pitch = p.Q * 4;
    return load4<true>(buf + row * pitch + g.j0, 0, 0);
}
__device__ __forceinline__ void store_dense(float* buf, long long row, const ShardParams& p, const Group& g, float4 v)
{
    store4<true>(buf + row * p.Q * 4 + g.j0, 0, 0, v);
}

template <bool VEC>
__device__ __forceinline__ void store_out(const ShardParams& p, const Group& g, int i, float4 v)
{
    store4<VEC>(p.out + (long long)i * p.ld, g.j0, p.d, v);
}

__device__ __forceinline__ float4 mix3(float4 a, float4 b, float4 c)
{
    return scale4(add4(add4(a, b), c), 0.333333343f);
}
__device__ __forceinline__ float4 half(float4 a, float4 b) { return scale4(add4(a, b), 0.5f); }

// ---- export ------------------------------------------------------------------------------------
// send[t][:] = half-step of local row first + t * stride, t < rows.
template <int NOISE, bool VEC>
__global__ void __launch_bounds__(kShardBlock) shard_export_rows_kernel(const ShardParams p, float* __restrict__ send,
                                                                         int first, int stride, int rows)
{
    const long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= p.Q) return;
    const Group g = group_of(p, q);
    int t = 0;
    for (; t + kRowsInFlight <= rows; t += kRowsInFlight) {
        RowIn r[kRowsInFlight];
#pragma unroll
        for (int u = 0; u < kRowsInFlight; ++u) r[u] = load_row<VEC>(p, g, first + (t + u) * stride);
#pragma unroll
        for (int u = 0; u < kRowsInFlight; ++u)
            store_dense(send, t + u, p, g, finish_row<NOISE>(p, g, r[u], first + (t + u) * stride));
    }
    for (; t < rows; ++t) store_dense(send, t, p, g, half_step_row<NOISE, VEC>(p, g, first + t * stride));
}

// Column sums of the half-step over the local rows, as the global-average kernel forms them:
// rows pairwise in fp32 in groups of four, groups in fp64 in row order.  sums[4 q .. 4 q + 3].
template <int NOISE, bool VEC>
__global__ void __launch_bounds__(kShardBlock) shard_export_sums_kernel(const ShardParams p, double* __restrict__ sums)
{
    const long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= p.Q) return;
    const Group g = group_of(p, q);
    double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
    const int n = (int)p.n;
    int i = 0;
    for (; i + 4 <= n; i += 4) {
        RowIn r[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) r[u] = load_row<VEC>(p, g, i + u);
        const float4 y0 = finish_row<NOISE>(p, g, r[0], i), y1 = finish_row<NOISE>(p, g, r[1], i + 1);
        const float4 y2 = finish_row<NOISE>(p, g, r[2], i + 2), y3 = finish_row<NOISE>(p, g, r[3], i + 3);
        const float4 t = add4(add4(y0, y1), add4(y2, y3));
        s0 += (double)t.x; s1 += (double)t.y; s2 += (double)t.z; s3 += (double)t.w;
    }
    const int rest = n - i;   // an unfinished last group (only when the shard is the whole problem)
    if (rest >= 1) {
        float4 a = half_step_row<NOISE, VEC>(p, g, i);
        if (rest >= 2) a = add4(a, half_step_row<NOISE, VEC>(p, g, i + 1));
        s0 += (double)a.x; s1 += (double)a.y; s2 += (double)a.z; s3 += (double)a.w;
    }
    if (rest == 3) {
        const float4 b = half_step_row<NOISE, VEC>(p, g, i + 2);
        s0 += (double)b.x; s1 += (double)b.y; s2 += (double)b.z; s3 += (double)b.w;
    }
    double* o = sums + 4 * q;
    o[0] = s0; o[1] = s1; o[2] = s2; o[3] = s3;
}

// ---- export with the send fused in ---------------------------------------------------------------
// The same rows, stored straight to where their receivers will read them instead of (or besides) a
// send buffer: row t goes to dst0 row t when t < split, else to dst1 row t - split (ring: split = 1,
// the first row to the shard above, the last one to the shard below; exponential graph: all rows to
// the one partner shard).  dst0 / dst1 may be another device's memory mapped for peer access: the
// kernel only stores there, 16 bytes per thread and row, adjacent threads adjacent addresses.
// `keep` (may be null) also gets every row, for a step that averages the exported rows themselves.
template <int NOISE, bool VEC>
__global__ void __launch_bounds__(kShardBlock) shard_export_rows_to_kernel(const ShardParams p, float* __restrict__ keep,
                                                                            float* __restrict__ dst0,
                                                                            float* __restrict__ dst1, int split,
                                                                            int first, int stride, int rows)
{
    const long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= p.Q) return;
    const Group g = group_of(p, q);
    auto put = [&](int t, float4 y) {
        if (t < split) store_dense(dst0, t, p, g, y);
        else store_dense(dst1, t - split, p, g, y);
        if (keep) store_dense(keep, t, p, g, y);
    };
    int t = 0;
    for (; t + kRowsInFlight <= rows; t += kRowsInFlight) {
        RowIn r[kRowsInFlight];
#pragma unroll
        for (int u = 0; u < kRowsInFlight; ++u) r[u] = load_row<VEC>(p, g, first + (t + u) * stride);
#pragma unroll
        for (int u = 0; u < kRowsInFlight; ++u) put(t + u, finish_row<NOISE>(p, g, r[u], first + (t + u) * stride));
    }
    for (; t < rows; ++t) put(t, half_step_row<NOISE, VEC>(p, g, first + t * stride));
}

// The shard's column sums, stored into every shard's gather area (its own included): an all-gather
// done by the producer's stores.  Same sums, formed in the same order, as shard_export_sums_kernel.
template <int NOISE, bool VEC>
__global__ void __launch_bounds__(kShardBlock) shard_export_sums_to_kernel(const ShardParams p, const ShardSumDests dl)
{
    const long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= p.Q) return;
    const Group g = group_of(p, q);
    double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
    const int n = (int)p.n;
    int i = 0;
    for (; i + 4 <= n; i += 4) {
        RowIn r[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) r[u] = load_row<VEC>(p, g, i + u);
        const float4 y0 = finish_row<NOISE>(p, g, r[0], i), y1 = finish_row<NOISE>(p, g, r[1], i + 1);
        const float4 y2 = finish_row<NOISE>(p, g, r[2], i + 2), y3 = finish_row<NOISE>(p, g, r[3], i + 3);
        const float4 t = add4(add4(y0, y1), add4(y2, y3));
        s0 += (double)t.x; s1 += (double)t.y; s2 += (double)t.z; s3 += (double)t.w;
    }
    const int rest = n - i;
    if (rest >= 1) {
        float4 a = half_step_row<NOISE, VEC>(p, g, i);
        if (rest >= 2) a = add4(a, half_step_row<NOISE, VEC>(p, g, i + 1));
        s0 += (double)a.x; s1 += (double)a.y; s2 += (double)a.z; s3 += (double)a.w;
    }
    if (rest == 3) {
        const float4 b = half_step_row<NOISE, VEC>(p, g, i + 2);
        s0 += (double)b.x; s1 += (double)b.y; s2 += (double)b.z; s3 += (double)b.w;
    }
    for (int t = 0; t < dl.count; ++t) {
        double2* o = reinterpret_cast<double2*>(dl.dst[t] + 4 * q);
        o[0] = make_double2(s0, s1);
        o[1] = make_double2(s2, s3);
    }
}

// ---- step --------------------------------------------------------------------------------------
// Ring: recv[0] = half-step of the node above local row 0, recv[1] = of the node below the last.
// A three-row window slides down the local rows, four rows' loads in flight.
// interior = true: only the rows whose neighbours are both local (1 .. n - 2); recv is not read.
template <int NOISE, bool VEC>
__global__ void __launch_bounds__(kShardBlock, 3) shard_ring_kernel(const ShardParams p, const float* __restrict__ recv,
                                                                     bool interior)
{
    const long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= p.Q) return;
    const Group g = group_of(p, q);
    const int n = (int)p.n;
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    float4 a = interior ? zero : load_dense<VEC>(recv, 0, p, g);
    const float4 below = interior ? zero : load_dense<VEC>(recv, 1, p, g);
    float4 b = half_step_row<NOISE, VEC>(p, g, 0);
    int i = 1;
    for (; i + kRowsInFlight <= n; i += kRowsInFlight) {
        RowIn r[kRowsInFlight];
#pragma unroll
        for (int u = 0; u < kRowsInFlight; ++u) r[u] = load_row<VEC>(p, g, i + u);
#pragma unroll
        for (int u = 0; u < kRowsInFlight; ++u) {
            const float4 v = finish_row<NOISE>(p, g, r[u], i + u);
            if (!interior || i + u > 1) store_out<VEC>(p, g, i + u - 1, mix3(a, b, v));
            a = b;
            b = v;
        }
    }
    for (; i < n; ++i) {
        const float4 v = half_step_row<NOISE, VEC>(p, g, i);
        if (!interior || i > 1) store_out<VEC>(p, g, i - 1, mix3(a, b, v));
        a = b;
        b = v;
    }
    if (!interior) store_out<VEC>(p, g, n - 1, mix3(a, b, below));
}

// The two rows of a ring shard that have a remote neighbour: row 0 (the node above it is recv[0])
// and row n - 1 (the node below it is recv[1]); reads local rows 0, 1, n - 2, n - 1.
template <int NOISE, bool VEC>
__global__ void __launch_bounds__(kShardBlock) shard_ring_boundary_kernel(const ShardParams p, const float* __restrict__ recv)
{
    const long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= p.Q) return;
    const Group g = group_of(p, q);
    const int n = (int)p.n;
    const float4 above = load_dense<VEC>(recv, 0, p, g), below = load_dense<VEC>(recv, 1, p, g);
    const RowIn r0 = load_row<VEC>(p, g, 0), r1 = load_row<VEC>(p, g, n > 1 ? 1 : 0);
    const RowIn r2 = load_row<VEC>(p, g, n > 1 ? n - 2 : 0), r3 = load_row<VEC>(p, g, n - 1);
    const float4 y0 = finish_row<NOISE>(p, g, r0, 0);
    if (n == 1) {
        store_out<VEC>(p, g, 0, mix3(above, y0, below));
        return;
    }
    const float4 y1 = finish_row<NOISE>(p, g, r1, 1);
    const float4 yl2 = finish_row<NOISE>(p, g, r2, n - 2), yl1 = finish_row<NOISE>(p, g, r3, n - 1);
    store_out<VEC>(p, g, 0, mix3(above, y0, y1));
    store_out<VEC>(p, g, n - 1, mix3(yl2, yl1, below));
}

// One-peer exponential graph with hop h: he = min(h, n_l) chains c, c + he, c + 2 he, ... of
// L = n_l / he local rows (powers of two); a row's partner is the next row of its chain, the last
// row's partner is recv[c] (the partner shard's row c).  The walk visits step t = c L + s (chain c,
// position s) at row c + s he, four steps' loads in flight; each local row is read, and its noise
// generated, once.
template <int NOISE, bool VEC>
__global__ void __launch_bounds__(kShardBlock, 3) shard_exp_kernel(const ShardParams p, const float* __restrict__ recv,
                                                                    int he_log2, int len_log2, bool interior)
{
    const long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= p.Q) return;
    const Group g = group_of(p, q);
    const int n = (int)p.n, lmask = (1 << len_log2) - 1;
    auto row_of = [=](int t) { return (t >> len_log2) + ((t & lmask) << he_log2); };
    float4 prev = make_float4(0.f, 0.f, 0.f, 0.f);
    int prev_row = 0;
    auto visit = [&](int t, int row, float4 y) {
        const int s = t & lmask;
        if (s != 0) store_out<VEC>(p, g, prev_row, half(prev, y));
        if (s == lmask && !interior) store_out<VEC>(p, g, row, half(y, load_dense<VEC>(recv, t >> len_log2, p, g)));
        prev = y;
        prev_row = row;
    };
    int t = 0;
    for (; t + kRowsInFlight <= n; t += kRowsInFlight) {
        RowIn r[kRowsInFlight];
#pragma unroll
        for (int u = 0; u < kRowsInFlight; ++u) r[u] = load_row<VEC>(p, g, row_of(t + u));
#pragma unroll
        for (int u = 0; u < kRowsInFlight; ++u) {
            const int row = row_of(t + u);
            visit(t + u, row, finish_row<NOISE>(p, g, r[u], row));
        }
    }
    for (; t < n; ++t) {
        const int row = row_of(t);
        visit(t, row, half_step_row<NOISE, VEC>(p, g, row));
    }
}

// The last he local rows of the exponential graph's shard, whose partners are recv[0 .. he - 1].
template <int NOISE, bool VEC>
__global__ void __launch_bounds__(kShardBlock) shard_exp_boundary_kernel(const ShardParams p, const float* __restrict__ recv,
                                                                          int he)
{
    const long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= p.Q) return;
    const Group g = group_of(p, q);
    const int first = (int)p.n - he;
    int c = 0;
    for (; c + kRowsInFlight <= he; c += kRowsInFlight) {
        RowIn r[kRowsInFlight];
        float4 z[kRowsInFlight];
#pragma unroll
        for (int u = 0; u < kRowsInFlight; ++u) {
            r[u] = load_row<VEC>(p, g, first + c + u);
            z[u] = load_dense<VEC>(recv, c + u, p, g);
        }
#pragma unroll
        for (int u = 0; u < kRowsInFlight; ++u)
            store_out<VEC>(p, g, first + c + u, half(finish_row<NOISE>(p, g, r[u], first + c + u), z[u]));
    }
    for (; c < he; ++c)
        store_out<VEC>(p, g, first + c, half(half_step_row<NOISE, VEC>(p, g, first + c), load_dense<VEC>(recv, c, p, g)));
}

// The same when every local row's partner is remote (hop >= n_l) and the rows' half-steps are still in
// the send buffer the export wrote: x_i^(k+1) = (send[i] + recv[i]) / 2, 12 bytes per update.
__global__ void __launch_bounds__(kShardBlock) shard_exp_exported_kernel(const ShardParams p, const float* __restrict__ own,
                                                                          const float* __restrict__ recv, bool vec)
{
    const long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= p.Q) return;
    const Group g = group_of(p, q);
    const int n = (int)p.n;
    int i = 0;
    for (; i + kRowsInFlight <= n; i += kRowsInFlight) {
        float4 y[kRowsInFlight], z[kRowsInFlight];
#pragma unroll
        for (int u = 0; u < kRowsInFlight; ++u) {
            y[u] = load_dense<true>(own, i + u, p, g);
            z[u] = load_dense<true>(recv, i + u, p, g);
        }
#pragma unroll
        for (int u = 0; u < kRowsInFlight; ++u) {
            if (vec) store_out<true>(p, g, i + u, half(y[u], z[u]));
            else store_out<false>(p, g, i + u, half(y[u], z[u]));
        }
    }
    for (; i < n; ++i) {
        const float4 v = half(load_dense<true>(own, i, p, g), load_dense<true>(recv, i, p, g));
        if (vec) store_out<true>(p, g, i, v);
        else store_out<false>(p, g, i, v);
    }
}

// Global average: recv holds `parts` vectors of column sums (4 Q doubles each), one per shard in
// shard order; mean = (sum of the parts in that order) / n_total, rounded once, to every local row.
template <bool VEC>
__global__ void __launch_bounds__(kShardBlock) shard_global_kernel(const ShardParams p, const double* __restrict__ recv,
                                                                    int parts)
{
    const long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= p.Q) return;
    const Group g = group_of(p, q);
    double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
    for (int t = 0; t < parts; ++t) {
        const double* v = recv + ((long long)t * p.Q + q) * 4;
        s0 += v[0]; s1 += v[1]; s2 += v[2]; s3 += v[3];
    }
    const double inv = (double)p.n_total;
    const float4 m = make_float4((float)(s0 / inv), (float)(s1 / inv), (float)(s2 / inv), (float)(s3 / inv));
    const int n = (int)p.n;
    for (int i = 0; i < n; ++i) store_out<VEC>(p, g, i, m);
}

unsigned grid_of(long long Q) { return (unsigned)((Q + kShardBlock - 1) / kShardBlock); }

}  // namespace

#define GPGA_SHARD_LAUNCH(kernel, noise, vec, ...)                                                                   \
    do {                                                                                                             \
        if (noise == SHARD_GRAD_QUAD_NOISE) {                                                                        \
            if (vec) kernel<SHARD_GRAD_QUAD_NOISE, true><<<grid_of(p.Q), kShardBlock, 0, s>>>(__VA_ARGS__);          \
            else kernel<SHARD_GRAD_QUAD_NOISE, false><<<grid_of(p.Q), kShardBlock, 0, s>>>(__VA_ARGS__);             \
        } else if (noise == SHARD_GRAD_QUAD) {                                                                       \
            if (vec) kernel<SHARD_GRAD_QUAD, true><<<grid_of(p.Q), kShardBlock, 0, s>>>(__VA_ARGS__);                \
            else kernel<SHARD_GRAD_QUAD, false><<<grid_of(p.Q), kShardBlock, 0, s>>>(__VA_ARGS__);                   \
        } else {                                                                                                     \
            if (vec) kernel<SHARD_GRAD_BUFFER, true><<<grid_of(p.Q), kShardBlock, 0, s>>>(__VA_ARGS__);              \
            else kernel<SHARD_GRAD_BUFFER, false><<<grid_of(p.Q), kShardBlock, 0, s>>>(__VA_ARGS__);                 \
        }                                                                                                            \
    } while (0)

cudaError_t launch_shard_export_rows(const ShardParams& p, bool vec, float* send, int first, int stride, int rows,
                                     cudaStream_t s)
{
    const int noise = p.grad;
    GPGA_SHARD_LAUNCH(shard_export_rows_kernel, noise, vec, p, send, first, stride, rows);
    return cudaGetLastError();
}

cudaError_t launch_shard_export_sums(const ShardParams& p, bool vec, double* sums, cudaStream_t s)
{
    const int noise = p.grad;
    GPGA_SHARD_LAUNCH(shard_export_sums_kernel, noise, vec, p, sums);
    return cudaGetLastError();
}

cudaError_t launch_shard_export_rows_to(const ShardParams& p, bool vec, float* keep, float* dst0, float* dst1, int split,
                                        int first, int stride, int rows, cudaStream_t s)
{
    const int noise = p.grad;
    GPGA_SHARD_LAUNCH(shard_export_rows_to_kernel, noise, vec, p, keep, dst0, dst1, split, first, stride, rows);
    return cudaGetLastError();
}

cudaError_t launch_shard_export_sums_to(const ShardParams& p, bool vec, const ShardSumDests& dl, cudaStream_t s)
{
    const int noise = p.grad;
    GPGA_SHARD_LAUNCH(shard_export_sums_to_kernel, noise, vec, p, dl);
    return cudaGetLastError();
}

cudaError_t launch_shard_ring(const ShardParams& p, bool vec, const float* recv, int part, cudaStream_t s)
{
    const int noise = p.grad;
    if (part == SHARD_BOUNDARY)
        GPGA_SHARD_LAUNCH(shard_ring_boundary_kernel, noise, vec, p, recv);
    else
        GPGA_SHARD_LAUNCH(shard_ring_kernel, noise, vec, p, recv, part == SHARD_INTERIOR);
    return cudaGetLastError();
}

cudaError_t launch_shard_exp(const ShardParams& p, bool vec, const float* recv, int he, int part, cudaStream_t s)
{
    const int noise = p.grad;
    if (part == SHARD_BOUNDARY) {
        GPGA_SHARD_LAUNCH(shard_exp_boundary_kernel, noise, vec, p, recv, he);
        return cudaGetLastError();
    }
    int he_log2 = 0, len_log2 = 0;
    while ((1 << (he_log2 + 1)) <= he) ++he_log2;
    while (((long long)he << (len_log2 + 1)) <= p.n) ++len_log2;
    GPGA_SHARD_LAUNCH(shard_exp_kernel, noise, vec, p, recv, he_log2, len_log2, part == SHARD_INTERIOR);
    return cudaGetLastError();
}

cudaError_t launch_shard_exp_exported(const ShardParams& p, bool vec, const float* own, const float* recv, cudaStream_t s)
{
    shard_exp_exported_kernel<<<grid_of(p.Q), kShardBlock, 0, s>>>(p, own, recv, vec);
    return cudaGetLastError();
}

cudaError_t launch_shard_global(const ShardParams& p, bool vec, const double* recv, int parts, cudaStream_t s)
{
    if (vec)
        shard_global_kernel<true><<<grid_of(p.Q), kShardBlock, 0, s>>>(p, recv, parts);
    else
        shard_global_kernel<false><<<grid_of(p.Q), kShardBlock, 0, s>>>(p, recv, parts);
    return cudaGetLastError();
}

}  // namespace gpga
