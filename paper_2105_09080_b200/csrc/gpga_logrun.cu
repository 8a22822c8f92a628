// Many Gossip-PGA iterations of the logistic objective in ONE launch (Algorithm 1 with the
// Section 5.1 loss), for states narrow enough that an iteration per launch is bound by the
// launch-to-launch dependency chain rather than by memory.
//
// A pair of blocks (one thread-block cluster of two) owns node i for the whole run:
//  - x_i stays on chip (every warp holds it in registers);
//  - the batch rows of A stream into per-warp shared-memory buffers by bulk asynchronous
//    copies, the copies of the next iteration's rows (their indices depend only on the seed,
//    the node and the iteration) already in flight while this iteration is reduced and mixed,
//    and the rows that no buffer is free for asked into L2 an iteration before they are copied;
//  - the per-warp gradient sums are added in shared memory; the chunk sums go to BOTH blocks of the
//    pair by asynchronous stores into their shared memory, which count themselves off on an
//    mbarrier there (no cluster-wide barrier in the loop); each block then finishes all columns
//    for itself (gradient, local update y_i = x_i - gamma g_i), so x_i^(k+1) never has to cross
//    from one block to the other, and publishes one half of them;
//  - y_i is published to global memory as 64-bit words (value, iteration tag), each written and
//    read whole, so a reader needs no flag and no fence: both blocks read the rows of the node's
//    neighbours (ring, one-peer exponential graph) or the column means (global average) until
//    the tags are this iteration's and form x_i^(k+1), which goes to the block's warps through
//    shared memory.
// Every sum is formed in the order the one-iteration kernels use (rows of a warp in order,
// eight warps of a chunk in order, chunks in order; ring (up + self) + down; global mean by
// groups of four rows in fp32, groups in fp64), so a run is bit-identical to the same number of
// single steps.
//
// Buffers of published rows.  Gossip iteration `it` of the launch uses buffer it % G, global-average
// iterations alternate between two buffers of their own.  A block overwrites what it published G
// gossip iterations (two global averages) earlier; every reader is done with that by then:
// on the ring a node publishes iteration it only after its neighbours' rows of it - 1, which they
// publish after reading its row of it - 2 (G = 2); on the one-peer exponential graph a node at
// iteration it has, through log2 n hops, waited for every node's row of it - log2 n
// (G = log2 n + 2); a global average waits for every node, and the one before it was read
// before those rows were published.
//
// Waiting: a block only waits for data of the SAME iteration, which its owner publishes before it
// waits for anything of that iteration, so the waits cannot form a cycle as long as all blocks
// are resident (checked against the device's capacity before the launch).
// Every wait is bounded; one that gives up raises the error word and a stop word that ends the
// other blocks' waits.  Both blocks of a pair meet at a cluster barrier before they exit, so no
// asynchronous store is ever aimed at a block that has left.
#include <cooperative_groups.h>

#include "../../include/gpga.h"
#include "gpga_launch.cuh"
#include "gpga_logrun.cuh"
#include "gpga_tma.cuh"

namespace cg = cooperative_groups;

namespace gpga {

constexpr int kRunThreads = 512;
constexpr int kRunWarps = kRunThreads / 32;   // 16 = two chunks of eight row-warps per block
constexpr int kRunMaxD = 1024;
constexpr int kRunGroups = kRunMaxD / 4 / 32;   // float4 per lane
constexpr int kRunMaxSlots = 4;                 // row buffers per warp
constexpr int kRunChunkRows = 32, kRunChunkWarps = 8;   // the batch is cut as by the one-iteration kernel
constexpr int kRunMaxChunks = 2 * kRunWarps / kRunChunkWarps;   // 4: batch <= 128
constexpr int kRunMaxNodes = 88;
constexpr int kRunSmemLimit = 226 * 1024;       // dynamic; the static arrays take under 1 KB

__device__ __forceinline__ int ld_relaxed_gpu(const int* p)
{
    int v;
    asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_gpu(int* p, int v)
{
    asm volatile("st.relaxed.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// ---- published rows: (value, tag) words -------------------------------------------------------
// A group of four columns is four 64-bit words, low half the fp32 value, high half the tag.  Each
// word is written and read by one 64-bit access, so a word whose tag matches carries its value.
__device__ __forceinline__ void publish4(unsigned long long* dst, float4 v, uint32_t tag)
{
    const unsigned long long t = (unsigned long long)tag << 32;
    const unsigned long long w0 = t | __float_as_uint(v.x), w1 = t | __float_as_uint(v.y);
    const unsigned long long w2 = t | __float_as_uint(v.z), w3 = t | __float_as_uint(v.w);
    asm volatile("st.relaxed.gpu.global.v2.b64 [%0], {%1, %2};" ::"l"(dst), "l"(w0), "l"(w1) : "memory");
    asm volatile("st.relaxed.gpu.global.v2.b64 [%0], {%1, %2};" ::"l"(dst + 2), "l"(w2), "l"(w3) : "memory");
}
// Reads the group until all four tags equal `tag`.  Gives up after `tries` reads, or as soon
// as *stop is set; returns false then (v is not meaningful).
__device__ __forceinline__ bool read4(const unsigned long long* src, uint32_t tag, const int* stop, uint32_t tries,
                                      float4* v)
{
    for (uint32_t t = 0; t < tries; ++t) {
        unsigned long long w0, w1, w2, w3;
        asm volatile("ld.relaxed.gpu.global.v2.b64 {%0, %1}, [%2];" : "=l"(w0), "=l"(w1) : "l"(src) : "memory");
        asm volatile("ld.relaxed.gpu.global.v2.b64 {%0, %1}, [%2];" : "=l"(w2), "=l"(w3) : "l"(src + 2) : "memory");
        const uint32_t t0 = (uint32_t)(w0 >> 32), t1 = (uint32_t)(w1 >> 32), t2 = (uint32_t)(w2 >> 32),
                       t3 = (uint32_t)(w3 >> 32);
        if (t0 == tag && t1 == tag && t2 == tag && t3 == tag) {
            *v = make_float4(__uint_as_float((uint32_t)w0), __uint_as_float((uint32_t)w1),
                             __uint_as_float((uint32_t)w2), __uint_as_float((uint32_t)w3));
            return true;
        }
        if ((t & 63u) == 63u && ld_relaxed_gpu(stop) != 0) return false;
    }
    return false;
}

// One read of the group, no retry: true if all four tags equal `tag`.
__device__ __forceinline__ bool try4(const unsigned long long* src, uint32_t tag, float4* v)
{
    unsigned long long w0, w1, w2, w3;
    asm volatile("ld.relaxed.gpu.global.v2.b64 {%0, %1}, [%2];" : "=l"(w0), "=l"(w1) : "l"(src) : "memory");
    asm volatile("ld.relaxed.gpu.global.v2.b64 {%0, %1}, [%2];" : "=l"(w2), "=l"(w3) : "l"(src + 2) : "memory");
    *v = make_float4(__uint_as_float((uint32_t)w0), __uint_as_float((uint32_t)w1), __uint_as_float((uint32_t)w2),
                     __uint_as_float((uint32_t)w3));
    return (uint32_t)(w0 >> 32) == tag && (uint32_t)(w1 >> 32) == tag && (uint32_t)(w2 >> 32) == tag &&
           (uint32_t)(w3 >> 32) == tag;
}
// Polls one word until its tag equals `tag` (bounded, ends on the stop word).
__device__ __forceinline__ bool wait_tag(const unsigned long long* word, uint32_t tag, const int* stop, uint32_t tries)
{
    for (uint32_t t = 0; t < tries; ++t) {
        unsigned long long w;
        asm volatile("ld.relaxed.gpu.global.b64 %0, [%1];" : "=l"(w) : "l"(word) : "memory");
        if ((uint32_t)(w >> 32) == tag) return true;
        if ((t & 63u) == 63u && ld_relaxed_gpu(stop) != 0) return false;
    }
    return false;
}
// The same for a whole warp reading 32 adjacent groups of one row, all written by one warp of the
// publisher with the same two store instructions: lane 0 alone polls the last word of the segment
// (`gate`), then every active lane reads and checks its own group (and keeps reading in the rare
// case that its words are not there yet).  One poller per warp keeps the polling traffic small.
// The whole warp must call.
__device__ __forceinline__ bool read4_warp(bool active, const unsigned long long* src, const unsigned long long* gate,
                                           uint32_t tag, const int* stop, uint32_t tries, float4* v)
{
    int ok = 1;
    if ((threadIdx.x & 31) == 0) {
        ok = 0;
        for (uint32_t t = 0; t < tries; ++t) {
            unsigned long long w;
            asm volatile("ld.relaxed.gpu.global.b64 %0, [%1];" : "=l"(w) : "l"(gate) : "memory");
            if ((uint32_t)(w >> 32) == tag) {
                ok = 1;
                break;
            }
            if ((t & 63u) == 63u && ld_relaxed_gpu(stop) != 0) break;
        }
    }
    ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
    if (!ok) return false;
    return active ? read4(src, tag, stop, tries, v) : true;
}

// ---- counted asynchronous stores into a block of the pair (distributed shared memory) ----------
// Address of a shared-memory location of this block as seen in block `rank` of the cluster.
__device__ __forceinline__ uint32_t cluster_addr(const void* smem_ptr, uint32_t rank)
{
    uint32_t a;
    asm("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a) : "r"(smem_u32(smem_ptr)), "r"(rank));
    return a;
}
// 16 bytes to `dst`; on arrival they count as 16 bytes of the current phase of the barrier at `bar`
// (both cluster addresses of the same block).
__device__ __forceinline__ void send4(uint32_t dst, uint32_t bar, float4 v)
{
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];" ::
                     "r"(dst),
                 "r"(__float_as_uint(v.x)), "r"(__float_as_uint(v.y)), "r"(__float_as_uint(v.z)),
                 "r"(__float_as_uint(v.w)), "r"(bar)
                 : "memory");
}
// Waits for the phase of `bar` with the given parity; gives up after `tries` polls, or as soon
// as *stop is set.
__device__ __forceinline__ bool wait_phase(uint64_t* bar, uint32_t parity, const int* stop, uint32_t tries)
{
    for (uint32_t t = 0; t < tries; ++t) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((t & 255u) == 255u && ld_relaxed_gpu(stop) != 0) return false;
    }
    return false;
}

__device__ __forceinline__ void add4_to(float4& s, const float4 v)
{
    s.x += v.x;
    s.y += v.y;
    s.z += v.z;
    s.w += v.w;
}

// Shared-memory plan for row width d: row buffers [16 warps][slots][d], the (group, row) items of
// a column mean [512], the chunk sums [4][d / 4] and x_i [d].  The per-warp
// gradient sums have no area of their own: a warp parks them in the buffer of the row it consumed
// last, which is refilled only after the chunk sums have been formed.
struct RunSmem {
    int slots;
    size_t bytes;
};
__host__ __device__ inline RunSmem run_smem_plan(int d)
{
    const int d4 = d >> 2;
    RunSmem s;
    const size_t fixed = ((size_t)kRunThreads + (size_t)kRunMaxChunks * d4 + (size_t)d4) * sizeof(float4);
    const size_t per_slot = (size_t)kRunWarps * d * sizeof(float);
    long long slots = ((long long)kRunSmemLimit - (long long)fixed) / (long long)per_slot;
    if (slots > kRunMaxSlots) slots = kRunMaxSlots;
    s.slots = (int)slots;
    s.bytes = fixed + (size_t)(slots > 0 ? slots : 0) * per_slot;
    return s;
}

// FULL: d == kRunMaxD, every lane holds kRunGroups whole groups (no guards in the row loop).
template <bool FULL>
__global__ void __launch_bounds__(kRunThreads, 1) logreg_run_kernel(const LogRunParams p, int slots)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t bars[kRunWarps * kRunMaxSlots];
    __shared__ __align__(8) uint64_t sums_bar;          // the chunk sums of both blocks have arrived
    __shared__ int stage_at[kRunWarps];                 // where each warp parked its gradient sums (float4 index)
    cg::cluster_group cluster = cg::this_cluster();
    const int r = (int)cluster.block_rank();   // which half of the columns this block publishes
    const int i = (int)(blockIdx.x >> 1);      // node
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = p.n, d = p.d, d4 = d >> 2;
    const int h0 = (d4 + 1) >> 1;              // block 0 publishes groups [0, h0), block 1 [h0, d4)
    const int g_lo = r ? h0 : 0;
    const int owned = r ? d4 - h0 : h0;
    const int chunks = (p.batch + kRunChunkRows - 1) / kRunChunkRows;
    const float inv_batch = 1.0f / (float)p.batch;
    const int gossip_bufs = p.nbuf - 2;        // then two buffers for global-average iterations
    const size_t buf_words = (size_t)n * d;

    float* slot_base = reinterpret_cast<float*>(smem_raw);
    float4* items = reinterpret_cast<float4*>(slot_base + (size_t)kRunWarps * slots * d);   // [kRunThreads]
    float4* pbuf = items + kRunThreads;             // [chunk][d4]: the four chunk sums of every group
    float4* xnew = pbuf + kRunMaxChunks * d4;       // [d4]: x_i^(k+1)
    // the same locations in both blocks of the pair, as cluster addresses
    const uint32_t pbuf_at[2] = {cluster_addr(pbuf, 0), cluster_addr(pbuf, 1)};
    const uint32_t sums_bar_at[2] = {cluster_addr(&sums_bar, 0), cluster_addr(&sums_bar, 1)};
    const int* stop = p.stop;

    // ---- this warp's rows: warp (chunk c, w) of the one-iteration kernel ----------------------
    const int pair = r * kRunWarps + warp;
    const int c = pair / kRunChunkWarps, w = pair % kRunChunkWarps;
    const int nrows_c = c < chunks ? min(kRunChunkRows, p.batch - c * kRunChunkRows) : 0;
    const int my_rows = w < nrows_c ? (nrows_c - w + kRunChunkWarps - 1) / kRunChunkWarps : 0;
    const int depth = min(slots, my_rows);   // copies this warp keeps in flight
    const uint32_t t_mine = (uint32_t)(c * kRunChunkRows + w + lane * kRunChunkWarps);   // lane rho <-> row rho
    const float* A = p.A + (long long)i * p.m * d;
    const float* labels = p.y + (long long)i * p.m;
    float* mine = slot_base + (size_t)warp * slots * d;
    uint64_t* bar = bars + warp * kRunMaxSlots;
    const uint32_t row_bytes = (uint32_t)d * 4u;

    uint32_t idx_cur = 0u, idx_nxt = 0u;   // lane rho: row rho of this / the next iteration
    float y_cur = 0.f, y_nxt = 0.f;
    if (lane < my_rows) {
        idx_cur = batch_row(t_mine, (uint32_t)i, p.k0, (uint32_t)p.m, p.keys);
        y_cur = labels[idx_cur];
        if (lane >= slots) bulk_prefetch_l2(A + (long long)idx_cur * d, row_bytes);   // not copied yet
        if (p.steps > 1) {
            idx_nxt = batch_row(t_mine, (uint32_t)i, p.k0 + 1u, (uint32_t)p.m, p.keys);
            y_nxt = labels[idx_nxt];
            bulk_prefetch_l2(A + (long long)idx_nxt * d, row_bytes);
        }
    }
    if (lane == 0) {
        for (int s = 0; s < slots; ++s) mbar_init(&bar[s], 1);
        if (warp == 0) mbar_init(&sums_bar, 1);
        mbar_init_fence();
    }
    __syncwarp();
    // Row rho of local iteration it is position it * my_rows + rho of this warp's stream; position q
    // goes through buffer q % depth, phase (q / depth) & 1 of its barrier.
    int issued = 0, consumed = 0;
    int issue_slot = 0, wait_slot = 0;
    uint32_t wait_parity = 0u;
    auto issue = [&](uint32_t idx) {   // whole warp calls; lane 0 starts the copy
        if (lane == 0) {
            mbar_arrive_expect_tx(&bar[issue_slot], row_bytes);
            bulk_copy_g2s(mine + (size_t)issue_slot * d, A + (long long)idx * d, row_bytes, &bar[issue_slot]);
        }
        issue_slot = (issue_slot + 1 == depth) ? 0 : issue_slot + 1;
        ++issued;
    };
    for (int rho = 0; rho < depth; ++rho) issue(__shfl_sync(0xFFFFFFFFu, idx_cur, rho));
    // the rows of the iteration after the next: indices and labels
    auto roll = [&](int it) {
        idx_cur = idx_nxt;
        y_cur = y_nxt;
        if (it + 2 < p.steps && lane < my_rows) {
            idx_nxt = batch_row(t_mine, (uint32_t)i, p.k0 + (uint32_t)(it + 2), (uint32_t)p.m, p.keys);
            y_nxt = labels[idx_nxt];
        }
    };

    ulonglong2 xr[kRunGroups];   // x_i, group lane + 32 j, as two packed pairs
    const ulonglong2 zero2 = make_ulonglong2(0ull, 0ull);
    {
        const ulonglong2* x4 = reinterpret_cast<const ulonglong2*>(p.x_in + (long long)i * p.ldx);
#pragma unroll
        for (int j = 0; j < kRunGroups; ++j) {
            const int g = lane + 32 * j;
            xr[j] = (FULL || g < d4) ? x4[g] : zero2;
        }
    }
    const bool finisher = tid < d4;      // finishes group tid (in both blocks alike)
    const bool publishes = finisher && tid >= g_lo && tid < g_lo + owned;   // and publishes it
    float4 xo = make_float4(0.f, 0.f, 0.f, 0.f);
    if (finisher) xo = reinterpret_cast<const float4*>(p.x_in + (long long)i * p.ldx)[tid];
    cluster.sync();   // the partner's barriers are set up before anything is sent to them

    bool failed = false;
    int it = 0;
    for (; it < p.steps; ++it) {
        const long long k = (long long)p.k0 + it;
        const uint32_t tag = (uint32_t)it + 1u;
        const uint32_t phase = (uint32_t)it & 1u;
        if (tid == 0) mbar_arrive_expect_tx(&sums_bar, (uint32_t)(chunks * d4) * 16u);   // what this iteration will send to this block
        // ---- gradient sums of this warp's rows ----------------------------------------------------
        ulonglong2 acc[kRunGroups];
#pragma unroll
        for (int j = 0; j < kRunGroups; ++j) acc[j] = zero2;
        bool deferred = false;
        uint32_t deferred_idx = 0u;
        int stage_slot = 0;   // a warp without rows parks its zeros in its first buffer
        for (int rho = 0; rho < my_rows; ++rho) {
            stage_slot = wait_slot;
            if (!__all_sync(0xFFFFFFFFu, mbar_wait_bounded(&bar[wait_slot], wait_parity, p.copy_tries))) {
                failed = true;
                break;
            }
            const ulonglong2* a4 = reinterpret_cast<const ulonglong2*>(mine + (size_t)wait_slot * d);
            ulonglong2 a[kRunGroups];
            f32x2_t z01 = 0ull, z23 = 0ull;   // the four running sums z0 .. z3 of the scalar form
#pragma unroll
            for (int j = 0; j < kRunGroups; ++j) {
                const int g = lane + 32 * j;
                a[j] = (FULL || g < d4) ? a4[g] : zero2;
                z01 = fma2(a[j].x, xr[j].x, z01);
                z23 = fma2(a[j].y, xr[j].y, z23);
            }
            const float2 za = unpack2(z01), zb = unpack2(z23);
            const float z = warp_sum_f((za.x + za.y) + (zb.x + zb.y));   // every lane holds the sum
            ++consumed;
            if (++wait_slot == depth) {
                wait_slot = 0;
                wait_parity ^= 1u;
            }
            // the sum needed every lane's loads, so the buffer is free: start the copy of the row
            // `depth` positions ahead (this iteration's, or the next one's) into it
            const int ahead = rho + depth;
            if (ahead < my_rows) {
                issue(__shfl_sync(0xFFFFFFFFu, idx_cur, ahead));
            } else if (it + 1 < p.steps) {
                const uint32_t idx = __shfl_sync(0xFFFFFFFFu, idx_nxt, ahead - my_rows);
                if (rho + 1 < my_rows) {
                    issue(idx);
                } else {   // the last row's buffer first carries this warp's sums to the chunk sums
                    deferred = true;
                    deferred_idx = idx;
                }
            }
            // the rows of the next iteration that no buffer is free for yet: ask them into L2 now, one
            // per row step (a copy of a row that is in L2 lands in about 640 cycles instead of 1100;
            // asking for every row of the next iteration here was measured and is slower: the requests
            // then compete with the copies this iteration is waiting for)
            if (rho + depth < my_rows && it + 1 < p.steps) {
                const uint32_t later = __shfl_sync(0xFFFFFFFFu, idx_nxt, rho + depth);
                if (lane == 0) bulk_prefetch_l2(A + (long long)later * d, row_bytes);
            }
            const float yr = __shfl_sync(0xFFFFFFFFu, y_cur, rho);
            const float sc = -yr / (1.0f + expf(yr * z));
            const f32x2_t sc2 = pack2(sc, sc);
#pragma unroll
            for (int j = 0; j < kRunGroups; ++j) {
                acc[j].x = fma2(sc2, a[j].x, acc[j].x);
                acc[j].y = fma2(sc2, a[j].y, acc[j].y);
            }
        }
        {
            ulonglong2* stage = reinterpret_cast<ulonglong2*>(mine + (size_t)stage_slot * d);
#pragma unroll
            for (int j = 0; j < kRunGroups; ++j) {
                const int g = lane + 32 * j;
                if (FULL || g < d4) stage[g] = acc[j];
            }
            if (lane == 0) stage_at[warp] = (warp * slots + stage_slot) * d4;
        }
        __syncthreads();
        // ---- chunk sums (eight warps in order), sent to both blocks -------------------------------
        {
            const int cl = tid >> 8, g = tid & 255;
            const int cc = 2 * r + cl;
            if (g < d4 && cc < chunks) {
                const float4* all = reinterpret_cast<const float4*>(slot_base) + g;
                float4 sum = all[stage_at[cl * kRunChunkWarps]];
#pragma unroll
                for (int ww = 1; ww < kRunChunkWarps; ++ww) add4_to(sum, all[stage_at[cl * kRunChunkWarps + ww]]);
                const uint32_t off = (uint32_t)(cc * d4 + g) * 16u;
                send4(pbuf_at[0] + off, sums_bar_at[0], sum);
                send4(pbuf_at[1] + off, sums_bar_at[1], sum);
            }
        }
        __syncthreads();   // every parked sum has been read: the buffers that carried them can be refilled
        if (deferred) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // this warp's writes before the copy's
            issue(deferred_idx);
        }
        const bool finisher_warp = warp * 32 < d4;
        if (!finisher_warp) roll(it);   // off the path that the next iteration waits for
        // ---- gradient, local update (all columns), publication of this block's half of y_i --------
        const bool glob = p.H > 0 && ((k + 1) % p.H) == 0;
        const int buf = glob ? gossip_bufs + (int)(((k + 1) / p.H) & 1) : it % gossip_bufs;
        unsigned long long* ybuf = p.ytag + (size_t)buf * buf_words;
        float4 yv = make_float4(0.f, 0.f, 0.f, 0.f);
        if (finisher) {
            if (!wait_phase(&sums_bar, phase, stop, p.copy_tries)) failed = true;
            float4 gs = pbuf[tid];
            for (int cc = 1; cc < chunks; ++cc) add4_to(gs, pbuf[cc * d4 + tid]);
            const float4 gr = make_float4(fmaf(gs.x, inv_batch, p.l2 * xo.x), fmaf(gs.y, inv_batch, p.l2 * xo.y),
                                          fmaf(gs.z, inv_batch, p.l2 * xo.z), fmaf(gs.w, inv_batch, p.l2 * xo.w));
            yv = make_float4(fmaf(-p.gamma, gr.x, xo.x), fmaf(-p.gamma, gr.y, xo.y), fmaf(-p.gamma, gr.z, xo.z),
                             fmaf(-p.gamma, gr.w, xo.w));
            if (publishes && !failed) publish4(ybuf + (size_t)i * d + 4 * tid, yv, tag);
        }
        // ---- mix ------------------------------------------------------------------------------------
        float4 xp = yv;
        if (glob) {
            // Column mean in two hops.  The column groups of this half are dealt out over the nodes:
            // block (i, r) takes local groups i, i + n, ...; it reads those groups of every node's row,
            // forms their means exactly as the one-iteration kernels do (rows added in fp32 in groups
            // of four, (y0 + y1) + (y2 + y3), the group sums in fp64 in row order) and publishes them;
            // then every block reads the means of all groups.  A block reads n * (groups / 2n) + groups
            // words instead of n * groups.
            const int mine_cnt = i < owned ? (owned - i + n - 1) / n : 0;   // groups this block averages
            unsigned long long* means = p.ytag + (size_t)p.nbuf * buf_words + (size_t)(buf - gossip_bufs) * d;
            if (tid < mine_cnt * n) {
                const int j = tid / n, row = tid - j * n;
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                if (!read4(ybuf + (size_t)row * d + 4 * (g_lo + i + j * n), tag, stop, p.poll_tries, &v)) failed = true;
                items[tid] = v;   // [j][row]
            }
            __syncthreads();
            if (tid < 4 * mine_cnt) {   // four threads per column group, one per component
                const int j = tid >> 2, comp = tid & 3;
                const float* col = reinterpret_cast<const float*>(items + j * n) + comp;   // [row * 4]
                double sum = 0.0;
                int q = 0;
                for (; q + 4 <= n; q += 4)
                    sum += (double)((col[4 * q] + col[4 * (q + 1)]) + (col[4 * (q + 2)] + col[4 * (q + 3)]));
                const int rest = n - q;
                if (rest >= 1) sum += (double)(rest >= 2 ? col[4 * q] + col[4 * (q + 1)] : col[4 * q]);
                if (rest == 3) sum += (double)col[4 * (q + 2)];
                float mean;
                if ((n & (n - 1)) == 0)   // 1/n is exact: the product equals the quotient
                    mean = (float)(sum * (1.0 / (double)n));
                else
                    mean = (float)(sum / (double)n);
                // one (value, tag) word per component
                const unsigned long long word = ((unsigned long long)tag << 32) | __float_as_uint(mean);
                asm volatile("st.relaxed.gpu.global.b64 [%0], %1;" ::"l"(means + 4 * (g_lo + i + j * n) + comp), "l"(word)
                             : "memory");
            }
            if (finisher && !read4(means + 4 * tid, tag, stop, p.poll_tries, &xp)) failed = true;
        } else if (finisher_warp) {
            const int seg_last = min(warp * 32 + 31, d4 - 1);
            const unsigned long long* col = ybuf + 4 * min(tid, d4 - 1);
            const unsigned long long* gate = ybuf + 4 * seg_last + 3;
            if (p.topology == GPGA_TOPO_RING) {
                const int up = (i == 0) ? n - 1 : i - 1, dn = (i == n - 1) ? 0 : i + 1;
                float4 yu = yv, yd = yv;
                if (lane < 2 && !wait_tag(gate + (size_t)(lane ? dn : up) * d, tag, stop, p.poll_tries)) failed = true;
                __syncwarp();
                if (finisher && !failed) {
                    const bool ok_u = try4(col + (size_t)up * d, tag, &yu), ok_d = try4(col + (size_t)dn * d, tag, &yd);
                    if (!ok_u && !read4(col + (size_t)up * d, tag, stop, p.poll_tries, &yu)) failed = true;
                    if (!ok_d && !read4(col + (size_t)dn * d, tag, stop, p.poll_tries, &yd)) failed = true;
                }
                const float third = 0.333333343f;
                xp = make_float4((yu.x + yv.x + yd.x) * third, (yu.y + yv.y + yd.y) * third,
                                 (yu.z + yv.z + yd.z) * third, (yu.w + yv.w + yd.w) * third);
            } else {
                const int hop_log2 = p.log2n > 0 ? (int)(k % p.log2n) : 0;
                const int peer = (i + (1 << hop_log2)) & (n - 1);
                float4 yp = yv;
                if (!read4_warp(finisher, col + (size_t)peer * d, gate + (size_t)peer * d, tag, stop, p.poll_tries, &yp)) failed = true;
                xp = make_float4((yv.x + yp.x) * 0.5f, (yv.y + yp.y) * 0.5f, (yv.z + yp.z) * 0.5f,
                                 (yv.w + yp.w) * 0.5f);
            }
        }
        // ---- x_i^(k+1) to the warps of this block ---------------------------------------------------
        if (finisher && !failed) {
            xnew[tid] = xp;
            if (publishes && it == p.steps - 1) reinterpret_cast<float4*>(p.x_out + (long long)i * p.ldx)[tid] = xp;
        }
        if (finisher_warp) roll(it);
        if (failed) {   // tell everyone; the partner's and the other nodes' waits end on the stop word
            st_relaxed_gpu(p.stop, 1);
            if (p.error_flag) atomicExch(p.error_flag, 1);
        }
        if (__syncthreads_or(failed)) break;
#pragma unroll
        for (int j = 0; j < kRunGroups; ++j) {
            const int g = lane + 32 * j;
            if (FULL || g < d4) xr[j] = reinterpret_cast<const ulonglong2*>(xnew)[g];
        }
        if (finisher) xo = xp;
    }
    // Copies still in flight target this block's shared memory: give each a bounded chance to land
    // (none is in flight after a run that went through).
    for (int q = consumed; q < issued; ++q)
        mbar_wait_bounded(&bar[q % depth], (uint32_t)(q / depth) & 1u, p.copy_tries);
    cluster.sync();   // neither block leaves while the other may still send to it
}

namespace {

cudaError_t run_config(cudaLaunchConfig_t* cfg, cudaLaunchAttribute* attrs, int n, size_t smem, cudaStream_t s)
{
    *cfg = cudaLaunchConfig_t{};
    cfg->gridDim = dim3((unsigned)(2 * n));
    cfg->blockDim = dim3(kRunThreads);
    cfg->dynamicSmemBytes = smem;
    cfg->stream = s;
    attrs[0].id = cudaLaunchAttributeClusterDimension;
    attrs[0].val.clusterDim.x = 2;
    attrs[0].val.clusterDim.y = 1;
    attrs[0].val.clusterDim.z = 1;
    cfg->attrs = attrs;
    cfg->numAttrs = 1;
    static unsigned long long limit_set = 0, limit_set_full = 0;
    const cudaError_t e = ensure_smem_limit(logreg_run_kernel<false>, kRunSmemLimit, limit_set);
    return e != cudaSuccess ? e : ensure_smem_limit(logreg_run_kernel<true>, kRunSmemLimit, limit_set_full);
}

}  // namespace

cudaError_t logreg_run_supported(int n, int d, int batch, int topology, long long H, bool* ok)
{
    *ok = false;
    if (topology != GPGA_TOPO_RING && topology != GPGA_TOPO_EXP) return cudaSuccess;
    if (d < 4 || d > kRunMaxD || (d & 3) != 0 || batch < 1 || batch > kRunChunkRows * kRunMaxChunks) return cudaSuccess;
    if (n < 1 || n > kRunMaxNodes || H < 0 || H >= (1ll << 31)) return cudaSuccess;
    if (run_smem_plan(d).slots < 1) return cudaSuccess;
    // All 2 n blocks must be resident at once: they wait for one another.  The widest rows take the
    // most shared memory, so the number of pairs that fit then holds for every width.
    static int max_clusters[64] = {0};   // per device
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    int& cached = max_clusters[dev & 63];
    if (cached == 0) {
        cudaLaunchConfig_t cfg;
        cudaLaunchAttribute attrs[1];
        e = run_config(&cfg, attrs, kRunMaxNodes, (size_t)kRunSmemLimit, nullptr);
        if (e != cudaSuccess) return e;
        int clusters = 0;
        e = cudaOccupancyMaxActiveClusters(&clusters, logreg_run_kernel<false>, &cfg);
        if (e != cudaSuccess) {
            (void)cudaGetLastError();
            clusters = -1;   // the query is not available: do not use the kernel
        }
        cached = clusters > 0 ? clusters : -1;
    }
    *ok = cached >= n;
    return cudaSuccess;
}

// A plain launch of clusters of two.  Residency of all blocks is what logreg_run_supported checked
// for an otherwise idle device; if other work holds multiprocessors for longer than the kernel's
// bounded waits last, the run ends with the error word set instead of hanging.
cudaError_t launch_logreg_run(const LogRunParams& p, cudaStream_t s)
{
    const RunSmem plan = run_smem_plan(p.d);
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attrs[1];
    // (launch_nodes < n only in the self-test of the bounded waits: the rows of the nodes left out are never published)
    const cudaError_t e = run_config(&cfg, attrs, p.launch_nodes > 0 ? p.launch_nodes : p.n, plan.bytes, s);
    if (e != cudaSuccess) return e;
    return cudaLaunchKernelEx(&cfg, p.d == kRunMaxD ? logreg_run_kernel<true> : logreg_run_kernel<false>, p, plan.slots);
}

}  // namespace gpga
