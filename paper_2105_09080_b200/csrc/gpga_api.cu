// C ABI of libgpga: handle, argument checks, schedule, launches.  See include/gpga.h.
#include <cmath>
#include <cstdio>
#include <new>
#include <string>
#include <vector>

#include "../../include/gpga.h"
#include "gpga_kernels.cuh"
#include "gpga_logreg.cuh"
#include "gpga_logrun.cuh"
#include "gpga_loss.cuh"
#include "gpga_shard.cuh"
#include "gpga_tile.cuh"

using namespace gpga;

// Scratch layout: [reduction partials | result double | G | gradient chunk partials | published rows]
struct ScratchLayout {
    int64_t slots = 0, partials_off = 0, result_off = 0, G_off = 0, chunk_off = 0, ytag_off = 0, ytag_bytes = 0, total = 0;
};

struct gpga_ctx {
    int64_t n = 0, d = 0, H = 0;
    int32_t topology = 0;
    float gamma = 0.f;
    uint64_t seed = 0;
    int32_t objective = GPGA_OBJ_QUADRATIC;
    float sigma = 0.f, l2 = 0.f;
    int64_t m = 0, batch = 0;
    int64_t grid_cols = 0;
    int64_t col0 = 0;
    int64_t ld = 0;   // row stride of X and b in floats
    int64_t shards = 1, shard = 0;   // node sharding: this handle holds nodes shard * n .. (shard + 1) * n - 1
    const void* exported = nullptr;  // send buffer of the last gpga_shard_export and its iteration
    int64_t exported_k = -1;
    int64_t shard_grad_k = -1;       // iteration whose logistic gradient matrix sits in the scratch area
    float* x[2] = {nullptr, nullptr};
    float* data = nullptr;
    const float* labels = nullptr;
    char* scratch = nullptr;
    int64_t scratch_bytes = 0;
    ScratchLayout L;   // layout of the scratch area, fixed by gpga_bind (the host entry narrows d per chunk)
    int cur = 0;
    int64_t k = 0;
    int64_t launches = 0;
    bool bound = false;
    bool flag_cleared = false;   // the device error word in scratch has been zeroed since bind
    int32_t sticky = GPGA_OK;
    std::string err;
    PhiloxKeys keys;
    SparseW sparse;   // topology SPARSE: caller-owned CSR arrays on the device
    // gpga_run_host only: copy streams and per-chunk events, created on first use
    cudaStream_t up = nullptr, down = nullptr;
    std::vector<cudaEvent_t> events;

    ~gpga_ctx()
    {
        for (cudaEvent_t ev : events) cudaEventDestroy(ev);
        if (up) cudaStreamDestroy(up);
        if (down) cudaStreamDestroy(down);
    }
};

static thread_local std::string g_create_error;

namespace {

constexpr int64_t kMaxTileNodes = 4096;   // shared-memory tile path: n * 16 B <= 64 KB
constexpr int64_t kNarrowGroups = 148 * 32;   // fewer column groups than this: use the tile kernel

int32_t fail(gpga_ctx* c, int32_t code, const std::string& msg)
{
    if (c) c->err = msg; else g_create_error = msg;
    return code;
}

int32_t cuda_fail(gpga_ctx* c, cudaError_t e, const char* where)
{
    c->sticky = GPGA_ERR_CUDA;
    c->err = std::string(where) + ": " + cudaGetErrorString(e);
    return GPGA_ERR_CUDA;
}

bool is_pow2(int64_t v) { return v > 0 && (v & (v - 1)) == 0; }
int log2_floor(int64_t v) { int t = 0; while ((int64_t(1) << (t + 1)) <= v) ++t; return t; }
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
int64_t round_up(int64_t v, int64_t a) { return (v + a - 1) / a * a; }

ScratchLayout scratch_layout(const gpga_ctx* c)
{
    ScratchLayout L;
    int64_t slots = kMaxReduceBlocks;
    if (c->n > slots) slots = c->n;
    // the consensus distance writes one partial per 256 column groups
    if (consensus_blocks((c->d + 3) / 4) > slots) slots = consensus_blocks((c->d + 3) / 4);
    L.slots = slots;
    L.partials_off = 0;
    L.result_off = round_up(slots * 8, 256);
    L.total = L.result_off + 256;
    if (c->objective == GPGA_OBJ_LOGISTIC) {
        L.G_off = L.total;
        L.chunk_off = L.G_off + round_up(c->n * c->d * 4, 256);
        L.total = L.chunk_off + round_up(int64_t(logreg_chunks(c->batch)) * c->n * c->d * 4, 256);
        // rows published by the many-iterations-per-launch kernel (narrow states only)
        if (c->d <= 1024 && c->n <= 88 && (c->topology == GPGA_TOPO_RING || c->topology == GPGA_TOPO_EXP)) {
            const int nbuf = 2 + logreg_run_buffers(c->topology == GPGA_TOPO_EXP, log2_floor(c->n));
            L.ytag_off = L.total;
            L.ytag_bytes = (int64_t)logreg_run_ytag_bytes((int)c->n, (int)c->d, nbuf);
            L.total = L.ytag_off + round_up(L.ytag_bytes, 256);
        }
    }
    return L;
}

// Algorithm 1: global average exactly when mod(k + 1, H) = 0 (H = 0: never).
bool is_global_step(int64_t k, int64_t H) { return H > 0 && ((k + 1) % H) == 0; }

// 128-bit path: every row starts 16-byte aligned and ends on a whole group of four.
bool vec_ok(const gpga_ctx* c) { return (c->d % 4) == 0 && (c->ld % 4) == 0; }

int32_t check_ready(gpga_ctx* c)
{
    if (!c) return fail(nullptr, GPGA_ERR_NOT_READY, "NULL handle");
    if (c->sticky != GPGA_OK) return c->sticky;
    if (!c->bound) return fail(c, GPGA_ERR_NOT_READY, "buffers not bound (call gpga_bind)");
    return GPGA_OK;
}

LogregParams logreg_params(const gpga_ctx* c, int64_t k)
{
    const ScratchLayout& L = c->L;
    LogregParams lp;
    lp.A = c->data;
    lp.y = c->labels;
    lp.x = c->x[c->cur];
    lp.ldx = c->ld;
    lp.G = reinterpret_cast<float*>(c->scratch + L.G_off);
    lp.error_flag = reinterpret_cast<int*>(c->scratch + L.result_off + 8);
    lp.partial = reinterpret_cast<float*>(c->scratch + L.chunk_off);
    lp.n = c->n; lp.d = c->d; lp.m = c->m; lp.batch = c->batch;
    lp.node0 = c->shard * c->n;
    lp.k = (uint32_t)k;
    lp.l2 = c->l2;
    lp.keys = c->keys;
    return lp;
}

// One iteration; `global` chosen by the caller (fixed or adaptive period).
int32_t do_step(gpga_ctx* c, int64_t k, bool global, cudaStream_t s, bool after_own_step = false)
{
    if (k < 0 || k >= (int64_t(1) << 32)) return fail(c, GPGA_ERR_INVALID_ARG, "k must be in [0, 2^32)");
    StepParams p;
    p.x = c->x[c->cur];
    p.out = c->x[c->cur ^ 1];
    p.b = c->data;
    p.n = c->n; p.d = c->d; p.ld = c->ld; p.ldb = c->ld; p.Q = (c->d + 3) / 4;
    p.q_base = (uint32_t)(c->col0 >> 2);
    p.k = (uint32_t)k;
    p.gamma = c->gamma; p.sigma = c->sigma;
    p.hop_log2 = 0; p.len_log2 = 0;
    p.grid_cols = (int)c->grid_cols;
    p.chunks = 0; p.inv_batch = 0.f; p.l2 = 0.f;
    p.keys = c->keys;
    const bool vec = vec_ok(c);
    int mode = (c->sigma != 0.f) ? GRAD_QUAD_NOISE : GRAD_QUAD;
    // Narrow states (few column groups) go through the tile kernel, which spreads threads over
    // (row, group) cells; one thread per group would leave most of the GPU idle.
    const bool narrow = p.Q < kNarrowGroups && tile_supports(c->n);
    const bool tile_topology = c->topology != GPGA_TOPO_RING && c->topology != GPGA_TOPO_EXP;
    cudaError_t e;
    if (c->objective == GPGA_OBJ_LOGISTIC) {
        LogregParams lp = logreg_params(c, k);
        lp.after_own_step = after_own_step && narrow;   // the narrow path's step kernel releases its successor early
        if (!c->flag_cleared) {   // kernels with bounded waits report through this word
            e = cudaMemsetAsync(lp.error_flag, 0, sizeof(int), s);
            if (e != cudaSuccess) return cuda_fail(c, e, "error word clear");
            c->flag_cleared = true;
        }
        if (narrow) {   // the step kernel adds the chunk partials itself: one launch fewer
            e = launch_logreg_partial(lp, s);
            c->launches += 1;
            p.b = lp.partial;
            p.chunks = logreg_chunks(c->batch);
            p.inv_batch = 1.0f / (float)c->batch;
            p.l2 = c->l2;
            mode = GRAD_PARTIALS;
        } else {
            e = launch_logreg_grad(lp, s);
            c->launches += 2;
            p.b = lp.G;
            mode = GRAD_BUFFER;
        }
        if (e != cudaSuccess) return cuda_fail(c, e, "logistic gradient launch");
        p.ldb = c->d;
    }
    if (c->topology == GPGA_TOPO_EXP) {
        const int tau = log2_floor(c->n);
        if (tau > 0) {
            p.hop_log2 = (int)(k % tau);
            p.len_log2 = tau - p.hop_log2;
        }
    }
    if (c->topology == GPGA_TOPO_SPARSE && !c->sparse.row_ptr)
        return fail(c, GPGA_ERR_NOT_READY, "topology SPARSE needs gpga_set_weight_matrix");
    if (narrow || (tile_topology && !global)) {
        e = launch_step_tile_w(p, mode, vec, global ? (int)TILE_MIX_GLOBAL : c->topology, c->sparse, s);
    } else if (global) {
        e = launch_step_global(p, mode, vec, s);
    } else if (c->topology == GPGA_TOPO_RING) {
        e = launch_step_ring(p, mode, vec, s);
    } else {
        e = launch_step_exp(p, mode, vec, s);
    }
    c->launches += 1;
    if (e != cudaSuccess) return cuda_fail(c, e, "step launch");
    c->cur ^= 1;
    c->k = k + 1;
    return GPGA_OK;
}

// K iterations starting at c->k.  Columns evolve independently, so a strip of columns can be taken
// through many iterations on chip (launch_run_tile) with HBM touched once per launch; the time per
// iteration is then set by the noise arithmetic, not by memory.  That path is taken
//  - for a state small enough to sit in L2 (one launch per iteration would be launch-bound), and
//  - for n <= kFusedWideNodes (one cell per thread) and runs of at least kFusedMinSteps iterations at any
//    size: there the arithmetic bound (7.6-7.8e11 updates/s measured at n = 16 and 64, 6.5e11 at
//    n = 256) is above what the row-streaming kernels reach from HBM (at most 5.6e11), also when
//    every iteration is a global average (H = 1: 2.90 against 3.05-3.16 ms at n = 64, d = 25,557,032;
//    8.55 against 10.18 ms at n = 16, d = 335,141,888), and the launch's fixed cost is amortised: it
//    loads and stores the state once and dispatches one small block per strip (10.5 M blocks, about
//    25 ms, at n = 16, d = 335,141,888).  Whole calls measured, single steps against one launch:
//    n = 16, d = 335,141,888: K = 4: 39.0 / 38.8 ms, 8: 79.6 / 64.9, 20: 198.8 / 145.2; n = 64,
//    d = 25,557,032: K = 4: 12.0 / 13.7, 6: 18.3 / 15.9, 20: 62.2 / 44.5; n = 128, d = 2^20: K = 6:
//    1.65 / 2.04, 8: 2.17 / 2.11, 20: 5.48 / 3.94; n = 256, d = 786,432: K = 6: 2.36 / 2.41, 8: 3.17 /
//    3.09, 20: 7.93 / 6.64 -- one launch wins from 8 iterations on at every n.
//    Wider n would go through the several-cells-per-thread kernel, which is far slower.
// A launch is kept to about half a second of work; a longer run is cut into launches of equal length
// (a short last launch would pay the fixed cost for a few iterations).
constexpr int64_t kFusedStateBytes = 64ll << 20;
constexpr int64_t kFusedSteps = 1024;
constexpr int64_t kFusedWideNodes = 256, kFusedMinSteps = 8;
constexpr double kFusedUpdatesPerLaunch = 2.75e11;

// Logistic objective, narrow state: many iterations per launch with x_i resident on chip (a pair of
// blocks per node, see gpga_logrun.cu); bit-identical to single steps.  The rows the blocks publish
// to one another have their own part of the scratch area; the stop word is the first word of its
// reduction area (not in use between iterations).
constexpr int64_t kLogRunMinSteps = 2;
constexpr int64_t kLogRunSteps = 1 << 14;   // per launch: about a tenth of a second

int32_t run_logistic_resident(gpga_ctx* c, int64_t K, cudaStream_t s)
{
    const ScratchLayout& L = c->L;
    const int64_t k_end = c->k + K;
    cudaError_t e;
    if (!c->flag_cleared) {
        e = cudaMemsetAsync(c->scratch + L.result_off + 8, 0, sizeof(int), s);
        if (e != cudaSuccess) return cuda_fail(c, e, "error word clear");
        c->flag_cleared = true;
    }
    while (c->k < k_end) {
        const int64_t steps = (k_end - c->k < kLogRunSteps) ? k_end - c->k : kLogRunSteps;
        LogRunParams p;
        p.A = c->data;
        p.y = c->labels;
        p.x_in = c->x[c->cur];
        p.x_out = c->x[c->cur ^ (int)(steps & 1)];
        p.ldx = c->ld;
        p.ytag = reinterpret_cast<unsigned long long*>(c->scratch + L.ytag_off);
        p.nbuf = 2 + logreg_run_buffers(c->topology == GPGA_TOPO_EXP, log2_floor(c->n));
        p.stop = reinterpret_cast<int*>(c->scratch + L.partials_off);
        p.error_flag = reinterpret_cast<int*>(c->scratch + L.result_off + 8);
        p.n = (int)c->n; p.d = (int)c->d; p.m = (int)c->m; p.batch = (int)c->batch;
        p.k0 = (uint32_t)c->k;
        p.steps = (int)steps;
        p.topology = c->topology;
        p.H = (int)c->H;
        p.log2n = log2_floor(c->n);
        p.gamma = c->gamma; p.l2 = c->l2;
        p.keys = c->keys;
        e = cudaMemsetAsync(p.stop, 0, sizeof(int), s);
        if (e == cudaSuccess) e = cudaMemsetAsync(p.ytag, 0, (size_t)L.ytag_bytes, s);   // no tag of an earlier launch survives
        if (e != cudaSuccess) return cuda_fail(c, e, "published-row buffers clear");
        e = launch_logreg_run(p, s);
        c->launches += 1;
        if (e != cudaSuccess) return cuda_fail(c, e, "resident logistic launch");
        c->cur ^= (int)(steps & 1);
        c->k += steps;
    }
    return GPGA_OK;
}

int32_t run_steps(gpga_ctx* c, int64_t K, cudaStream_t s)
{
    const int64_t k_end = c->k + K;
    if (k_end > (int64_t(1) << 32)) return fail(c, GPGA_ERR_INVALID_ARG, "iteration index must stay below 2^32");
    if (c->topology == GPGA_TOPO_SPARSE && !c->sparse.row_ptr)
        return fail(c, GPGA_ERR_NOT_READY, "topology SPARSE needs gpga_set_weight_matrix");
    const bool fused = c->objective == GPGA_OBJ_QUADRATIC && K >= 2 && run_tile_supports(c->n) &&
                       (12 * c->n * c->ld <= kFusedStateBytes ||
                        (c->n <= kFusedWideNodes && K >= kFusedMinSteps));
    int64_t per_launch = (int64_t)(kFusedUpdatesPerLaunch / ((double)c->n * (double)c->d));
    if (per_launch > kFusedSteps) per_launch = kFusedSteps;
    if (per_launch < 16) per_launch = 16;
    // A global-average iteration costs the one-launch kernel two trips through L2 and a wait for the
    // slowest node, a gossip iteration costs single steps more the more nodes there are.  Measured
    // (us per iteration, single steps against one launch, d = 1024, batch 128): H = 1: 7.8 / 8.7 at
    // n = 8, 8.9 / 9.3 at n = 32, 11.6 / 10.6 at n = 64; H = 2 at n = 64: 10.5 / 9.7; H = 4: 7.6 / 7.9
    // at n = 8, 8.6 / 8.3 at n = 32, 10.3 / 9.1 at n = 64; no global average: 7.6 / 7.5 at n = 8,
    // 10.0 / 7.9 at n = 64.
    const bool run_pays = c->H == 0 || c->H >= 3 || (c->H == 2 && c->n >= 24) || (c->H == 1 && c->n >= 48);
    if (c->objective == GPGA_OBJ_LOGISTIC && K >= kLogRunMinSteps && run_pays) {
        bool ok = false;
        const cudaError_t e = logreg_run_supported((int)c->n, (int)c->d, (int)c->batch, c->topology, c->H, &ok);
        if (e != cudaSuccess) return cuda_fail(c, e, "occupancy query");
        if (ok && c->L.ytag_bytes > 0) return run_logistic_resident(c, K, s);
    }
    if (!fused) {
        for (int64_t k = c->k; k < k_end; ++k) {
            // from the second iteration on, the launch before the gradient kernel is our own step kernel
            const int32_t st = do_step(c, k, is_global_step(k, c->H), s, k > k_end - K);
            if (st) return st;
        }
        return GPGA_OK;
    }
    int64_t launches_left = (K + per_launch - 1) / per_launch;
    while (c->k < k_end) {
        const int64_t steps = (k_end - c->k + launches_left - 1) / launches_left;
        --launches_left;
        StepParams p;
        p.x = c->x[c->cur];
        p.out = c->x[c->cur ^ 1];
        p.b = c->data;
        p.n = c->n; p.d = c->d; p.ld = c->ld; p.ldb = c->ld; p.Q = (c->d + 3) / 4;
        p.q_base = (uint32_t)(c->col0 >> 2);
        p.k = (uint32_t)c->k;
        p.gamma = c->gamma; p.sigma = c->sigma;
        p.hop_log2 = 0; p.len_log2 = 0;
        p.grid_cols = (int)c->grid_cols;
        p.chunks = 0; p.inv_batch = 0.f; p.l2 = 0.f;
        p.keys = c->keys;
        const cudaError_t e = launch_run_tile(p, (c->sigma != 0.f) ? GRAD_QUAD_NOISE : GRAD_QUAD, vec_ok(c),
                                              c->topology, c->H, (int)steps, c->sparse, s);
        c->launches += 1;
        if (e != cudaSuccess) return cuda_fail(c, e, "fused run launch");
        c->cur ^= 1;
        c->k += steps;
    }
    return GPGA_OK;
}

int32_t mean_loss_async(gpga_ctx* c, cudaStream_t s, double** result_dev)
{
    const ScratchLayout& L = c->L;
    double* partials = reinterpret_cast<double*>(c->scratch + L.partials_off);
    double* result = reinterpret_cast<double*>(c->scratch + L.result_off);
    cudaError_t e;
    if (c->objective == GPGA_OBJ_LOGISTIC) {
        if (c->k >= (int64_t(1) << 32)) return fail(c, GPGA_ERR_INVALID_ARG, "k must be in [0, 2^32)");
        e = launch_logreg_loss(logreg_params(c, c->k), partials, result, s);
    } else {
        e = launch_quadratic_loss(c->x[c->cur], c->data, c->n, c->d, c->ld, vec_ok(c), partials, result, s);
    }
    c->launches += 2;
    if (e != cudaSuccess) return cuda_fail(c, e, "loss launch");
    *result_dev = result;
    return GPGA_OK;
}

// Reads the result double and, if it has been armed, the device error word beside it.
int32_t read_double(gpga_ctx* c, const double* dev, cudaStream_t s, double* out_host)
{
    struct { double value; int flag; int pad; } host = {0.0, 0, 0};
    const size_t bytes = c->flag_cleared ? 12 : sizeof(double);
    cudaError_t e = cudaMemcpyAsync(&host, dev, bytes, cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return cuda_fail(c, e, "result copy");
    e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(c, e, "stream synchronize");
    *out_host = host.value;
    if (host.flag != 0) {
        c->sticky = GPGA_ERR_TIMEOUT;
        return fail(c, GPGA_ERR_TIMEOUT, "a bounded wait inside a kernel gave up (asynchronous copy did not complete)");
    }
    return GPGA_OK;
}

}  // namespace

extern "C" {

int32_t gpga_create(int64_t n, int64_t d, int32_t topology, int64_t H, float gamma, uint64_t seed,
                    gpga_t** out)
{
    if (!out) return fail(nullptr, GPGA_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    if (n < 1 || n >= (int64_t(1) << 31)) return fail(nullptr, GPGA_ERR_INVALID_ARG, "n must be in [1, 2^31)");
    if (d < 1 || d >= (int64_t(1) << 34)) return fail(nullptr, GPGA_ERR_INVALID_ARG, "d must be in [1, 2^34)");
    if (H < 0) return fail(nullptr, GPGA_ERR_INVALID_ARG, "H must be >= 0 (0 = never average globally)");
    if (!std::isfinite(gamma) || gamma < 0.f) return fail(nullptr, GPGA_ERR_INVALID_ARG, "gamma must be finite and >= 0");
    if (topology < GPGA_TOPO_RING || topology > GPGA_TOPO_SPARSE)
        return fail(nullptr, GPGA_ERR_INVALID_ARG, "unknown topology");
    if ((topology == GPGA_TOPO_EXP || topology == GPGA_TOPO_STATIC_EXP) && !is_pow2(n))
        return fail(nullptr, GPGA_ERR_UNSUPPORTED, "exponential graphs need n to be a power of two");
    if ((topology == GPGA_TOPO_GRID || topology == GPGA_TOPO_STATIC_EXP || topology == GPGA_TOPO_NONE ||
         topology == GPGA_TOPO_SPARSE) &&
        n > kMaxTileNodes)
        return fail(nullptr, GPGA_ERR_UNSUPPORTED, "this topology supports at most 4096 nodes");
    gpga_ctx* c = new (std::nothrow) gpga_ctx;
    if (!c) return fail(nullptr, GPGA_ERR_INVALID_ARG, "out of host memory");
    c->n = n; c->d = d; c->ld = d; c->topology = topology; c->H = H; c->gamma = gamma; c->seed = seed;
    c->keys = make_philox_keys((uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32));
    if (topology == GPGA_TOPO_GRID) {   // default: the most square torus
        int64_t cols = (int64_t)std::floor(std::sqrt((double)n));
        while (cols > 1 && n % cols != 0) --cols;
        c->grid_cols = n / cols;
    }
    *out = c;
    return GPGA_OK;
}

int32_t gpga_set_objective(gpga_t* c, int32_t objective, float sigma, float l2, int64_t m, int64_t batch)
{
    if (!c) return fail(nullptr, GPGA_ERR_NOT_READY, "NULL handle");
    if (c->bound) return fail(c, GPGA_ERR_INVALID_ARG, "set the objective before gpga_bind");
    if (objective == GPGA_OBJ_QUADRATIC) {
        if (!std::isfinite(sigma) || sigma < 0.f) return fail(c, GPGA_ERR_INVALID_ARG, "sigma must be finite and >= 0");
        c->objective = objective; c->sigma = sigma; c->l2 = 0.f; c->m = 0; c->batch = 0;
        return GPGA_OK;
    }
    if (objective == GPGA_OBJ_LOGISTIC) {
        if (!std::isfinite(l2) || l2 < 0.f) return fail(c, GPGA_ERR_INVALID_ARG, "l2 must be finite and >= 0");
        if (m < 1 || m >= (int64_t(1) << 31)) return fail(c, GPGA_ERR_INVALID_ARG, "m must be in [1, 2^31)");
        if (batch < 1 || batch > (int64_t(1) << 20)) return fail(c, GPGA_ERR_INVALID_ARG, "batch must be in [1, 2^20]");
        if (c->d % 4 != 0) return fail(c, GPGA_ERR_UNSUPPORTED, "logistic objective needs d % 4 == 0");
        if (c->d > 48 * 1024) return fail(c, GPGA_ERR_UNSUPPORTED, "logistic objective needs d <= 49152");
        if (c->n > 65535 || c->n * (c->d / 4) >= (int64_t(1) << 31))
            return fail(c, GPGA_ERR_UNSUPPORTED, "logistic objective: n too large");
        c->objective = objective; c->sigma = 0.f; c->l2 = l2; c->m = m; c->batch = batch;
        return GPGA_OK;
    }
    return fail(c, GPGA_ERR_INVALID_ARG, "unknown objective");
}

int32_t gpga_set_grid_cols(gpga_t* c, int64_t cols)
{
    if (!c) return fail(nullptr, GPGA_ERR_NOT_READY, "NULL handle");
    if (cols < 1 || c->n % cols != 0) return fail(c, GPGA_ERR_INVALID_ARG, "cols must divide n");
    c->grid_cols = cols;
    return GPGA_OK;
}

int32_t gpga_set_weight_matrix(gpga_t* c, const int32_t* row_ptr_dev, const int32_t* col_idx_dev,
                               const float* weights_dev, int64_t nnz)
{
    if (!c) return fail(nullptr, GPGA_ERR_NOT_READY, "NULL handle");
    if (c->topology != GPGA_TOPO_SPARSE) return fail(c, GPGA_ERR_INVALID_ARG, "handle was not created with topology SPARSE");
    if (!row_ptr_dev || !col_idx_dev || !weights_dev || nnz < c->n)
        return fail(c, GPGA_ERR_INVALID_ARG, "need non-NULL CSR arrays with at least one entry per row");
    c->sparse.row_ptr = row_ptr_dev;
    c->sparse.col = col_idx_dev;
    c->sparse.w = weights_dev;
    return GPGA_OK;
}

int32_t gpga_set_row_stride(gpga_t* c, int64_t ld)
{
    if (!c) return fail(nullptr, GPGA_ERR_NOT_READY, "NULL handle");
    if (c->bound) return fail(c, GPGA_ERR_INVALID_ARG, "set the row stride before gpga_bind");
    if (ld < c->d || ld >= (int64_t(1) << 35)) return fail(c, GPGA_ERR_INVALID_ARG, "row stride must be >= d");
    c->ld = ld;
    return GPGA_OK;
}

int32_t gpga_set_column_offset(gpga_t* c, int64_t col0)
{
    if (!c) return fail(nullptr, GPGA_ERR_NOT_READY, "NULL handle");
    if (col0 < 0 || (col0 % 4) != 0 || col0 + c->d >= (int64_t(1) << 34))
        return fail(c, GPGA_ERR_INVALID_ARG, "col0 must be >= 0, a multiple of 4, col0 + d < 2^34");
    c->col0 = col0;
    return GPGA_OK;
}

int64_t gpga_scratch_bytes(const gpga_t* c)
{
    if (!c) return 0;
    return scratch_layout(c).total;
}

int32_t gpga_bind(gpga_t* c, void* x_a, void* x_b, void* data, const void* labels, void* scratch,
                  int64_t scratch_bytes)
{
    if (!c) return fail(nullptr, GPGA_ERR_NOT_READY, "NULL handle");
    if (!x_a || !x_b || !data || !scratch) return fail(c, GPGA_ERR_INVALID_ARG, "NULL buffer");
    if (x_a != x_b) {   // the same buffer twice means "update in place"; anything between is a mistake
        const uintptr_t a = reinterpret_cast<uintptr_t>(x_a), b = reinterpret_cast<uintptr_t>(x_b);
        const uintptr_t bytes = (uintptr_t)c->n * (uintptr_t)c->ld * sizeof(float);
        if ((a < b ? b - a : a - b) < bytes) return fail(c, GPGA_ERR_INVALID_ARG, "x_a and x_b overlap partly");
    }
    if (!aligned16(x_a) || !aligned16(x_b) || !aligned16(data) || !aligned16(scratch) ||
        (labels && !aligned16(labels)))
        return fail(c, GPGA_ERR_INVALID_ARG, "device pointers must be 16-byte aligned");
    if (c->objective == GPGA_OBJ_LOGISTIC && !labels)
        return fail(c, GPGA_ERR_INVALID_ARG, "logistic objective needs labels");
    if (c->objective == GPGA_OBJ_LOGISTIC && (c->ld % 4) != 0)
        return fail(c, GPGA_ERR_INVALID_ARG, "logistic objective needs a row stride that is a multiple of 4");
    if (scratch_bytes < scratch_layout(c).total) return fail(c, GPGA_ERR_INVALID_ARG, "scratch too small");
    c->x[0] = static_cast<float*>(x_a);
    c->x[1] = static_cast<float*>(x_b);
    c->data = static_cast<float*>(data);
    c->labels = static_cast<const float*>(labels);
    c->scratch = static_cast<char*>(scratch);
    c->scratch_bytes = scratch_bytes;
    c->L = scratch_layout(c);
    c->exported_k = -1;
    c->shard_grad_k = -1;
    c->cur = 0;
    c->k = 0;
    c->bound = true;
    c->flag_cleared = false;
    return GPGA_OK;
}

int32_t gpga_init_from_seed(gpga_t* c, int32_t x0_kind, float x0_std, float b_shift, void* stream)
{
    int32_t st = check_ready(c);
    if (st) return st;
    if (c->objective != GPGA_OBJ_QUADRATIC) return fail(c, GPGA_ERR_UNSUPPORTED, "seeded fill is for the quadratic objective");
    if (x0_kind < GPGA_X0_ZERO || x0_kind > GPGA_X0_PER_NODE_NORMAL) return fail(c, GPGA_ERR_INVALID_ARG, "unknown x0 kind");
    if (!std::isfinite(x0_std) || !std::isfinite(b_shift)) return fail(c, GPGA_ERR_INVALID_ARG, "non-finite argument");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool vec = vec_ok(c);
    const uint32_t q_base = (uint32_t)(c->col0 >> 2);
    const uint32_t row0 = (uint32_t)(c->shard * c->n);   // a node shard fills its own rows of the whole problem
    cudaError_t e = launch_init_b(c->data, c->n, c->d, c->ld, q_base, row0, b_shift, vec, c->keys, s);
    if (e != cudaSuccess) return cuda_fail(c, e, "init b launch");
    e = launch_init_x0(c->x[0], c->n, c->d, c->ld, q_base, row0, x0_kind, x0_std, vec, c->keys, s);
    if (e != cudaSuccess) return cuda_fail(c, e, "init x0 launch");
    c->launches += 2;
    c->cur = 0;
    c->k = 0;
    return GPGA_OK;
}

int32_t gpga_step(gpga_t* c, int64_t k, void* stream)
{
    int32_t st = check_ready(c);
    if (st) return st;
    return do_step(c, k, is_global_step(k, c->H), static_cast<cudaStream_t>(stream));
}

int32_t gpga_run(gpga_t* c, int64_t K, void* stream)
{
    int32_t st = check_ready(c);
    if (st) return st;
    if (K < 0) return fail(c, GPGA_ERR_INVALID_ARG, "K must be >= 0");
    return run_steps(c, K, static_cast<cudaStream_t>(stream));
}

namespace {

// Column chunks of the host entry: a sixteenth of one n x d buffer, between 16 MB and 128 MB, in
// whole 128-byte lines per row.  Small enough that the first upload and the last chunk's
// iterations and download, which nothing overlaps, are a small part of the job; large enough that
// a chunk's step kernels fill the GPU.
constexpr int64_t kHostChunkMinBytes = 16ll << 20, kHostChunkMaxBytes = 128ll << 20;

int32_t host_streams(gpga_ctx* c, size_t events)
{
    cudaError_t e;
    if (!c->up && (e = cudaStreamCreateWithFlags(&c->up, cudaStreamNonBlocking)) != cudaSuccess)
        return cuda_fail(c, e, "copy stream");
    if (!c->down && (e = cudaStreamCreateWithFlags(&c->down, cudaStreamNonBlocking)) != cudaSuccess)
        return cuda_fail(c, e, "copy stream");
    while (c->events.size() < events) {
        cudaEvent_t ev;
        if ((e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(c, e, "event");
        c->events.push_back(ev);
    }
    return GPGA_OK;
}

}  // namespace

// Columns evolve independently of one another (W acts on rows; gradient and noise are element-wise
// and keyed by the absolute column), so the job is cut into column chunks that move through three
// streams: upload of chunk c+1, the K iterations of chunk c and the download of chunk c-1 run at
// the same time, and every element goes through exactly the arithmetic of the unchunked run.
int32_t gpga_run_host(gpga_t* c, const float* x0_host, const float* data_host, int64_t K,
                      float* x_out_host, void* stream)
{
    int32_t st = check_ready(c);
    if (st) return st;
    if (c->objective != GPGA_OBJ_QUADRATIC) return fail(c, GPGA_ERR_UNSUPPORTED, "host entry is for the quadratic objective");
    if (!data_host || !x_out_host) return fail(c, GPGA_ERR_INVALID_ARG, "NULL host buffer");
    if (K < 0) return fail(c, GPGA_ERR_INVALID_ARG, "K must be >= 0");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t host_pitch = (size_t)c->d * sizeof(float), pitch = (size_t)c->ld * sizeof(float);
    // whole column groups only (d % 4 == 0), so that every chunk takes the 128-bit path of the full run
    int64_t chunks = 1;
    if (vec_ok(c) && 12 * c->n * c->ld > kFusedStateBytes) {
        const int64_t buffer_bytes = c->n * c->d * 4;
        int64_t chunk_bytes = buffer_bytes / 16;
        if (chunk_bytes < kHostChunkMinBytes) chunk_bytes = kHostChunkMinBytes;
        if (chunk_bytes > kHostChunkMaxBytes) chunk_bytes = kHostChunkMaxBytes;
        chunks = (buffer_bytes + chunk_bytes - 1) / chunk_bytes;
    }
    const int64_t width = chunks > 1 ? round_up((c->d + chunks - 1) / chunks, 32) : c->d;
    chunks = (c->d + width - 1) / width;
    st = host_streams(c, (size_t)(2 * chunks + 2));
    if (st) return st;
    cudaEvent_t* ev = c->events.data();   // [0]: work already on s; [1 + 2c]: chunk c uploaded; [2 + 2c]: chunk c done
    cudaError_t e = cudaEventRecord(ev[0], s);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(c->up, ev[0], 0);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(c->down, ev[0], 0);
    if (e != cudaSuccess) return cuda_fail(c, e, "stream order");
    // the full-width view, put back whatever happens
    float* const x0_full = c->x[0];
    float* const x1_full = c->x[1];
    float* const data_full = c->data;
    const int64_t d_full = c->d, col0_full = c->col0;
    auto restore = [&]() {
        c->x[0] = x0_full; c->x[1] = x1_full; c->data = data_full; c->d = d_full; c->col0 = col0_full;
    };
    const char* where = nullptr;
    for (int64_t ch = 0; ch < chunks && !st && !where; ++ch) {
        const int64_t j0 = ch * width;
        const int64_t w = (d_full - j0 < width) ? d_full - j0 : width;
        const size_t wb = (size_t)w * sizeof(float);
        if (x0_host)
            e = cudaMemcpy2DAsync(x0_full + j0, pitch, x0_host + j0, host_pitch, wb, (size_t)c->n, cudaMemcpyHostToDevice, c->up);
        else   // X^(0) = 0 on every node: nothing to upload (all-zero bits are 0.0f)
            e = cudaMemset2DAsync(x0_full + j0, pitch, 0, wb, (size_t)c->n, c->up);
        if (e == cudaSuccess)
            e = cudaMemcpy2DAsync(data_full + j0, pitch, data_host + j0, host_pitch, wb, (size_t)c->n, cudaMemcpyHostToDevice, c->up);
        if (e == cudaSuccess) e = cudaEventRecord(ev[1 + 2 * ch], c->up);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(s, ev[1 + 2 * ch], 0);
        if (e != cudaSuccess) { where = "upload"; break; }
        c->x[0] = x0_full + j0; c->x[1] = x1_full + j0; c->data = data_full + j0;
        c->d = w; c->col0 = col0_full + j0;
        c->cur = 0;
        c->k = 0;
        st = run_steps(c, K, s);
        restore();
        if (st) break;
        e = cudaEventRecord(ev[2 + 2 * ch], s);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(c->down, ev[2 + 2 * ch], 0);
        if (e == cudaSuccess)
            e = cudaMemcpy2DAsync(x_out_host + j0, host_pitch, c->x[c->cur] + j0, pitch, wb, (size_t)c->n,
                                  cudaMemcpyDeviceToHost, c->down);
        if (e != cudaSuccess) where = "download";
    }
    // nothing of this call stays in flight when it returns, whatever happened
    const cudaError_t e_up = cudaStreamSynchronize(c->up);
    const cudaError_t e_s = cudaStreamSynchronize(s);
    const cudaError_t e_down = cudaStreamSynchronize(c->down);
    if (st) return st;
    if (where) return cuda_fail(c, e, where);
    if (e_up != cudaSuccess) return cuda_fail(c, e_up, "upload stream");
    if (e_s != cudaSuccess) return cuda_fail(c, e_s, "stream synchronize");
    if (e_down != cudaSuccess) return cuda_fail(c, e_down, "download stream");
    return GPGA_OK;
}

int32_t gpga_consensus_distance(gpga_t* c, void* stream, double* out_host)
{
    int32_t st = check_ready(c);
    if (st) return st;
    if (!out_host) return fail(c, GPGA_ERR_INVALID_ARG, "out_host is NULL");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const ScratchLayout& L = c->L;
    double* partials = reinterpret_cast<double*>(c->scratch + L.partials_off);
    double* result = reinterpret_cast<double*>(c->scratch + L.result_off);
    cudaError_t e = launch_consensus(c->x[c->cur], c->n, c->d, c->ld, vec_ok(c), partials, result, s);
    c->launches += 2;
    if (e != cudaSuccess) return cuda_fail(c, e, "consensus launch");
    return read_double(c, result, s, out_host);
}

int32_t gpga_mean_loss(gpga_t* c, void* stream, double* out_host)
{
    int32_t st = check_ready(c);
    if (st) return st;
    if (!out_host) return fail(c, GPGA_ERR_INVALID_ARG, "out_host is NULL");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    double* result = nullptr;
    st = mean_loss_async(c, s, &result);
    if (st) return st;
    return read_double(c, result, s, out_host);
}

int32_t gpga_global_loss(gpga_t* c, void* stream, double* out_host)
{
    int32_t st = check_ready(c);
    if (st) return st;
    if (!out_host) return fail(c, GPGA_ERR_INVALID_ARG, "out_host is NULL");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const ScratchLayout& L = c->L;
    double* partials = reinterpret_cast<double*>(c->scratch + L.partials_off);
    double* result = reinterpret_cast<double*>(c->scratch + L.result_off);
    cudaError_t e;
    if (c->objective == GPGA_OBJ_LOGISTIC) {
        // xbar borrows the gradient buffer, which is dead between iterations
        float* xbar = reinterpret_cast<float*>(c->scratch + L.G_off);
        e = launch_logistic_global_loss(c->data, c->labels, c->x[c->cur], c->ld, c->n, c->d, c->m, c->l2, xbar,
                                        partials, L.slots, result, s);
        c->launches += 3;
    } else {
        e = launch_quadratic_global_loss(c->x[c->cur], c->data, c->n, c->d, c->ld, vec_ok(c), partials, result, s);
        c->launches += 2;
    }
    if (e != cudaSuccess) return cuda_fail(c, e, "global loss launch");
    return read_double(c, result, s, out_host);
}

int32_t gpga_selftest_bounded_wait(gpga_t* c, void* stream)
{
    int32_t st = check_ready(c);
    if (st) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int* flag = reinterpret_cast<int*>(c->scratch + c->L.result_off + 8);
    cudaError_t e = cudaMemsetAsync(flag, 0, sizeof(int), s);
    if (e != cudaSuccess) return cuda_fail(c, e, "error word clear");
    c->flag_cleared = true;
    e = launch_bounded_wait_selftest(flag, s);
    c->launches += 1;
    if (e != cudaSuccess) return cuda_fail(c, e, "self-test launch");
    return GPGA_OK;
}

// Node 0's pair of blocks of the one-launch logistic kernel, alone, with short wait limits: its
// neighbours' rows are never published, so its waits run out; it raises the error and stop words and
// both blocks leave through their common barrier.
int32_t gpga_selftest_run_wait(gpga_t* c, void* stream)
{
    int32_t st = check_ready(c);
    if (st) return st;
    bool ok = false;
    if (c->objective == GPGA_OBJ_LOGISTIC && c->topology == GPGA_TOPO_RING && c->n >= 2 && c->L.ytag_bytes > 0) {
        const cudaError_t q = logreg_run_supported((int)c->n, (int)c->d, (int)c->batch, c->topology, 0, &ok);
        if (q != cudaSuccess) return cuda_fail(c, q, "occupancy query");
    }
    if (!ok) return fail(c, GPGA_ERR_UNSUPPORTED, "needs a logistic ring problem with n >= 2 that the one-launch kernel takes");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const ScratchLayout& L = c->L;
    LogRunParams p;
    p.A = c->data;
    p.y = c->labels;
    p.x_in = c->x[c->cur];
    p.x_out = c->x[c->cur];
    p.ldx = c->ld;
    p.ytag = reinterpret_cast<unsigned long long*>(c->scratch + L.ytag_off);
    p.nbuf = 2 + logreg_run_buffers(0, log2_floor(c->n));
    p.stop = reinterpret_cast<int*>(c->scratch + L.partials_off);
    p.error_flag = reinterpret_cast<int*>(c->scratch + L.result_off + 8);
    p.n = (int)c->n; p.d = (int)c->d; p.m = (int)c->m; p.batch = (int)c->batch;
    p.k0 = 0u;
    p.steps = 2;
    p.topology = c->topology;
    p.H = 0;
    p.log2n = log2_floor(c->n);
    p.gamma = c->gamma; p.l2 = c->l2;
    p.keys = c->keys;
    p.poll_tries = 4096u;      // a few milliseconds
    p.launch_nodes = 1;
    cudaError_t e = cudaMemsetAsync(p.error_flag, 0, sizeof(int), s);
    if (e == cudaSuccess) e = cudaMemsetAsync(p.stop, 0, sizeof(int), s);
    if (e == cudaSuccess) e = cudaMemsetAsync(p.ytag, 0, (size_t)L.ytag_bytes, s);
    if (e != cudaSuccess) return cuda_fail(c, e, "self-test clear");
    c->flag_cleared = true;
    e = launch_logreg_run(p, s);
    c->launches += 1;
    if (e != cudaSuccess) return cuda_fail(c, e, "self-test launch");
    return GPGA_OK;
}

// ---- node sharding ------------------------------------------------------------------------------
namespace {

int64_t shard_row_bytes(int64_t d) { return (d + 3) / 4 * 16; }   // one exchanged row: whole groups of four floats

ShardParams shard_params(const gpga_ctx* c, int64_t k)
{
    ShardParams p;
    p.x = c->x[c->cur];
    p.b = c->data;
    p.ldb = c->ld;
    p.grad = c->sigma != 0.f ? SHARD_GRAD_QUAD_NOISE : SHARD_GRAD_QUAD;
    if (c->objective == GPGA_OBJ_LOGISTIC) {   // the gradient matrix G of this iteration (shard_gradient)
        p.b = reinterpret_cast<const float*>(c->scratch + c->L.G_off);
        p.ldb = c->d;
        p.grad = SHARD_GRAD_BUFFER;
    }
    p.out = c->x[c->cur ^ 1];
    p.n = c->n; p.n_total = c->n * c->shards; p.row0 = c->shard * c->n;
    p.d = c->d; p.ld = c->ld; p.Q = (c->d + 3) / 4;
    p.q_base = (uint32_t)(c->col0 >> 2);
    p.k = (uint32_t)k;
    p.gamma = c->gamma; p.sigma = c->sigma;
    p.keys = c->keys;
    return p;
}

int32_t shard_ready(gpga_ctx* c, int64_t k)
{
    int32_t st = check_ready(c);
    if (st) return st;
    if (c->topology != GPGA_TOPO_RING && c->topology != GPGA_TOPO_EXP)
        return fail(c, GPGA_ERR_UNSUPPORTED, "node sharding: ring or one-peer exponential graph");
    if (k < 0 || k >= (int64_t(1) << 32)) return fail(c, GPGA_ERR_INVALID_ARG, "k must be in [0, 2^32)");
    return GPGA_OK;
}

// Logistic objective: the mini-batch gradient matrix of the local nodes at iteration k (their draws
// keyed by the global node index), once per iteration, into the scratch area.
int32_t shard_gradient(gpga_ctx* c, int64_t k, cudaStream_t s)
{
    if (c->objective != GPGA_OBJ_LOGISTIC || c->shard_grad_k == k) return GPGA_OK;
    LogregParams lp = logreg_params(c, k);
    cudaError_t e = cudaSuccess;
    if (!c->flag_cleared) {
        e = cudaMemsetAsync(lp.error_flag, 0, sizeof(int), s);
        if (e != cudaSuccess) return cuda_fail(c, e, "error word clear");
        c->flag_cleared = true;
    }
    e = launch_logreg_grad(lp, s);
    c->launches += 2;
    if (e != cudaSuccess) return cuda_fail(c, e, "logistic gradient launch");
    c->shard_grad_k = k;
    return GPGA_OK;
}

}  // namespace

int32_t gpga_shard_plan(int32_t topology, int64_t H, int64_t n_total, int64_t shards, int64_t shard, int64_t d,
                        int64_t k, gpga_shard_plan_t* out)
{
    if (!out) return fail(nullptr, GPGA_ERR_INVALID_ARG, "out is NULL");
    *out = gpga_shard_plan_t{};
    if (topology != GPGA_TOPO_RING && topology != GPGA_TOPO_EXP)
        return fail(nullptr, GPGA_ERR_UNSUPPORTED, "node sharding: ring or one-peer exponential graph");
    if (H < 0 || n_total < 1 || n_total >= (int64_t(1) << 31) || shards < 1 || n_total % shards != 0 || shard < 0 ||
        shard >= shards || d < 1 || k < 0)
        return fail(nullptr, GPGA_ERR_INVALID_ARG, "need H >= 0, shards dividing n_total, 0 <= shard < shards, d >= 1, k >= 0");
    if (topology == GPGA_TOPO_EXP && (!is_pow2(n_total) || !is_pow2(shards)))
        return fail(nullptr, GPGA_ERR_UNSUPPORTED, "the one-peer exponential graph needs n and the number of shards to be powers of two");
    const int64_t n_l = n_total / shards, row = shard_row_bytes(d);
    const int32_t up = (int32_t)((shard + shards - 1) % shards), dn = (int32_t)((shard + 1) % shards);
    if (is_global_step(k, H)) {   // every shard's column sums to every shard, in shard order
        out->kind = GPGA_SHARD_GLOBAL;
        out->gather_bytes = (d + 3) / 4 * 4 * (int64_t)sizeof(double);
        return GPGA_OK;
    }
    if (topology == GPGA_TOPO_RING) {
        out->kind = GPGA_SHARD_RING;
        out->messages = 2;
        // message 0: this shard's first row goes up (it is the lower neighbour of the shard above's last
        // node); message 1: its last row goes down.  Received: slot 0 = the row above, slot 1 = the row below.
        out->send_to[0] = up; out->send_offset[0] = 0;   out->dst_offset[0] = row; out->bytes[0] = row;
        out->send_to[1] = dn; out->send_offset[1] = row; out->dst_offset[1] = 0;   out->bytes[1] = row;
        out->recv_from[0] = up; out->recv_offset[0] = 0;
        out->recv_from[1] = dn; out->recv_offset[1] = row;
        return GPGA_OK;
    }
    const int tau = log2_floor(n_total);
    const int64_t hop = tau > 0 ? (int64_t(1) << (k % tau)) : 1;
    const int64_t he = hop < n_l ? hop : n_l;              // rows that cross the shard boundary
    const int64_t ahead = hop < n_l ? 1 : hop / n_l;       // the partner rows live this many shards ahead
    out->kind = GPGA_SHARD_EXP;
    out->hop = hop;
    out->messages = 1;
    out->send_to[0] = (int32_t)(((shard - ahead) % shards + shards) % shards);
    out->recv_from[0] = (int32_t)((shard + ahead) % shards);
    out->bytes[0] = he * row;
    return GPGA_OK;
}

int32_t gpga_set_node_shard(gpga_t* c, int64_t shards, int64_t shard)
{
    if (!c) return fail(nullptr, GPGA_ERR_NOT_READY, "NULL handle");
    if (shards < 1 || shard < 0 || shard >= shards || c->n * shards >= (int64_t(1) << 31))
        return fail(c, GPGA_ERR_INVALID_ARG, "need shards >= 1, 0 <= shard < shards, n * shards < 2^31");
    if (c->topology != GPGA_TOPO_RING && c->topology != GPGA_TOPO_EXP)
        return fail(c, GPGA_ERR_UNSUPPORTED, "node sharding: ring or one-peer exponential graph");
    if (c->topology == GPGA_TOPO_EXP && !is_pow2(shards))
        return fail(c, GPGA_ERR_UNSUPPORTED, "the one-peer exponential graph needs a power-of-two number of shards");
    if (shards > 1 && (c->n % 4) != 0)
        return fail(c, GPGA_ERR_UNSUPPORTED, "with several shards a shard holds a multiple of four nodes (the column mean adds rows in groups of four)");
    c->shards = shards;
    c->shard = shard;
    return GPGA_OK;
}

int64_t gpga_shard_exchange_bytes(const gpga_t* c)
{
    if (!c) return 0;
    const int64_t row = shard_row_bytes(c->d);
    int64_t rows = c->n > 2 ? c->n : 2;
    int64_t bytes = rows * row;
    const int64_t sums = c->shards * ((c->d + 3) / 4 * 4) * (int64_t)sizeof(double);
    return bytes > sums ? bytes : sums;
}

int32_t gpga_shard_export(gpga_t* c, int64_t k, void* send_dev, void* stream)
{
    int32_t st = shard_ready(c, k);
    if (st) return st;
    if (!send_dev || !aligned16(send_dev)) return fail(c, GPGA_ERR_INVALID_ARG, "send buffer must be a 16-byte aligned device pointer");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    st = shard_gradient(c, k, s);
    if (st) return st;
    const ShardParams p = shard_params(c, k);
    const bool vec = vec_ok(c);
    cudaError_t e;
    if (is_global_step(k, c->H)) {
        e = launch_shard_export_sums(p, vec, static_cast<double*>(send_dev), s);
    } else if (c->topology == GPGA_TOPO_RING) {
        // the first and the last local row (one and the same when the shard holds a single node)
        e = launch_shard_export_rows(p, vec, static_cast<float*>(send_dev), 0, (int)(c->n - 1), 2, s);
    } else {
        const int tau = log2_floor(p.n_total);
        const int64_t hop = tau > 0 ? (int64_t(1) << (k % tau)) : 1;
        e = launch_shard_export_rows(p, vec, static_cast<float*>(send_dev), 0, 1, (int)(hop < c->n ? hop : c->n), s);
    }
    c->launches += 1;
    if (e != cudaSuccess) return cuda_fail(c, e, "shard export launch");
    c->exported = send_dev;
    c->exported_k = k;
    return GPGA_OK;
}

int32_t gpga_shard_export_to(gpga_t* c, int64_t k, void* keep_dev, void* const* dest_host, int32_t ndest, void* stream)
{
    int32_t st = shard_ready(c, k);
    if (st) return st;
    const bool global = is_global_step(k, c->H);
    const bool ring = c->topology == GPGA_TOPO_RING;
    const int32_t want = global ? (int32_t)c->shards : (ring ? 2 : 1);
    if (global && c->shards > kShardMaxDirect)
        return fail(c, GPGA_ERR_UNSUPPORTED, "the fused all-gather of the column sums serves at most 32 shards");
    if (!dest_host || ndest != want)
        return fail(c, GPGA_ERR_INVALID_ARG, "destinations: 2 on the ring, 1 on the exponential graph, one per shard for a global average");
    for (int32_t m = 0; m < ndest; ++m)
        if (!dest_host[m] || !aligned16(dest_host[m]))
            return fail(c, GPGA_ERR_INVALID_ARG, "every destination must be a 16-byte aligned device address");
    if (keep_dev && !aligned16(keep_dev)) return fail(c, GPGA_ERR_INVALID_ARG, "keep buffer must be 16-byte aligned");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    st = shard_gradient(c, k, s);
    if (st) return st;
    const ShardParams p = shard_params(c, k);
    const bool vec = vec_ok(c);
    cudaError_t e;
    bool kept = false;
    if (global) {
        ShardSumDests dl{};
        dl.count = ndest;
        for (int32_t m = 0; m < ndest; ++m) dl.dst[m] = static_cast<double*>(dest_host[m]);
        e = launch_shard_export_sums_to(p, vec, dl, s);
    } else if (ring) {
        e = launch_shard_export_rows_to(p, vec, nullptr, static_cast<float*>(dest_host[0]), static_cast<float*>(dest_host[1]),
                                        1, 0, (int)(c->n - 1), 2, s);
    } else {
        const int tau = log2_floor(p.n_total);
        const int64_t hop = tau > 0 ? (int64_t(1) << (k % tau)) : 1;
        const int rows = (int)(hop < c->n ? hop : c->n);
        kept = hop >= c->n && keep_dev != nullptr;   // the step will average these rows with the received ones
        e = launch_shard_export_rows_to(p, vec, kept ? static_cast<float*>(keep_dev) : nullptr,
                                        static_cast<float*>(dest_host[0]), nullptr, rows, 0, 1, rows, s);
    }
    c->launches += 1;
    if (e != cudaSuccess) return cuda_fail(c, e, "shard export launch");
    c->exported = kept ? keep_dev : nullptr;
    c->exported_k = kept ? k : -1;
    return GPGA_OK;
}

namespace {

// Second half of a shard's iteration, whole or in two parts (see ShardPart).
int32_t shard_step_part(gpga_ctx* c, int64_t k, const void* recv_dev, int part, cudaStream_t s)
{
    int32_t st = shard_ready(c, k);
    if (st) return st;
    if (part != SHARD_INTERIOR && (!recv_dev || !aligned16(recv_dev)))
        return fail(c, GPGA_ERR_INVALID_ARG, "receive buffer must be a 16-byte aligned device pointer");
    if (part != SHARD_ALL && c->x[0] == c->x[1])
        return fail(c, GPGA_ERR_UNSUPPORTED, "the two-part step needs the double buffer (x_a != x_b)");
    st = shard_gradient(c, k, s);   // normally formed by the export of this iteration already
    if (st) return st;
    const ShardParams p = shard_params(c, k);
    const bool vec = vec_ok(c);
    const int tau = log2_floor(p.n_total);
    const int64_t hop = tau > 0 ? (int64_t(1) << (k % tau)) : 1;
    const bool global = is_global_step(k, c->H);
    const bool ring = c->topology == GPGA_TOPO_RING;
    // rows that need nothing remote: ring 1 .. n - 2, exponential graph 0 .. n - hop - 1; none for a
    // global average or a hop of at least n nodes
    const bool has_interior = !global && (ring ? c->n >= 3 : hop < c->n);
    cudaError_t e = cudaSuccess;
    if (part == SHARD_INTERIOR) {
        if (has_interior) {
            e = ring ? launch_shard_ring(p, vec, nullptr, SHARD_INTERIOR, s)
                     : launch_shard_exp(p, vec, nullptr, (int)hop, SHARD_INTERIOR, s);
            c->launches += 1;
        }
        if (e != cudaSuccess) return cuda_fail(c, e, "shard step launch");
        return GPGA_OK;   // the buffers flip when the boundary part has run
    }
    const int rest = (part == SHARD_BOUNDARY && has_interior) ? SHARD_BOUNDARY : SHARD_ALL;
    if (global) {
        e = launch_shard_global(p, vec, static_cast<const double*>(recv_dev), (int)c->shards, s);
    } else if (ring) {
        e = launch_shard_ring(p, vec, static_cast<const float*>(recv_dev), rest, s);
    } else if (hop >= c->n && c->exported && c->exported_k == k) {   // every row was exported: take the half-steps from there
        e = launch_shard_exp_exported(p, vec, static_cast<const float*>(c->exported),
                                      static_cast<const float*>(recv_dev), s);
    } else {
        e = launch_shard_exp(p, vec, static_cast<const float*>(recv_dev), (int)(hop < c->n ? hop : c->n), rest, s);
    }
    c->launches += 1;
    c->exported_k = -1;
    c->shard_grad_k = -1;   // the state moves on: the gradient matrix belongs to the old one
    if (e != cudaSuccess) return cuda_fail(c, e, "shard step launch");
    c->cur ^= 1;
    c->k = k + 1;
    return GPGA_OK;
}

}  // namespace

int32_t gpga_shard_step(gpga_t* c, int64_t k, const void* recv_dev, void* stream)
{
    return shard_step_part(c, k, recv_dev, SHARD_ALL, static_cast<cudaStream_t>(stream));
}

int32_t gpga_shard_step_interior(gpga_t* c, int64_t k, void* stream)
{
    return shard_step_part(c, k, nullptr, SHARD_INTERIOR, static_cast<cudaStream_t>(stream));
}

int32_t gpga_shard_step_boundary(gpga_t* c, int64_t k, const void* recv_dev, void* stream)
{
    return shard_step_part(c, k, recv_dev, SHARD_BOUNDARY, static_cast<cudaStream_t>(stream));
}

int32_t gpga_shard_state_sums(gpga_t* c, void* sums_dev, void* stream)
{
    int32_t st = check_ready(c);
    if (st) return st;
    if (!sums_dev || !aligned16(sums_dev)) return fail(c, GPGA_ERR_INVALID_ARG, "sums buffer must be a 16-byte aligned device pointer");
    const cudaError_t e = launch_shard_state_sums(c->x[c->cur], c->n, c->d, c->ld, vec_ok(c), static_cast<double*>(sums_dev),
                                                  static_cast<cudaStream_t>(stream));
    c->launches += 1;
    if (e != cudaSuccess) return cuda_fail(c, e, "state sums launch");
    return GPGA_OK;
}

int32_t gpga_shard_diagnostics(gpga_t* c, const void* gathered_dev, void* stream, double* consensus_part_host,
                               double* loss_part_host)
{
    int32_t st = check_ready(c);
    if (st) return st;
    if (!gathered_dev || !aligned16(gathered_dev)) return fail(c, GPGA_ERR_INVALID_ARG, "gathered sums must be a 16-byte aligned device pointer");
    if (!consensus_part_host && !loss_part_host) return fail(c, GPGA_ERR_INVALID_ARG, "nothing asked for");
    if (c->shards >= (int64_t(1) << 31)) return fail(c, GPGA_ERR_INVALID_ARG, "too many shards");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const ScratchLayout& L = c->L;
    double* partials = reinterpret_cast<double*>(c->scratch + L.partials_off);
    double* result = reinterpret_cast<double*>(c->scratch + L.result_off);
    const double* gathered = static_cast<const double*>(gathered_dev);
    const long long n_total = c->n * c->shards;
    cudaError_t e;
    if (consensus_part_host) {
        e = launch_shard_consensus_part(c->x[c->cur], c->n, c->d, c->ld, vec_ok(c), gathered, (int)c->shards, n_total,
                                        partials, result, s);
        c->launches += 2;
        if (e != cudaSuccess) return cuda_fail(c, e, "shard consensus launch");
        st = read_double(c, result, s, consensus_part_host);
        if (st) return st;
    }
    if (loss_part_host) {
        if (c->objective == GPGA_OBJ_LOGISTIC) {
            float* xbar = reinterpret_cast<float*>(c->scratch + L.G_off);   // dead between iterations
            e = launch_shard_logistic_loss_part(c->data, c->labels, c->n, c->d, c->m, c->l2, gathered, (int)c->shards,
                                                n_total, xbar, partials, L.slots, result, s);
            c->shard_grad_k = -1;   // the gradient matrix of the coming iteration, if any, has been overwritten
            c->launches += 3;
        } else {
            e = launch_shard_quadratic_loss_part(c->data, c->n, c->d, c->ld, vec_ok(c), gathered, (int)c->shards, n_total,
                                                 partials, result, s);
            c->launches += 2;
        }
        if (e != cudaSuccess) return cuda_fail(c, e, "shard loss launch");
        st = read_double(c, result, s, loss_part_host);
        if (st) return st;
    }
    return GPGA_OK;
}

int32_t gpga_aga_update(int64_t k, int64_t warmup_iters, int64_t H_init, double F, double* F_init_inout, int64_t* H_inout)
{
    if (!F_init_inout || !H_inout) return fail(nullptr, GPGA_ERR_INVALID_ARG, "F_init_inout and H_inout must not be NULL");
    if (k < 0 || warmup_iters < 0 || H_init < 1) return fail(nullptr, GPGA_ERR_INVALID_ARG, "need k >= 0, warmup_iters >= 0, H_init >= 1");
    if (k < warmup_iters) {
        *F_init_inout = 0.5 * (*F_init_inout + F);
    } else if (F > 0.0 && std::isfinite(*F_init_inout / F)) {
        const double h = std::ceil(*F_init_inout / F * (double)H_init);
        *H_inout = h < 1.0 ? 1 : (h > 9.0e15 ? (int64_t)9.0e15 : (int64_t)h);
    }
    return GPGA_OK;
}

int32_t gpga_run_adaptive(gpga_t* c, int64_t K, int64_t H_init, int64_t warmup_iters, void* stream,
                          int64_t* periods_host, int64_t max_periods, int64_t* num_periods_host)
{
    int32_t st = check_ready(c);
    if (st) return st;
    if (K < 0 || H_init < 1 || warmup_iters < 0 || max_periods < 0)
        return fail(c, GPGA_ERR_INVALID_ARG, "need K >= 0, H_init >= 1, warmup_iters >= 0");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int64_t H = H_init, C = 0, periods = 0;
    double F_init = 0.0;
    int64_t k = c->k;
    const int64_t k_end = k + K;
    while (k < k_end) {
        // the gossip iterations before the counter reaches the period, as one run (which takes the
        // multi-iteration launches where they pay): the handle's own period is out of play meanwhile
        int64_t gossip = H - 1 - C;
        if (gossip > k_end - k) gossip = k_end - k;
        if (gossip > 0) {
            const int64_t H_handle = c->H;
            c->H = 0;
            st = run_steps(c, gossip, s);
            c->H = H_handle;
            if (st) return st;
            C += gossip;
            k += gossip;
            continue;
        }
        // C + 1 == H: a global average; the loss of this iteration is taken at x^(k) as Algorithm 2 does
        double F = 0.0;
        double* result = nullptr;
        st = mean_loss_async(c, s, &result);
        if (st) return st;
        st = read_double(c, result, s, &F);
        if (st) return st;
        st = do_step(c, k, true, s);
        if (st) return st;
        if (periods_host && periods < max_periods) periods_host[periods] = H;
        ++periods;
        C = 0;
        gpga_aga_update(k, warmup_iters, H_init, F, &F_init, &H);
        ++k;
    }
    if (num_periods_host) *num_periods_host = periods;
    return GPGA_OK;
}

int32_t gpga_get_x(const gpga_t* c, void** x_cur)
{
    if (!c || !x_cur) return GPGA_ERR_NOT_READY;
    if (!c->bound) return GPGA_ERR_NOT_READY;
    *x_cur = c->x[c->cur];
    return GPGA_OK;
}

int32_t gpga_get_k(const gpga_t* c, int64_t* k)
{
    if (!c || !k) return GPGA_ERR_NOT_READY;
    *k = c->k;
    return GPGA_OK;
}

int32_t gpga_set_k(gpga_t* c, int64_t k)
{
    if (!c) return fail(nullptr, GPGA_ERR_NOT_READY, "NULL handle");
    if (k < 0 || k >= (int64_t(1) << 32)) return fail(c, GPGA_ERR_INVALID_ARG, "k must be in [0, 2^32)");
    c->k = k;
    return GPGA_OK;
}

int32_t gpga_set_gamma(gpga_t* c, float gamma)
{
    if (!c) return fail(nullptr, GPGA_ERR_NOT_READY, "NULL handle");
    if (!std::isfinite(gamma) || gamma < 0.f) return fail(c, GPGA_ERR_INVALID_ARG, "gamma must be finite and >= 0");
    c->gamma = gamma;
    return GPGA_OK;
}

int32_t gpga_set_period(gpga_t* c, int64_t H)
{
    if (!c) return fail(nullptr, GPGA_ERR_NOT_READY, "NULL handle");
    if (H < 0) return fail(c, GPGA_ERR_INVALID_ARG, "H must be >= 0");
    c->H = H;
    return GPGA_OK;
}

int64_t gpga_launch_count(const gpga_t* c) { return c ? c->launches : 0; }

const char* gpga_last_error(const gpga_t* c) { return c ? c->err.c_str() : g_create_error.c_str(); }

int32_t gpga_destroy(gpga_t* c)
{
    delete c;
    return GPGA_OK;
}

int32_t gpga_philox_words(const uint32_t* ctr_dev, uint32_t key0, uint32_t key1, int64_t count,
                          uint32_t* out_dev, void* stream)
{
    if (count < 0 || (count > 0 && (!ctr_dev || !out_dev))) return fail(nullptr, GPGA_ERR_INVALID_ARG, "bad argument");
    cudaError_t e = launch_philox_words(ctr_dev, make_philox_keys(key0, key1), count, out_dev,
                                        static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? GPGA_OK : fail(nullptr, GPGA_ERR_CUDA, cudaGetErrorString(e));
}

int32_t gpga_box_muller_words(const uint32_t* a_dev, const uint32_t* b_dev, int64_t count,
                              float* z_dev, void* stream)
{
    if (count < 0 || (count > 0 && (!a_dev || !b_dev || !z_dev))) return fail(nullptr, GPGA_ERR_INVALID_ARG, "bad argument");
    cudaError_t e = launch_box_muller_words(a_dev, b_dev, count, z_dev, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? GPGA_OK : fail(nullptr, GPGA_ERR_CUDA, cudaGetErrorString(e));
}

int32_t gpga_normal_fill(uint64_t seed, uint32_t stream_id, uint32_t k, uint32_t i, uint32_t q0,
                         int64_t count, float* out_dev, void* stream)
{
    if (count < 0 || (count > 0 && !out_dev)) return fail(nullptr, GPGA_ERR_INVALID_ARG, "bad argument");
    cudaError_t e = launch_normal_fill(make_philox_keys((uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32)),
                                       stream_id, k, i, q0, count, out_dev, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? GPGA_OK : fail(nullptr, GPGA_ERR_CUDA, cudaGetErrorString(e));
}

}  // extern "C"
