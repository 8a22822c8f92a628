/*
 * gpga.h -- C ABI of libgpga: one Gossip-PGA iteration over n simulated nodes
 * held as an n x d fp32 matrix X (row i = node i's parameters) on one GPU.
 *
 * Paper: "Accelerating Gossip SGD with Periodic Global Averaging".
 * Each entry point below names the passage of the paper that defines what it
 * computes.  Notation follows the paper: n nodes, d parameters, k the 0-based
 * iteration index of Algorithm 1, gamma the learning rate, H the global
 * averaging period, W the doubly-stochastic weight matrix (Section 3).
 *
 * Conventions
 *  - Every function returns an int32 status (GPGA_OK = 0).  Nothing throws,
 *    aborts or traps.  After a non-zero status gpga_last_error() gives text.
 *  - The handle is owned by the library.  ALL device memory is owned by the
 *    caller and must outlive the handle; the library never allocates or frees
 *    device memory.
 *  - "device pointer" / "host pointer" is stated per argument.  Device
 *    pointers must be 16-byte aligned.  Matrices are row-major fp32 with row
 *    stride ld >= d (default ld = d, see gpga_set_row_stride): element (i, j) of
 *    an n x d matrix is at index i * ld + j (64-bit).
 *  - `stream` arguments are a cudaStream_t passed as void* (NULL = default
 *    stream).  Calls are asynchronous on that stream unless stated otherwise.
 *  - Kernels are launched on the device that is current in the calling thread.
 *    All buffers of a handle, and the streams given with it, must belong to that
 *    device; make it current (cudaSetDevice) before every call on the handle.  A
 *    handle is used from one host thread at a time.
 *  - Random numbers are Philox4x32-10 (Salmon et al., SC'11) keyed by
 *    key = (seed low word, seed high word), counter = (column >> 2, node i,
 *    iteration k, stream id); the four output words give four normals for
 *    columns 4q..4q+3 by Box-Muller with u1 = ((w >> 8) + 1) / 2^24,
 *    u2 = (w' >> 8) / 2^24.  They are generated in registers and never stored.
 */
#ifndef GPGA_H_
#define GPGA_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct gpga_ctx gpga_t;

enum {
    GPGA_OK = 0,
    GPGA_ERR_INVALID_ARG = 1,
    GPGA_ERR_NOT_READY = 2,   /* NULL handle, buffers not bound */
    GPGA_ERR_CUDA = 3,        /* a CUDA call failed; sticky */
    GPGA_ERR_UNSUPPORTED = 4,
    GPGA_ERR_TIMEOUT = 5      /* a bounded wait inside a kernel gave up; reported by the next
                                 synchronising call (consensus distance, mean loss); sticky */
};

/* Gossip topologies (Section 3; Section 5 for the one-peer exponential graph). */
enum {
    GPGA_TOPO_RING = 0,       /* w = 1/3 on i-1, i, i+1 (indices mod n) */
    GPGA_TOPO_EXP = 1,        /* step k: average with (i + 2^(k mod log2 n)) mod n, w = 1/2; n = 2^m */
    GPGA_TOPO_GRID = 2,       /* r x c torus, w = 1/5 on the node and its 4 neighbours */
    GPGA_TOPO_STATIC_EXP = 3, /* w = 1/(log2 n + 1) on i and (i + 2^t) mod n, t < log2 n */
    GPGA_TOPO_NONE = 4,       /* W = I (Local SGD between global averages) */
    GPGA_TOPO_SPARSE = 5      /* any doubly-stochastic W given in CSR form (gpga_set_weight_matrix) */
};

enum { GPGA_OBJ_QUADRATIC = 0, GPGA_OBJ_LOGISTIC = 1 };

/* Initial state kinds for gpga_init_from_seed. */
enum { GPGA_X0_ZERO = 0, GPGA_X0_SHARED_NORMAL = 1, GPGA_X0_PER_NODE_NORMAL = 2 };

/* Random stream ids (fourth counter word). */
enum {
    GPGA_STREAM_NOISE = 0,
    GPGA_STREAM_B = 1,
    GPGA_STREAM_X0 = 2,
    GPGA_STREAM_NODE_SHIFT = 3,
    GPGA_STREAM_BATCH = 4
};

/*
 * Create a handle for problem (1) of the paper, min_x (1/n) sum_i f_i(x), solved
 * by Algorithm 1 with learning rate gamma, weight matrix W given by `topology`
 * and averaging period H.  H = 0 encodes H -> infinity (plain Gossip SGD,
 * Section 3); H = 1 is parallel SGD.  The default objective is the quadratic
 * f_i(x) = 1/2 ||x - b_i||^2 with sigma = 0.
 * Errors: INVALID_ARG for n < 1, d < 1, n >= 2^31, d >= 2^34, H < 0, gamma not
 * finite or negative, unknown topology, NULL out; UNSUPPORTED for EXP or
 * STATIC_EXP with n not a power of two.
 */
int32_t gpga_create(int64_t n, int64_t d, int32_t topology, int64_t H, float gamma, uint64_t seed,
                    gpga_t** out);

/*
 * Choose the stochastic-gradient model (Assumption 2: unbiased, bounded variance).
 *  QUADRATIC: g_ij = (x_ij - b_ij) + sigma * xi_kij, xi standard normal (stream NOISE).
 *             l2, m, batch ignored.
 *  LOGISTIC:  Section 5.1 loss f_i(x) = (1/m) sum_r ln(1 + exp(-y_r a_r^T x)) + (l2/2)||x||^2;
 *             g_i = mini-batch gradient over `batch` rows drawn with replacement:
 *             draw t = word (t & 3) of Philox counter (t >> 2, i, k, BATCH), reduced mod m.
 *             sigma ignored.
 * Errors: INVALID_ARG for negative / non-finite sigma or l2, m < 1, batch < 1, m >= 2^31.
 * Must be called before gpga_bind.
 */
int32_t gpga_set_objective(gpga_t* ctx, int32_t objective, float sigma, float l2, int64_t m,
                           int64_t batch);

/* Grid topology only: number of columns c of the r x c torus (n = r * c).
 * Errors: INVALID_ARG unless c >= 1 and c divides n. */
int32_t gpga_set_grid_cols(gpga_t* ctx, int64_t cols);

/*
 * Topology SPARSE: the weight matrix W of Section 3 (doubly stochastic, w_ij > 0 only between
 * neighbours or for i = j) in CSR form, DEVICE pointers owned by the caller: row_ptr (n + 1
 * int32), col_idx and weights (nnz entries; row i holds x_i^(k+1) = sum_e w[e] y_{col_idx[e]}).
 * The library does not check stochasticity (the arrays live on the device).  n <= 4096.
 * Errors: INVALID_ARG for NULL pointers, nnz < n or a handle with another topology.
 */
int32_t gpga_set_weight_matrix(gpga_t* ctx, const int32_t* row_ptr_dev, const int32_t* col_idx_dev,
                               const float* weights_dev, int64_t nnz);

/*
 * Row stride ld (in floats, ld >= d) of the X buffers and, for the quadratic objective, of b:
 * element (i, j) is at index i * ld + j.  Default ld = d.  Choosing ld a multiple of 32
 * starts every node's parameter vector on a 128-byte line, which is worth several per cent
 * of bandwidth when d itself is not a multiple of 32.  Padding columns d .. ld-1 are never
 * read or written.  The 128-bit access path needs d % 4 == 0 and ld % 4 == 0; other shapes
 * take a scalar path.  The logistic data A and labels stay dense.  Call before gpga_bind.
 * Errors: INVALID_ARG for ld < d or after gpga_bind.
 */
int32_t gpga_set_row_stride(gpga_t* ctx, int64_t ld);

/*
 * Column sharding: this handle holds global columns col0 .. col0 + d - 1 of a wider
 * problem.  Only the random-number counters depend on it; W acts on rows, so column
 * ranges evolve independently (matrix form of the recursion, Appendix A).
 * Errors: INVALID_ARG unless col0 >= 0, col0 % 4 == 0 and col0 + d < 2^34.
 */
int32_t gpga_set_column_offset(gpga_t* ctx, int64_t col0);

/* Bytes of scratch device memory gpga_bind must be given (reduction partials, and
 * for the logistic objective the per-chunk gradient partials). */
int64_t gpga_scratch_bytes(const gpga_t* ctx);

/*
 * Bind caller-owned device buffers.
 *  x_a, x_b : two n*ld fp32 buffers (double buffer for X^(k), X^(k+1)); x_a holds the
 *             current state.  x_b == x_a selects the in-place update: every kernel gives all n
 *             rows of a column group to one thread (or one block's shared-memory tile), which
 *             has read a row before it overwrites it, so X^(k+1) may replace X^(k) and the
 *             footprint drops from three n*ld buffers to two.  Results are bit-identical.
 *  data     : QUADRATIC: b, n*ld fp32.  LOGISTIC: A, n*m*d fp32 (node-major, then sample).
 *  labels   : LOGISTIC: y, n*m fp32 in {-1,+1}; otherwise NULL.
 *  scratch  : at least gpga_scratch_bytes() bytes (scratch_bytes is what was given).
 * Errors: INVALID_ARG for NULL / misaligned pointers, x_a and x_b overlapping without being
 * equal, too little scratch.
 */
int32_t gpga_bind(gpga_t* ctx, void* x_a, void* x_b, void* data, const void* labels,
                  void* scratch, int64_t scratch_bytes);

/*
 * Fill the bound buffers on the device from the seed (quadratic objective only):
 *  b_ij = z_ij + b_shift * s_i,  z from stream B, s_i the first normal of stream
 *  NODE_SHIFT for node i;  X^(0) per x0_kind with standard deviation x0_std
 *  (Algorithm 1 requires equal initial rows: kinds ZERO and SHARED_NORMAL).
 * Also resets the iteration counter to 0 and makes x_a the current buffer.
 * On a node shard (gpga_set_node_shard) local row i is filled as node shard * n + i of the whole
 * problem, so the shards together hold exactly what the unsharded handle would.
 */
int32_t gpga_init_from_seed(gpga_t* ctx, int32_t x0_kind, float x0_std, float b_shift,
                            void* stream);

/*
 * One iteration of Algorithm 1 for iteration index k: gradient, local update
 * x^(k+1/2) = x^(k) - gamma g^(k), then the global average if mod(k+1, H) = 0, else one
 * gossip step with W.  Reads the current buffer, writes the other, flips them, and sets
 * the internal counter to k + 1.  A pure function of (current X, data, seed, k, params).
 * Errors: NOT_READY if unbound; INVALID_ARG for k < 0 or k >= 2^32.
 */
int32_t gpga_step(gpga_t* ctx, int64_t k, void* stream);

/* K iterations k0 .. k0+K-1 starting at the internal counter k0 (Algorithm 1's loop).  Columns of X
 * evolve independently, so under the quadratic objective a strip of columns can be advanced many
 * iterations per launch with its cells held on chip (HBM touched once per launch, the time per
 * iteration set by the noise arithmetic).  gpga_run does so for a state of at most 64 MB (X, X+ and b
 * together), and at any size for n <= 256 and K >= 8, where that is faster than
 * streaming the state from HBM every iteration; otherwise it takes one launch per iteration.  Results are bit-identical
 * to K calls of gpga_step either way.
 * Logistic objective: within one call the launches of consecutive iterations overlap (the rows of A and
 * the labels of iteration k+1 are fetched while iteration k finishes); A and the labels are inputs that
 * no kernel of the library writes, and the caller must not write them while the call's work is in
 * flight on the stream.  For a narrow state (d <= 1024, batch <= 128, ring or one-peer exponential
 * graph, H = 0 or H >= 3, H = 2 with at least 24 nodes, H = 1 with at least 48 (below that single steps
 * are faster), and as many nodes as the device holds pairs of blocks at once: 74 on a B200)
 * and K >= 2 the whole call is one launch per 16384 iterations: a pair of thread blocks per node keeps
 * x_i on chip and exchanges the half-step rows with its neighbours' pairs through the scratch area.
 * That launch expects the device to itself: its blocks wait for one another, every wait is bounded,
 * and if other work keeps some of them from starting for seconds the call's work ends early and the
 * next synchronising call returns GPGA_ERR_TIMEOUT (the state is then unusable).  Only the current
 * buffer holds a defined state after such a call (the other one is not X^(k-1)).
 * Results are bit-identical to K calls of gpga_step either way. */
int32_t gpga_run(gpga_t* ctx, int64_t K, void* stream);

/*
 * Same as gpga_run with HOST buffers (quadratic objective): copies x0_host and data_host
 * (dense n*d fp32 each) into the bound device buffers (row stride ld), resets the counter to 0, runs K
 * iterations, copies X^(K) to x_out_host and returns when all of that is done.  Host buffers
 * should be pinned for full copy speed.  x0_host may be NULL: X^(0) = 0 on every node (Algorithm 1
 * asks for equal initial rows; zero is the common choice), filled on the device, nothing uploaded.
 * Columns of X evolve independently (W mixes rows; gradient and noise are element-wise and keyed by
 * the absolute column), so a state above 64 MB with d % 4 == 0 moves through the call as column
 * chunks (a sixteenth of a buffer, between 16 and 128 MB): the upload of one chunk, the K iterations of the one before
 * and the download of the one before that run at the same time on two internal copy streams and on
 * `stream`.  Every element goes through the same arithmetic as in the unchunked run (results
 * bit-identical to bind + gpga_run), and on return the bound device buffers hold the whole X^(K).
 * Work already queued on `stream` is waited for; the internal streams and events are created on
 * the first call and released by gpga_destroy.
 * Not re-entrant: while the call runs, the handle's view (d, column offset, buffer pointers) is
 * narrowed to the chunk in hand and put back before it returns, so no other call on the same
 * handle (gpga_get_x included) may run beside it from another host thread.
 */
int32_t gpga_run_host(gpga_t* ctx, const float* x0_host, const float* data_host, int64_t K,
                      float* x_out_host, void* stream);

/*
 * Consensus distance sum_i ||x_i - xbar||^2 of the current state (Section 4; Appendix A
 * notation ||X - Xbar||_F^2), accumulated in fp64.  Synchronises the stream; *out_host is
 * a host double.
 */
int32_t gpga_consensus_distance(gpga_t* ctx, void* stream, double* out_host);

/*
 * Mean over nodes of the local loss at each node's own iterate, (1/n) sum_i F_i(x_i)
 * (the quantity Algorithm 2 averages).  QUADRATIC: F_i = 1/2 ||x_i - b_i||^2 (the additive
 * noise model has no per-sample loss).  LOGISTIC: the loss over the mini-batch that node i
 * draws for the current iteration counter k, plus (l2/2)||x_i||^2.  Synchronises the stream.
 */
int32_t gpga_mean_loss(gpga_t* ctx, void* stream, double* out_host);

/*
 * Global loss of problem (1) at the node average: f(xbar) = (1/n) sum_i f_i(xbar),
 * xbar = (1/n) sum_i x_i (the quantity the paper's convergence figures plot).
 * QUADRATIC: f_i = 1/2 ||x - b_i||^2.  LOGISTIC: the Section 5.1 loss over all m local samples
 * of every node plus (l2/2)||x||^2.  fp64 accumulation.  Synchronises the stream.
 */
int32_t gpga_global_loss(gpga_t* ctx, void* stream, double* out_host);

/*
 * Gossip-AGA (Algorithm 2, period rule with the exponent removed as its appendix states):
 * K iterations with an adaptive period.  A counter C counts iterations since the last
 * global average; when C == H the step is a global average, the mean loss F of that
 * iteration's state is taken, and H is updated: F_init <- (F_init + F)/2 while
 * k < warmup_iters, afterwards H <- ceil(F_init / F * H_init).  Synchronises at each
 * global-average iteration; the gossip iterations between two of them are advanced like a gpga_run
 * call of that length (in one launch where that is faster), with the same results as single steps.  periods_host (may be NULL) receives up to max_periods period
 * lengths in order; *num_periods_host their count.
 */
int32_t gpga_run_adaptive(gpga_t* ctx, int64_t K, int64_t H_init, int64_t warmup_iters,
                          void* stream, int64_t* periods_host, int64_t max_periods,
                          int64_t* num_periods_host);

/*
 * Diagnostics of the WHOLE problem on node shards: the consensus distance sum_i ||x_i - xbar||^2
 * (Section 4) and the global loss f(xbar) = (1/n) sum_i f_i(xbar) of problem (1) need the mean over
 * all nodes.  gpga_shard_state_sums writes the fp64 column sums of this shard's current rows
 * (ceil(d/4)*4 doubles, the size and place of a shard's column sums in a global-average exchange:
 * gpga_shard_plan's gather_bytes) to sums_dev; the caller all-gathers them in shard order, like the
 * column sums of a global average; gpga_shard_diagnostics then forms xbar = (sum of the gathered
 * vectors) / (n * shards) and returns this shard's parts,
 *     *consensus_part_host = sum over the local nodes of ||x_i - xbar||^2,
 *     *loss_part_host      = (1 / (n * shards)) sum over the local nodes of f_i(xbar),
 * whose sums over the shards are the whole problem's consensus distance and global loss (f_i as for
 * gpga_global_loss).  Either host pointer may be NULL.  Synchronises the stream.  On a logistic shard
 * the call borrows the gradient buffer: a gradient formed by gpga_shard_export for an iteration not yet
 * stepped is formed again by the step.
 * Errors: NOT_READY before gpga_bind; INVALID_ARG for NULL or misaligned device buffers or when both
 * host pointers are NULL; TIMEOUT / CUDA as for the other synchronising calls.
 */
int32_t gpga_shard_state_sums(gpga_t* ctx, void* sums_dev, void* stream);
int32_t gpga_shard_diagnostics(gpga_t* ctx, const void* gathered_dev, void* stream, double* consensus_part_host,
                               double* loss_part_host);

/*
 * Algorithm 2's period rule by itself (host arithmetic only), for a caller that drives the
 * iterations itself -- the node-sharded deployment, where the mean loss F is the all-reduced mean of
 * the shards' gpga_mean_loss values.  Called at a global-average iteration k with that iteration's
 * F: while k < warmup_iters, F_init <- (F_init + F) / 2 and the period stays; afterwards
 * H <- ceil(F_init / F * H_init), at least 1 (left as it is when F <= 0 or the ratio is not finite).
 * Errors: INVALID_ARG for NULL pointers, k < 0, warmup_iters < 0 or H_init < 1.
 */
int32_t gpga_aga_update(int64_t k, int64_t warmup_iters, int64_t H_init, double F, double* F_init_inout,
                        int64_t* H_inout);

/*
 * Node sharding: the deployment of Section 3, where the n nodes live on several devices, a gossip
 * step exchanges the half-step vectors x^(k+1/2) of neighbouring nodes and the global average is
 * an All-Reduce ("All-Reduce v.s. multiple Gossips"); the appendix's implementation details: on
 * the one-peer exponential graph a worker sends one copy of its parameters and receives one.
 * Here a shard is a handle holding n consecutive nodes (all d columns) of an (n * shards)-node
 * problem; ring or one-peer exponential graph; quadratic objective, or the logistic one (the
 * shard binds its own nodes' A and labels; gpga_shard_export first forms the mini-batch gradient
 * of the local nodes, their draws keyed by the global node index).  One iteration k on a shard:
 *     gpga_shard_export(k, send)   forms what other shards need of this shard's half-step
 *     -- the caller delivers the messages gpga_shard_plan lists (copies, or send/recv and an
 *        all-gather of a communication library) --
 *     gpga_shard_step(k, recv)     local update + mix of the local rows with what was received
 * Results equal the unsharded iteration's (same operations in the same order; the column mean adds
 * the shards' fp64 sums in shard order).  The diagnostics of a shard handle (gpga_consensus_distance,
 * gpga_mean_loss, gpga_global_loss) are over the shard's own nodes; gpga_mean_loss values of equal shards
 * average to the whole problem's.  Send and receive buffers are caller-owned device memory,
 * 16-byte aligned, gpga_shard_exchange_bytes() each; an exchanged row is ceil(d/4)*4 floats.
 * The library reads remote rows only from the receive buffer in this device's own memory.
 */
enum { GPGA_SHARD_RING = 0, GPGA_SHARD_EXP = 1, GPGA_SHARD_GLOBAL = 2 };

typedef struct gpga_shard_plan {
    int32_t kind;            /* what iteration k is: GPGA_SHARD_RING / EXP (a gossip step) or GLOBAL */
    int32_t messages;        /* point-to-point messages this shard sends, and as many it receives:
                                ring 2 (first row up, last row down), exponential graph 1, global 0 */
    int32_t send_to[2];      /* message m goes to this shard ...                                    */
    int32_t recv_from[2];    /* ... and received message m comes from this one                     */
    int64_t send_offset[2];  /* byte offset of message m in this shard's send buffer               */
    int64_t dst_offset[2];   /* byte offset in the DESTINATION's receive buffer where it lands     */
    int64_t recv_offset[2];  /* byte offset in this shard's receive buffer of received message m   */
    int64_t bytes[2];        /* size of sent message m (received message m has the same size)      */
    int64_t gather_bytes;    /* GLOBAL: bytes of one shard's column sums (ceil(d/4)*4 doubles at the
                                start of its send buffer); the receive buffer holds every shard's,
                                shard s at offset s * gather_bytes (an all-gather)                  */
    int64_t hop;             /* exponential graph: 2^(k mod log2 n)                                 */
} gpga_shard_plan_t;

/* Who exchanges what at iteration k (host logic only; Algorithm 1's schedule, the ring's two
 * neighbours, the exponential graph's partner (i + 2^(k mod log2 n)) mod n).  With hop h and n_l
 * nodes per shard the partner rows of a shard are the first min(h, n_l) rows of the shard
 * max(1, h / n_l) places ahead.  With one shard every message goes to the shard itself.
 * Errors: INVALID_ARG / UNSUPPORTED as for gpga_create and gpga_set_node_shard. */
int32_t gpga_shard_plan(int32_t topology, int64_t H, int64_t n_total, int64_t shards, int64_t shard, int64_t d,
                        int64_t k, gpga_shard_plan_t* out);

/* Declares that this handle's n nodes are nodes shard*n .. (shard+1)*n - 1 of an (n*shards)-node
 * problem (the node index keys the noise generator and the mini-batch draws).  Errors: UNSUPPORTED
 * for another topology, for the exponential graph with a number of shards that is not a power of two, and for
 * several shards of a node count that is not a multiple of four. */
int32_t gpga_set_node_shard(gpga_t* ctx, int64_t shards, int64_t shard);

/* Bytes each of the send and the receive buffer must have (the largest message set of any iteration). */
int64_t gpga_shard_exchange_bytes(const gpga_t* ctx);

/* First half of iteration k on this shard: writes the outgoing messages (gpga_shard_plan's
 * send_offset / bytes, or the column sums) to send_dev.  Asynchronous on `stream`.  Leave the send
 * buffer as it is until gpga_shard_step of the same iteration has run: when every local row was
 * exported (a hop of at least n nodes) the step takes the half-step rows from there. */
int32_t gpga_shard_export(gpga_t* ctx, int64_t k, void* send_dev, void* stream);

/* gpga_shard_export with the send fused into the kernel (Section 3: a gossip step sends the node's
 * half-step vector to its neighbours; the appendix's implementation details: one copy sent, one
 * received per one-peer step): the kernel that forms the outgoing rows stores them straight to
 * where their receivers will read them, so no separate copy or send call follows.
 * dest_host is a HOST array of ndest device addresses, 16-byte aligned, on this device or on another
 * one whose memory is mapped for peer access (the kernel only stores there, 16 adjacent bytes per
 * thread; it never loads from a destination):
 *   ring (ndest = 2):       dest[m] = where message m of gpga_shard_plan lands, i.e. the receive
 *                           buffer of shard send_to[m] plus dst_offset[m];
 *   exponential graph (1):  dest[0] = the receive buffer of shard send_to[0];
 *   global average (ndest = shards, at most 32): dest[s] = the receive buffer of shard s plus
 *                           (this shard) * gather_bytes -- the all-gather of the column sums done by
 *                           the producer's stores; dest[this shard] is the shard's own receive buffer.
 * keep_dev (may be NULL) is a send-buffer-sized area of this device: when every local row is exported
 * (a hop of at least n nodes) the rows are stored there too and gpga_shard_step of the same iteration
 * averages them with the received ones instead of forming the half-step again; otherwise unused.
 * Ordering is the caller's: (a) a destination must no longer be needed by its owner's step of an
 * earlier iteration -- alternate between two receive buffers by the parity of k, which suffices when
 * (b) holds; (b) the receiver launches gpga_shard_step(k) only after the exports of all its senders
 * have completed (stream order or an event on one device; a barrier across the processes that own
 * the devices, placed in stream order after the export, otherwise).  No kernel of the library waits
 * for another one.  Asynchronous on `stream`.
 * Errors: as gpga_shard_export; INVALID_ARG for a wrong ndest, a NULL or misaligned destination;
 * UNSUPPORTED for a global average over more than 32 shards. */
int32_t gpga_shard_export_to(gpga_t* ctx, int64_t k, void* keep_dev, void* const* dest_host, int32_t ndest,
                             void* stream);

/* Second half: Algorithm 1's update and mix for the local rows, with recv_dev holding the received
 * messages (recv_offset) or all shards' column sums.  Reads the current buffer, writes the other,
 * flips them and sets the counter to k + 1, like gpga_step.  Asynchronous on `stream`. */
int32_t gpga_shard_step(gpga_t* ctx, int64_t k, const void* recv_dev, void* stream);

/* gpga_shard_step in two parts, so that the exchange overlaps the bulk of the arithmetic (double
 * buffer only: x_a != x_b).  gpga_shard_step_interior writes the rows of X^(k+1) whose neighbours
 * are all local -- ring: rows 1 .. n-2; exponential graph with hop h < n: rows 0 .. n-h-1; none for a
 * global average or a hop of at least n nodes (then it launches nothing) -- and needs nothing
 * received, so it can run while the messages of gpga_shard_export travel on another stream.
 * gpga_shard_step_boundary then writes the remaining rows from recv_dev, flips the buffers and
 * sets the counter to k + 1.  Together they give exactly gpga_shard_step's result.
 * Errors: as gpga_shard_step; UNSUPPORTED for the in-place update. */
int32_t gpga_shard_step_interior(gpga_t* ctx, int64_t k, void* stream);
int32_t gpga_shard_step_boundary(gpga_t* ctx, int64_t k, const void* recv_dev, void* stream);

/*
 * Self-test of the in-kernel wait limit (no counterpart in the paper): launches one block that
 * waits, a bounded number of polls, on a barrier that nothing will ever complete.  The wait must
 * give up and raise the handle's device error word, so that the NEXT synchronising call
 * (gpga_consensus_distance, gpga_mean_loss, gpga_global_loss) returns GPGA_ERR_TIMEOUT, after
 * which the handle stays in that state.  Nothing faults, traps or hangs.  For tests only.
 */
int32_t gpga_selftest_bounded_wait(gpga_t* ctx, void* stream);

/*
 * Self-test of the waits between blocks of the one-launch logistic kernel (no counterpart in the
 * paper).  Needs a bound logistic handle on the ring with n >= 2 that gpga_run would hand to that
 * kernel (d <= 1024, batch <= 128).  Launches node 0's pair of blocks alone, with wait limits of a
 * few thousand polls: the rows of its neighbours are never published, so its waits give up after
 * some milliseconds, raise the handle's error word, and both blocks leave together.  The NEXT
 * synchronising call returns GPGA_ERR_TIMEOUT and the handle stays in that state (its X is not
 * advanced).  Nothing faults, traps or hangs.  For tests only.
 * Errors: UNSUPPORTED for any other handle.
 */
int32_t gpga_selftest_run_wait(gpga_t* ctx, void* stream);

/* Accessors.  gpga_get_x returns the device pointer of the current state buffer. */
int32_t gpga_get_x(const gpga_t* ctx, void** x_cur);
int32_t gpga_get_k(const gpga_t* ctx, int64_t* k);
int32_t gpga_set_k(gpga_t* ctx, int64_t k);
int32_t gpga_set_gamma(gpga_t* ctx, float gamma);   /* e.g. the halving schedule of Section 5.1 */
int32_t gpga_set_period(gpga_t* ctx, int64_t H);
/* Kernels launched by this handle so far. */
int64_t gpga_launch_count(const gpga_t* ctx);

/* Text of the last error of this handle (or of gpga_create when ctx is NULL). */
const char* gpga_last_error(const gpga_t* ctx);

/* Frees the handle only. */
int32_t gpga_destroy(gpga_t* ctx);

/*
 * Generator surface (device pointers), used to check the device generator against its
 * published definition:
 *  gpga_philox_words:  out[4t..4t+3] = Philox4x32-10(counter = ctr[4t..4t+3], key).
 *  gpga_box_muller_words: z[2t], z[2t+1] = Box-Muller of the word pair (a[t], b[t]).
 *  gpga_normal_fill: out[4t..4t+3] = the four normals of counter (q0 + t, i, k, stream_id).
 */
int32_t gpga_philox_words(const uint32_t* ctr_dev, uint32_t key0, uint32_t key1, int64_t count,
                          uint32_t* out_dev, void* stream);
int32_t gpga_box_muller_words(const uint32_t* a_dev, const uint32_t* b_dev, int64_t count,
                              float* z_dev, void* stream);
int32_t gpga_normal_fill(uint64_t seed, uint32_t stream_id, uint32_t k, uint32_t i, uint32_t q0,
                         int64_t count, float* out_dev, void* stream);

/*
 * (No counterpart in the paper: a packaging variant of the logistic mini-batch gradient
 * above, for callers that cannot allocate device memory.)
 *
 * Some code cannot call cudaMalloc at the point where it needs a gradient: a serving or
 * training loop that must not synchronise the device, a plug-in that is handed tensors by
 * a host framework and has no allocator of its own, code running under another runtime's
 * memory pool.  This entry point computes the same mini-batch gradient matrix as the
 * logistic objective of gpga_step,
 *     G[i][:] = -(1/batch) sum_{r in batch(seed,k,i)} y_r a_r / (1 + exp(y_r a_r^T x_i)) + l2 x_i,
 * without a handle and without any caller-provided scratch: its intermediate partial sums
 * go to a fixed array of GPGA_NOALLOC_SCRATCH_BYTES built into the library.  Every GPU
 * that loads the library carries that array until the process exits.
 *
 *  A_dev : n*m*d fp32 (device), y_dev : n*m fp32 in {-1,+1} (device),
 *  x_dev : n rows of d fp32 with row stride ldx (device), G_dev : n*d fp32 OUTPUT (device).
 *  A_dev, x_dev, G_dev 16-byte aligned; d and ldx multiples of 4.
 *  needed_bytes_host (host, may be NULL) receives the scratch bytes this problem needs,
 *  ceil(batch/32) * n * d * 4.
 *
 * Behaviour to rely on:
 *  - It calls no allocating routine.  The first call on a device resolves the array's
 *    address (a symbol lookup); with CUDA's lazy module loading that first lookup or launch
 *    is also when the driver loads the library's device code and sets the array aside, and
 *    it may synchronise the device.  So make one warm-up call per device at start-up,
 *    before any stream capture begins and outside the region that must not stall; from
 *    the second call on, a call leaves the device's free memory unchanged.
 *  - The kernels run on the device that is current when the call is made and use that
 *    device's copy of the array: A_dev, y_dev, x_dev and G_dev must all be memory of that
 *    device (or managed memory) and `stream` a stream of it.  The call checks the pointers
 *    (a query, not an allocation) and returns INVALID_ARG, launching nothing, otherwise.
 *  - Asynchronous on `stream`.  All calls on a device share the one array, which keeps the
 *    previous call's contents; each call writes every element it later reads, so nothing
 *    has to be cleared, but calls that overlap on the GPU race.  Issue them on one stream.
 *  - Errors: INVALID_ARG for NULL or misaligned pointers, out-of-range sizes and buffers
 *    that are not the current device's; UNSUPPORTED when the problem needs more than
 *    GPGA_NOALLOC_SCRATCH_BYTES (the need is reported in *needed_bytes_host; use gpga_step
 *    with a bound scratch buffer instead); CUDA if a CUDA call fails (also: no device).
 *  - There is no handle, hence no error word for a later call to report.  The gradient
 *    kernels for d <= 8192 wait, a bounded number of polls (about a second), for the
 *    asynchronous copies of the batch rows; should such a wait give up, the block writes
 *    NaN over its slice of the partial sums, so the affected rows of G are NaN (never the
 *    previous call's values) while the status already returned stays GPGA_OK.  A caller
 *    that must know checks G for NaN; the handle path reports the same event as
 *    GPGA_ERR_TIMEOUT.
 */
#define GPGA_NOALLOC_SCRATCH_BYTES (4 * 1024 * 1024)
int32_t gpga_logistic_gradient_noalloc(const float* A_dev, const float* y_dev, const float* x_dev,
                                       int64_t ldx, int64_t n, int64_t d, int64_t m, int64_t batch,
                                       float l2, uint64_t seed, int64_t k, float* G_dev, void* stream,
                                       int64_t* needed_bytes_host);

#ifdef __cplusplus
}
#endif
#endif /* GPGA_H_ */
