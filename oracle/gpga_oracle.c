/*
 * gpga_oracle.c -- plain CPU oracle for one Gossip-PGA iteration.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct
 * restatement of the method that the CUDA library is checked against and that
 * the benchmark times as its CPU baseline.  It shares no code, header, table
 * or constant generator with the CUDA path and nothing in the product path may
 * call it.
 *
 * What it follows (paper: "Accelerating Gossip SGD with Periodic Global
 * Averaging"):
 *   - Algorithm 1 (Gossip-PGA), taken step by step in the paper's order:
 *     gradient, local update x^(k+1/2) = x^(k) - gamma g^(k), then either the
 *     global average (when mod(k+1,H) = 0) or one gossip step
 *     x_i^(k+1) = sum_j w_ij x_j^(k+1/2).
 *   - The matrix form of the same recursion in Appendix A
 *     ("Gossip-PGA in matrix notation").
 *   - Section 3: W is doubly stochastic, w_ij > 0 only for neighbours or i = j.
 *   - Section 4 / Appendix A: consensus distance sum_i ||x_i - xbar||^2.
 *   - Section 5.1: the logistic-regression local loss
 *     f_i(x) = (1/M) sum_m ln(1 + exp(-y_im h_im^T x)).
 *   - Algorithm 2 (Gossip-AGA): the period update rule.
 *
 * Precision: every intermediate is fp64.  Functions that take the state as
 * float round once per stored element at the end of an iteration; the *_f64
 * variants never round (used for the invariants).
 *
 * Random numbers: Philox4x32-10 exactly as published (Salmon, Moraes, Dror,
 * Shaw, "Parallel random numbers: as easy as 1, 2, 3", SC'11) followed by the
 * Box-Muller transform.  The keying below is this project's convention; the
 * CUDA library implements the same convention independently.
 *     key     = (seed low 32 bits, seed high 32 bits)
 *     counter = (q, i, k, stream)     q = column >> 2, i = node, k = iteration
 *     one call yields four words w0..w3 and four normals for columns 4q..4q+3:
 *         (z0, z1) = BM(w0, w1), (z2, z3) = BM(w2, w3)
 *         BM(a, b): u1 = ((a >> 8) + 1) / 2^24 in (0,1],  u2 = (b >> 8) / 2^24 in [0,1)
 *                   r = sqrt(-2 ln u1);  returns (r cos(2 pi u2), r sin(2 pi u2))
 *
 * Pins (see tests/test_oracle_pins.py): Philox known answers; ring spectral
 * gap against the beta values the paper prints in Section 5.1; closed forms
 * of the mean recursion; eigenvector contraction; finite-time consensus of
 * the one-peer exponential graph; dense-W agreement; finite differences for
 * the logistic gradient; brute force on tiny inputs.  tests/test_oracle_mutations.py
 * plants single mistakes in a copy of this file and requires a pin to fail for each.
 *
 * Parity unpinned: whole-run trajectories of the benchmark configurations (the paper
 * prints no loss or consensus-distance values for them); they are covered only by
 * the invariants above and by the comparison of the two implementations.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_STREAM_NOISE 0u
#define ORACLE_STREAM_B 1u
#define ORACLE_STREAM_X0 2u
#define ORACLE_STREAM_NODE_SHIFT 3u
#define ORACLE_STREAM_BATCH 4u

/* ------------------------------------------------------------------ */
/* Philox4x32-10 (SC'11, Section 4: the Philox round and key schedule) */
/* ------------------------------------------------------------------ */
void gpga_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Box-Muller on two 32-bit words; uniform mapping as stated in the header. */
void gpga_oracle_box_muller(uint32_t a, uint32_t b, double z[2])
{
    const double two_pi = 6.283185307179586476925286766559;
    double u1 = ((double)(a >> 8) + 1.0) / 16777216.0;
    double u2 = (double)(b >> 8) / 16777216.0;
    double r = sqrt(-2.0 * log(u1));
    z[0] = r * cos(two_pi * u2);
    z[1] = r * sin(two_pi * u2);
}

/* Four standard normals for columns 4q..4q+3 of node i at iteration k. */
void gpga_oracle_normal4(uint64_t seed, uint32_t stream, uint32_t k, uint32_t i, uint32_t q,
                         double z[4])
{
    uint32_t ctr[4] = {q, i, k, stream};
    uint32_t key[2] = {(uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32)};
    uint32_t w[4];
    gpga_oracle_philox4x32_10(ctr, key, w);
    gpga_oracle_box_muller(w[0], w[1], z);
    gpga_oracle_box_muller(w[2], w[3], z + 2);
}

/* One standard normal for global column j. */
static double normal_at(uint64_t seed, uint32_t stream, uint32_t k, uint32_t i, int64_t j)
{
    double z[4];
    gpga_oracle_normal4(seed, stream, k, i, (uint32_t)(j >> 2), z);
    return z[j & 3];
}

/* ------------------------------------------------------------------ */
/* Schedule (Algorithm 1: the test mod(k+1,H) = 0; H = 0 encodes H -> infinity) */
/* ------------------------------------------------------------------ */
int32_t gpga_oracle_is_global(int64_t k, int64_t H)
{
    return (H > 0 && ((k + 1) % H) == 0) ? 1 : 0;
}

/* Hop of the one-peer exponential graph at iteration k: 2^(k mod log2 n). */
int64_t gpga_oracle_exp_hop(int64_t k, int64_t n)
{
    int64_t tau = 0;
    while (((int64_t)1 << (tau + 1)) <= n) ++tau; /* floor(log2 n) */
    if (tau == 0) return 0;
    return (int64_t)1 << (k % tau);
}

/* ------------------------------------------------------------------ */
/* Local step (Algorithm 1: gradient and x^(k+1/2) = x^(k) - gamma g^(k)) */
/* ------------------------------------------------------------------ */

/* Quadratic objective f_i(x) = 1/2 ||x - b_i||^2 with additive noise:
 * g_ij = (x_ij - b_ij) + sigma xi_kij.  X, B, Y are n x dloc row-major and
 * hold global columns col0 .. col0 + dloc - 1.  Y = X - gamma G. */
void gpga_oracle_quadratic_half_step(int64_t n, int64_t dloc, int64_t col0, double gamma,
                                     double sigma, uint64_t seed, int64_t k, const double* X,
                                     const double* B, double* Y)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        for (int64_t j = 0; j < dloc; ++j) {
            double xi = 0.0;
            if (sigma != 0.0)
                xi = normal_at(seed, ORACLE_STREAM_NOISE, (uint32_t)k, (uint32_t)i, col0 + j);
            double x = X[i * dloc + j];
            double g = (x - B[i * dloc + j]) + sigma * xi;
            Y[i * dloc + j] = x - gamma * g;
        }
    }
}

/* Any objective whose gradient matrix G is given: Y = X - gamma G. */
void gpga_oracle_gradient_half_step(int64_t n, int64_t d, double gamma, const double* X,
                                    const double* G, double* Y)
{
    for (int64_t e = 0; e < n * d; ++e) Y[e] = X[e] - gamma * G[e];
}

/* ------------------------------------------------------------------ */
/* Mixing (Algorithm 1: the gossip step and the global average)        */
/* ------------------------------------------------------------------ */

/* Ring, weight 1/3 on i-1, i, i+1 (indices mod n). */
void gpga_oracle_mix_ring(int64_t n, int64_t d, const double* Y, double* Z)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        int64_t up = (i + n - 1) % n, dn = (i + 1) % n;
        for (int64_t j = 0; j < d; ++j)
            Z[i * d + j] = (Y[up * d + j] + Y[i * d + j] + Y[dn * d + j]) / 3.0;
    }
}

/* One-peer exponential graph: node i averages with node (i + hop) mod n, weight 1/2.
 * hop = 0 (n = 1) leaves Y unchanged. */
void gpga_oracle_mix_exp(int64_t n, int64_t d, int64_t hop, const double* Y, double* Z)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        int64_t p = (i + hop) % n;
        for (int64_t j = 0; j < d; ++j) Z[i * d + j] = (Y[i * d + j] + Y[p * d + j]) / 2.0;
    }
}

/* Global average: every row becomes the column mean. */
void gpga_oracle_mix_global(int64_t n, int64_t d, const double* Y, double* Z)
{
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < d; ++j) {
        double s = 0.0;
        for (int64_t i = 0; i < n; ++i) s += Y[i * d + j];
        double m = s / (double)n;
        for (int64_t i = 0; i < n; ++i) Z[i * d + j] = m;
    }
}

/* Two-dimensional torus grid of r x c nodes (n = r c, node i at row i / c, column i % c):
 * weight 1/5 on the node and its four neighbours (indices wrap). */
void gpga_oracle_mix_grid(int64_t r, int64_t c, int64_t d, const double* Y, double* Z)
{
    int64_t n = r * c;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        int64_t a = i / c, b = i % c;
        int64_t up = ((a + r - 1) % r) * c + b, dn = ((a + 1) % r) * c + b;
        int64_t lf = a * c + (b + c - 1) % c, rt = a * c + (b + 1) % c;
        for (int64_t j = 0; j < d; ++j)
            Z[i * d + j] =
                (Y[up * d + j] + Y[lf * d + j] + Y[i * d + j] + Y[rt * d + j] + Y[dn * d + j]) / 5.0;
    }
}

/* Static exponential graph: node i averages itself and nodes (i + 2^t) mod n,
 * t = 0 .. log2(n) - 1, each with weight 1 / (log2(n) + 1). */
void gpga_oracle_mix_static_exp(int64_t n, int64_t d, const double* Y, double* Z)
{
    int64_t tau = 0;
    while (((int64_t)1 << (tau + 1)) <= n) ++tau;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        for (int64_t j = 0; j < d; ++j) {
            double s = Y[i * d + j];
            for (int64_t t = 0; t < tau; ++t) s += Y[((i + ((int64_t)1 << t)) % n) * d + j];
            Z[i * d + j] = s / (double)(tau + 1);
        }
    }
}

/* ------------------------------------------------------------------ */
/* Consensus distance  sum_i ||x_i - xbar||^2  (un-normalised)        */
/* ------------------------------------------------------------------ */
double gpga_oracle_consensus_distance(int64_t n, int64_t d, const double* X)
{
    double total = 0.0;
    for (int64_t j = 0; j < d; ++j) {
        double s = 0.0;
        for (int64_t i = 0; i < n; ++i) s += X[i * d + j];
        double mean = s / (double)n;
        for (int64_t i = 0; i < n; ++i) {
            double dev = X[i * d + j] - mean;
            total += dev * dev;
        }
    }
    return total;
}

/* ------------------------------------------------------------------ */
/* Logistic regression (Section 5.1 loss, plus an l2 term lambda/2 ||x||^2) */
/* ------------------------------------------------------------------ */

/* Mini-batch row indices of node i at iteration k: draw t uses word (t & 3) of
 * Philox counter (t >> 2, i, k, BATCH), reduced mod m (sampling with replacement). */
void gpga_oracle_batch_indices(uint64_t seed, int64_t k, int64_t i, int64_t batch, int64_t m,
                               int32_t* idx)
{
    uint32_t key[2] = {(uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32)};
    for (int64_t t = 0; t < batch; ++t) {
        uint32_t ctr[4] = {(uint32_t)(t >> 2), (uint32_t)i, (uint32_t)k, ORACLE_STREAM_BATCH};
        uint32_t w[4];
        gpga_oracle_philox4x32_10(ctr, key, w);
        idx[t] = (int32_t)(w[t & 3] % (uint32_t)m);
    }
}

/* Full local loss f_i(x) = (1/m) sum_r ln(1 + exp(-y_r a_r^T x)) + (l2/2)||x||^2.
 * A is m x d row-major (node i's samples), y in {-1,+1}. */
double gpga_oracle_logistic_loss(int64_t m, int64_t d, const double* A, const double* y,
                                 const double* x, double l2)
{
    double total = 0.0;
    for (int64_t r = 0; r < m; ++r) {
        double z = 0.0;
        for (int64_t j = 0; j < d; ++j) z += A[r * d + j] * x[j];
        double t = -y[r] * z;
        /* ln(1 + e^t) without overflow */
        total += (t > 0.0) ? t + log1p(exp(-t)) : log1p(exp(t));
    }
    double reg = 0.0;
    for (int64_t j = 0; j < d; ++j) reg += x[j] * x[j];
    return total / (double)m + 0.5 * l2 * reg;
}

/* Gradient over the listed rows (count of them, duplicates allowed):
 * g = -(1/count) sum_r y_r a_r / (1 + exp(y_r a_r^T x)) + l2 x. */
void gpga_oracle_logistic_grad(int64_t d, const double* A, const double* y, const int32_t* rows,
                               int64_t count, const double* x, double l2, double* g)
{
    for (int64_t j = 0; j < d; ++j) g[j] = 0.0;
    for (int64_t t = 0; t < count; ++t) {
        int64_t r = rows[t];
        double z = 0.0;
        for (int64_t j = 0; j < d; ++j) z += A[r * d + j] * x[j];
        double s = -y[r] / (1.0 + exp(y[r] * z));
        for (int64_t j = 0; j < d; ++j) g[j] += s * A[r * d + j];
    }
    for (int64_t j = 0; j < d; ++j) g[j] = g[j] / (double)count + l2 * x[j];
}

/* Stochastic gradient matrix for all nodes: node i uses its own A_i (m x d), y_i (m)
 * and the mini-batch drawn for (seed, k, i).  G is n x d. */
void gpga_oracle_logistic_gradient_matrix(int64_t n, int64_t d, int64_t m, int64_t batch,
                                          uint64_t seed, int64_t k, const double* A,
                                          const double* y, const double* X, double l2, double* G)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        int32_t* idx = (int32_t*)malloc(sizeof(int32_t) * (size_t)batch);
        gpga_oracle_batch_indices(seed, k, i, batch, m, idx);
        gpga_oracle_logistic_grad(d, A + i * m * d, y + i * m, idx, batch, X + i * d, l2,
                                  G + i * d);
        free(idx);
    }
}

/* ------------------------------------------------------------------ */
/* Seeded synthetic data for the quadratic objective                   */
/* ------------------------------------------------------------------ */

/* b_ij = z_ij + shift * s_i,  z from stream B, s_i = first normal of stream NODE_SHIFT. */
void gpga_oracle_init_b(int64_t n, int64_t dloc, int64_t col0, uint64_t seed, double shift,
                        double* B)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        double s = 0.0;
        if (shift != 0.0) s = normal_at(seed, ORACLE_STREAM_NODE_SHIFT, 0u, (uint32_t)i, 0);
        for (int64_t j = 0; j < dloc; ++j)
            B[i * dloc + j] = normal_at(seed, ORACLE_STREAM_B, 0u, (uint32_t)i, col0 + j) + shift * s;
    }
}

/* kind 0: zeros.  kind 1: one N(0, std^2) row (node index 0 in the counter) shared
 * by all nodes.  kind 2: independent N(0, std^2) rows. */
void gpga_oracle_init_x0(int64_t n, int64_t dloc, int64_t col0, uint64_t seed, int32_t kind,
                         double std, double* X)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        for (int64_t j = 0; j < dloc; ++j) {
            double v = 0.0;
            if (kind == 1) v = std * normal_at(seed, ORACLE_STREAM_X0, 0u, 0u, col0 + j);
            if (kind == 2) v = std * normal_at(seed, ORACLE_STREAM_X0, 0u, (uint32_t)i, col0 + j);
            X[i * dloc + j] = v;
        }
    }
}

/* ------------------------------------------------------------------ */
/* Gossip-AGA period update (Algorithm 2, with the exponent removed as  */
/* Appendix F states): called at a global-average iteration k with the  */
/* mean loss F of that iteration.                                       */
/* ------------------------------------------------------------------ */
void gpga_oracle_aga_update(int64_t k, int64_t warmup_iters, int64_t H_init, double F,
                            double* F_init, int64_t* H)
{
    if (k < warmup_iters) {
        *F_init = 0.5 * (*F_init + F);
    } else {
        *H = (int64_t)ceil((*F_init / F) * (double)H_init);
    }
}

/* Box-Muller over arrays of word pairs: z[2t], z[2t+1] from (a[t], b[t]). */
void gpga_oracle_box_muller_many(const uint32_t* a, const uint32_t* b, int64_t count, double* z)
{
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < count; ++t) gpga_oracle_box_muller(a[t], b[t], z + 2 * t);
}

/* Mean over nodes of the local quadratic loss at each node's own iterate:
 * (1/n) sum_i 1/2 ||x_i - b_i||^2  (the loss Algorithm 2 averages, for f_i of the
 * quadratic objective). */
double gpga_oracle_quadratic_mean_loss(int64_t n, int64_t d, const double* X, const double* B)
{
    double total = 0.0;
    for (int64_t e = 0; e < n * d; ++e) {
        double r = X[e] - B[e];
        total += r * r;
    }
    return 0.5 * total / (double)n;
}
