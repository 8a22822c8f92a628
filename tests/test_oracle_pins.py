"""Pins for the CPU oracle: each test ties it to something other than itself --
values the paper prints, closed forms, invariants, library routines, brute force.
All CPU-only."""
from pathlib import Path

import numpy as np
import pytest

from oracle import gpga_oracle as o

GOLDEN = Path(__file__).resolve().parent / "golden"


def _rows(name):
    out = []
    for line in (GOLDEN / name).read_text().splitlines():
        line = line.strip()
        if line and not line.startswith("#"):
            out.append(line.split())
    return out


# ---------------------------------------------------------------- generator
def test_philox_known_answers():
    for row in _rows("philox4x32_10_kat.txt"):
        v = [int(t, 16) for t in row]
        got = o.philox4x32_10(v[0:4], v[4:6])
        assert [int(x) for x in got] == v[6:10]


def test_box_muller_special_values():
    top = (2**24 - 1) << 8
    # u1 = 1 -> radius 0
    assert np.allclose(o.box_muller(top, 12345 << 8), [0.0, 0.0], atol=0)
    # u1 = 2^-24 -> radius sqrt(48 ln 2); u2 = 0 -> angle 0
    r = np.sqrt(48.0 * np.log(2.0))
    z = o.box_muller(0, 0)
    assert abs(z[0] - r) < 1e-14 and abs(z[1]) < 1e-14
    # u2 = 1/4 -> (0, r); u2 = 1/2 -> (-r, 0)
    z = o.box_muller(0, (2**22) << 8)
    assert abs(z[0]) < 1e-14 and abs(z[1] - r) < 1e-14
    z = o.box_muller(0, (2**23) << 8)
    assert abs(z[0] + r) < 1e-14 and abs(z[1]) < 1e-14
    # the low 8 bits of each word are unused
    assert np.array_equal(o.box_muller(0x12345600, 0x9abcde00), o.box_muller(0x123456ff, 0x9abcdeff))


def test_normals_are_standard_normal():
    from scipy import stats
    z = np.concatenate([o.normal4(7, 0, k, i, q) for k in range(4) for i in range(5)
                        for q in range(2500)])
    assert z.size == 200000
    assert abs(z.mean()) < 5 / np.sqrt(z.size)
    assert abs(z.var() - 1.0) < 0.02
    assert abs(stats.kurtosis(z, fisher=False) - 3.0) < 0.1
    assert stats.kstest(z, "norm").pvalue > 1e-3
    # the four outputs of one call, and neighbouring counters, are uncorrelated
    z4 = z.reshape(-1, 4)
    c = np.corrcoef(z4.T)
    assert np.abs(c - np.eye(4)).max() < 0.02
    assert abs(np.corrcoef(z4[:-1, 0], z4[1:, 0])[0, 1]) < 0.02


def test_noise_keying_distinct_streams():
    a = o.normal4(1, 0, 3, 2, 10)
    assert not np.array_equal(a, o.normal4(2, 0, 3, 2, 10))      # seed
    assert not np.array_equal(a, o.normal4(1, 1, 3, 2, 10))      # stream
    assert not np.array_equal(a, o.normal4(1, 0, 4, 2, 10))      # iteration
    assert not np.array_equal(a, o.normal4(1, 0, 3, 3, 10))      # node
    assert not np.array_equal(a, o.normal4(1, 0, 3, 2, 11))      # column group
    assert np.array_equal(a, o.normal4(1, 0, 3, 2, 10))
    # seed high word is part of the key
    assert not np.array_equal(o.normal4(1, 0, 0, 0, 0), o.normal4(1 + (1 << 32), 0, 0, 0, 0))


# ---------------------------------------------------------------- schedule
def test_schedule_predicate():
    # Algorithm 1: global average exactly when mod(k+1, H) = 0, k counted from 0
    assert [k for k in range(12) if o.is_global(k, 4)] == [3, 7, 11]
    assert all(o.is_global(k, 1) for k in range(8))
    assert not any(o.is_global(k, 0) for k in range(100))           # H -> infinity
    assert [o.exp_hop(k, 32) for k in range(7)] == [1, 2, 4, 8, 16, 1, 2]
    assert [o.exp_hop(k, 16) for k in range(5)] == [1, 2, 4, 8, 1]
    assert o.exp_hop(3, 1) == 0


def test_consensual_exactly_when_iteration_index_is_multiple_of_H():
    # Section 3.1: x_i^(l) = xbar^(l) whenever mod(l, H) = 0
    rng = np.random.default_rng(0)
    n, d, H = 6, 8, 3
    B = rng.standard_normal((n, d))
    p = o.Problem(o.TOPO_RING, H, 0.1, 5, sigma=0.3, data=B)
    X = np.zeros((n, d), dtype=np.float32)
    for k in range(9):
        X = o.step(p, X, k)
        identical = bool(np.all(X == X[0]))
        assert identical == ((k + 1) % H == 0)
        if identical:
            assert o.consensus_distance(X) == 0.0


# ---------------------------------------------------------------- weight matrices
def test_ring_beta_matches_values_printed_in_paper():
    for n_s, beta_s in _rows("ring_beta_section_5_1.txt"):
        n, beta = int(n_s), float(beta_s)
        W = o.dense_w_ring(n)
        got = np.linalg.norm(W - np.full((n, n), 1.0 / n), 2)
        assert abs(got - beta) < 1e-3
        assert abs(got - (1 + 2 * np.cos(2 * np.pi / n)) / 3) < 1e-12


@pytest.mark.parametrize("n", [1, 2, 3, 4, 5, 8, 16])
def test_dense_w_doubly_stochastic(n):
    mats = [o.dense_w_ring(n), o.dense_w_global(n)]
    if n & (n - 1) == 0:
        mats += [o.dense_w_exp(n, o.exp_hop(k, n)) for k in range(5)]
        if n > 1:
            mats.append(o.dense_w_static_exp(n))
    if n % 2 == 0 and n >= 4:
        mats.append(o.dense_w_grid(n // 2, 2))
    for W in mats:
        assert (W >= 0).all()
        assert np.allclose(W.sum(0), 1, atol=1e-15) and np.allclose(W.sum(1), 1, atol=1e-15)
    assert np.count_nonzero(o.dense_w_ring(8)[0]) == 3          # |N_i| = 3 (Section 3.3)
    assert np.count_nonzero(o.dense_w_grid(4, 4)[5]) == 5       # |N_i| = 5 for the grid


@pytest.mark.parametrize("topo,n,gc", [(o.TOPO_RING, 1, 0), (o.TOPO_RING, 2, 0), (o.TOPO_RING, 3, 0),
                                       (o.TOPO_RING, 7, 0), (o.TOPO_EXP, 1, 0), (o.TOPO_EXP, 2, 0),
                                       (o.TOPO_EXP, 8, 0), (o.TOPO_EXP, 16, 0), (o.TOPO_GRID, 12, 4),
                                       (o.TOPO_GRID, 4, 2), (o.TOPO_STATIC_EXP, 8, 0),
                                       (o.TOPO_NONE, 5, 0)])
def test_sparse_path_equals_dense_w(topo, n, gc):
    rng = np.random.default_rng(n)
    d = 9
    B = rng.standard_normal((n, d))
    X = rng.standard_normal((n, d))
    p = o.Problem(topo, 3, 0.2, 11, sigma=0.5, data=B, grid_cols=gc)
    for k in range(7):
        a = o.step_f64(p, X, k, dense=False)
        b = o.step_f64(p, X, k, dense=True)
        assert np.allclose(a, b, rtol=1e-12, atol=1e-13)
        X = a


def test_mix_brute_force_tiny():
    rng = np.random.default_rng(3)
    for n in (2, 4, 8):
        Y = rng.standard_normal((n, 3))
        for k in range(4):
            h = o.exp_hop(k, n)
            want = np.array([[0.5 * (Y[i, j] + Y[(i + h) % n, j]) for j in range(3)]
                             for i in range(n)])
            assert np.array_equal(o.mix(Y, o.TOPO_EXP, k, False), want)
        want = np.array([[(Y[(i - 1) % n, j] + Y[i, j] + Y[(i + 1) % n, j]) / 3 for j in range(3)]
                         for i in range(n)])
        assert np.array_equal(o.mix(Y, o.TOPO_RING, 0, False), want)


# ---------------------------------------------------------------- mixing invariants
def test_ring_eigenvector_contracts_by_lambda2():
    # no gradient, no noise: on the second eigenvector the ring mix multiplies by
    # lambda_2 = (1 + 2 cos(2 pi / n)) / 3 exactly (Appendix A, ||(W - J)^k|| <= beta^k)
    n, d = 16, 5
    lam = (1 + 2 * np.cos(2 * np.pi / n)) / 3
    c = np.arange(1, d + 1, dtype=np.float64)
    X0 = np.cos(2 * np.pi * np.arange(n) / n)[:, None] * c[None, :]
    p = o.Problem(o.TOPO_RING, 0, 0.0, 1, sigma=0.0, data=np.zeros((n, d)))
    X = X0.copy()
    xi0 = o.consensus_distance(X0)
    for k in range(1, 9):
        X = o.step_f64(p, X, k - 1)
        assert np.allclose(X, lam**k * X0, rtol=1e-12, atol=1e-14)
        assert abs(np.sqrt(o.consensus_distance(X) / xi0) - lam**k) < 1e-12


@pytest.mark.parametrize("n", [2, 4, 8, 32])
def test_one_peer_exponential_reaches_exact_average_in_log2n_steps(n):
    # Section 3: the exact global average is reached after log2(n) one-peer gossips
    tau = int(np.log2(n))
    P = np.eye(n)
    for t in range(tau):
        P = o.dense_w_exp(n, 1 << t) @ P
    assert np.array_equal(P, np.full((n, n), 1.0 / n))      # powers of 1/2: exact in fp64
    rng = np.random.default_rng(n)
    X0 = rng.standard_normal((n, 6))
    p = o.Problem(o.TOPO_EXP, 0, 0.0, 1, sigma=0.0, data=np.zeros((n, 6)))
    X = o.run_f64(p, X0, 0, tau)
    assert o.consensus_distance(X) <= 1e-28 * o.consensus_distance(X0)
    assert np.allclose(X, X0.mean(0, keepdims=True), atol=1e-15)
    # one step fewer is not yet consensual
    assert o.consensus_distance(o.run_f64(p, X0, 0, tau - 1)) > 1e-3 or tau == 1
    # float32-stored state: consensus only up to rounding
    X32 = o.run(p, X0.astype(np.float32), 0, tau)
    assert o.consensus_distance(X32) <= 1e-12 * o.consensus_distance(X0)


def test_global_step_rows_identical_and_equal_library_mean():
    rng = np.random.default_rng(5)
    n, d = 7, 33
    X = rng.standard_normal((n, d)).astype(np.float32)
    B = rng.standard_normal((n, d))
    p = o.Problem(o.TOPO_RING, 1, 0.3, 2, sigma=0.0, data=B)
    Z = o.step(p, X, 0)
    assert np.all(Z == Z[0])
    Y = X.astype(np.float64) - 0.3 * (X.astype(np.float64) - B)
    assert np.allclose(Z[0], Y.mean(0), rtol=1e-7, atol=1e-7)
    Zf = o.step_f64(p, X.astype(np.float64), 0)
    assert np.allclose(Zf[3], Y.mean(0), rtol=1e-14, atol=1e-15)


@pytest.mark.parametrize("topo,gc", [(o.TOPO_RING, 0), (o.TOPO_EXP, 0), (o.TOPO_GRID, 4),
                                     (o.TOPO_STATIC_EXP, 0), (o.TOPO_NONE, 0)])
def test_mixing_preserves_node_mean(topo, gc):
    rng = np.random.default_rng(9)
    Y = rng.standard_normal((16, 21))
    for k in range(5):
        for g in (False, True):
            Z = o.mix(Y, topo, k, g, gc)
            assert np.allclose(Z.mean(0), Y.mean(0), rtol=1e-13, atol=1e-14)


# ---------------------------------------------------------------- whole recursion
def test_mean_recursion_closed_form_without_noise():
    # Averaging Algorithm 1 over nodes: xbar^(k+1) = xbar^(k) - (gamma/n) sum_i grad f_i;
    # for the quadratic, xbar^K = bbar + (1-gamma)^K (xbar^0 - bbar), for every W and H
    rng = np.random.default_rng(2)
    n, d, K, gamma = 8, 12, 15, 0.1
    B = rng.standard_normal((n, d))
    X0 = np.repeat(rng.standard_normal((1, d)), n, axis=0)
    want = B.mean(0) + (1 - gamma) ** K * (X0.mean(0) - B.mean(0))
    for topo, gc in ((o.TOPO_RING, 0), (o.TOPO_EXP, 0), (o.TOPO_GRID, 4), (o.TOPO_STATIC_EXP, 0),
                     (o.TOPO_NONE, 0)):
        for H in (0, 1, 4):
            p = o.Problem(topo, H, gamma, 1, sigma=0.0, data=B, grid_cols=gc)
            X = o.run_f64(p, X0, 0, K)
            assert np.allclose(X.mean(0), want, rtol=1e-12, atol=1e-13)


def test_mean_trajectory_independent_of_topology_and_period_with_noise():
    rng = np.random.default_rng(4)
    n, d, K, gamma, sigma, seed = 8, 8, 10, 0.1, 0.7, 99
    B = rng.standard_normal((n, d))
    X0 = np.zeros((n, d))
    # closed form driven by the generator's own numbers
    xbar = X0.mean(0)
    for k in range(K):
        xi = np.array([[o.normal4(seed, 0, k, i, j >> 2)[j & 3] for j in range(d)]
                       for i in range(n)])
        xbar = (1 - gamma) * xbar + gamma * B.mean(0) - gamma * sigma * xi.mean(0)
    for topo in (o.TOPO_RING, o.TOPO_EXP):
        for H in (0, 1, 3):
            p = o.Problem(topo, H, gamma, seed, sigma=sigma, data=B)
            X = o.run_f64(p, X0, 0, K)
            assert np.allclose(X.mean(0), xbar, rtol=1e-12, atol=1e-13)
            if H == 1:      # W = (1/n) 1 1^T: parallel SGD, every row is the mean
                assert np.allclose(X, xbar[None, :], rtol=1e-12, atol=1e-13)


def test_special_cases_of_section_3():
    rng = np.random.default_rng(6)
    n, d, K, gamma = 8, 6, 9, 0.2
    B = rng.standard_normal((n, d))
    X0 = np.zeros((n, d), dtype=np.float32)
    # H -> infinity is plain gossip SGD: same as any H larger than the run
    a = o.run(o.Problem(o.TOPO_RING, 0, gamma, 3, sigma=0.1, data=B), X0, 0, K)
    b = o.run(o.Problem(o.TOPO_RING, K + 5, gamma, 3, sigma=0.1, data=B), X0, 0, K)
    assert np.array_equal(a, b)
    # W = I is local SGD: each node runs its own recursion x_i^K = b_i + (1-gamma)^K (x0 - b_i)
    X = o.run_f64(o.Problem(o.TOPO_NONE, 0, gamma, 3, sigma=0.0, data=B), X0, 0, K)
    assert np.allclose(X, B * (1 - (1 - gamma) ** K), rtol=1e-12)


def test_column_slices_evolve_independently():
    # quadratic path: a run on columns [c0, c1) with col0 = c0 equals the slice of a full run
    rng = np.random.default_rng(8)
    n, d, K = 4, 40, 6
    B = rng.standard_normal((n, d)).astype(np.float32)
    X0 = rng.standard_normal((n, d)).astype(np.float32)
    full = o.run(o.Problem(o.TOPO_EXP, 3, 0.1, 17, sigma=0.4, data=B), X0, 0, K)
    for c0, c1 in ((0, 8), (12, 28), (36, 40)):
        part = o.run(o.Problem(o.TOPO_EXP, 3, 0.1, 17, sigma=0.4, data=B[:, c0:c1], col0=c0),
                     X0[:, c0:c1], 0, K)
        assert np.array_equal(part, full[:, c0:c1])


def test_noise_enters_with_the_stated_sign_and_scale():
    # X = B: g = sigma xi, so Y - X = -gamma sigma xi with xi from the NOISE stream
    n, d, gamma, sigma, seed, k = 3, 8, 0.25, 0.5, 21, 7
    X = np.arange(n * d, dtype=np.float64).reshape(n, d)
    Y = o.quadratic_half_step(X, X, gamma, sigma, seed, k)
    xi = np.array([[o.normal4(seed, 0, k, i, j >> 2)[j & 3] for j in range(d)] for i in range(n)])
    assert np.allclose(Y - X, -gamma * sigma * xi, rtol=1e-12, atol=1e-14)
    # and the gradient pulls towards b: sigma = 0, X = 0 gives Y = gamma b
    Bm = np.ones((n, d))
    assert np.allclose(o.quadratic_half_step(np.zeros((n, d)), Bm, gamma, 0.0, seed, k), gamma * Bm)


# ---------------------------------------------------------------- consensus distance
def test_consensus_distance_against_library_and_brute_force():
    rng = np.random.default_rng(10)
    X = rng.standard_normal((5, 7))
    want = np.linalg.norm(X - X.mean(0, keepdims=True), "fro") ** 2
    assert abs(o.consensus_distance(X) - want) < 1e-12
    brute = sum((X[i, j] - sum(X[r, j] for r in range(5)) / 5) ** 2 for i in range(5)
                for j in range(7))
    assert abs(o.consensus_distance(X) - brute) < 1e-12
    assert o.consensus_distance(np.repeat(X[:1], 4, axis=0)) == 0.0     # mean of 2^m copies is exact
    assert o.consensus_distance(np.repeat(X[:1], 5, axis=0)) < 1e-30


def test_consensus_contracts_by_lambda2_squared_on_ring():
    n, d = 20, 3
    lam = (1 + 2 * np.cos(2 * np.pi / n)) / 3
    X = np.sin(2 * np.pi * np.arange(n) / n)[:, None] * np.ones((1, d))
    p = o.Problem(o.TOPO_RING, 0, 0.0, 1, data=np.zeros((n, d)))
    x1 = o.step_f64(p, X, 0)
    assert abs(o.consensus_distance(x1) / o.consensus_distance(X) - lam**2) < 1e-12


# ---------------------------------------------------------------- logistic regression
def _tiny_logistic(seed=0, m=12, d=5):
    rng = np.random.default_rng(seed)
    A = rng.standard_normal((m, d))
    y = np.where(rng.standard_normal(m) > 0, 1.0, -1.0)
    x = rng.standard_normal(d)
    return A, y, x


def test_logistic_loss_equals_library_logaddexp():
    A, y, x = _tiny_logistic()
    l2 = 0.3
    want = np.mean(np.logaddexp(0.0, -y * (A @ x))) + 0.5 * l2 * np.dot(x, x)
    assert abs(o.logistic_loss(A, y, x, l2) - want) < 1e-13
    # large margins do not overflow
    assert np.isfinite(o.logistic_loss(1000 * A, y, x, 0.0))


def test_logistic_gradient_by_finite_differences():
    A, y, x = _tiny_logistic(1)
    l2 = 0.05
    g = o.logistic_grad(A, y, np.arange(A.shape[0]), x, l2)
    eps = 1e-6
    for j in range(x.size):
        e = np.zeros_like(x)
        e[j] = eps
        fd = (o.logistic_loss(A, y, x + e, l2) - o.logistic_loss(A, y, x - e, l2)) / (2 * eps)
        assert abs(fd - g[j]) < 1e-8


def test_logistic_minibatch_gradient_is_gradient_of_minibatch_loss():
    A, y, x = _tiny_logistic(2, m=16)
    rows = np.array([3, 3, 7, 0, 15, 7], dtype=np.int32)       # duplicates count twice
    g = o.logistic_grad(A, y, rows, x, 0.0)
    eps = 1e-6
    for j in range(x.size):
        e = np.zeros_like(x)
        e[j] = eps
        fd = (o.logistic_loss(A[rows], y[rows], x + e, 0.0)
              - o.logistic_loss(A[rows], y[rows], x - e, 0.0)) / (2 * eps)
        assert abs(fd - g[j]) < 1e-8


def test_batch_indices_range_determinism_uniformity():
    m, batch = 64, 128
    idx = o.batch_indices(5, 9, 2, batch, m)
    assert idx.min() >= 0 and idx.max() < m
    assert np.array_equal(idx, o.batch_indices(5, 9, 2, batch, m))
    assert not np.array_equal(idx, o.batch_indices(5, 10, 2, batch, m))
    assert not np.array_equal(idx, o.batch_indices(5, 9, 3, batch, m))
    # a prefix of a longer draw is the shorter draw
    assert np.array_equal(idx[:40], o.batch_indices(5, 9, 2, 40, m))
    # the draw is the generator's words reduced mod m
    w = np.concatenate([o.philox4x32_10([t, 2, 9, 4], [5, 0]) for t in range(batch // 4)])
    assert np.array_equal(idx, (w % m).astype(np.int32))
    allidx = np.concatenate([o.batch_indices(5, k, i, batch, m) for k in range(20)
                             for i in range(8)])
    counts = np.bincount(allidx, minlength=m)
    expect = allidx.size / m
    chi2 = ((counts - expect) ** 2 / expect).sum()
    assert chi2 < 2 * m      # mean m-1, sd ~ sqrt(2m)


def test_logistic_run_decreases_global_loss_and_matches_manual_step():
    rng = np.random.default_rng(3)
    n, m, d, batch, l2, gamma, seed = 4, 32, 6, 8, 1e-3, 0.5, 77
    A = rng.standard_normal((n, m, d)) / np.sqrt(d)
    xs = rng.standard_normal(d)
    y = np.where(A @ xs >= 0, 1.0, -1.0)
    p = o.Problem(o.TOPO_RING, 4, gamma, seed, objective="logistic", data=A, labels=y, l2=l2,
                  batch=batch)
    X = np.zeros((n, d))
    # one step by hand: per-node gradient on its own drawn rows, then the ring mix
    G = np.stack([o.logistic_grad(A[i], y[i], o.batch_indices(seed, 0, i, batch, m), X[i], l2)
                  for i in range(n)])
    Y = X - gamma * G
    want = np.stack([(Y[(i - 1) % n] + Y[i] + Y[(i + 1) % n]) / 3 for i in range(n)])
    assert np.allclose(o.step_f64(p, X, 0), want, rtol=1e-13, atol=1e-15)
    l0 = o.global_logistic_loss(A, y, X.mean(0), l2)
    X = o.run_f64(p, X, 0, 60)
    assert o.global_logistic_loss(A, y, X.mean(0), l2) < 0.8 * l0


# ---------------------------------------------------------------- seeded data, AGA
def test_init_streams():
    n, d, seed = 6, 4000, 31
    B = o.init_b(n, d, seed)
    assert abs(B.mean()) < 0.03 and abs(B.std() - 1) < 0.02
    Bs = o.init_b(n, d, seed, shift=0.5)
    s = np.array([o.normal4(seed, 3, 0, i, 0)[0] for i in range(n)])
    assert np.allclose(Bs - B, 0.5 * s[:, None], atol=1e-15)
    assert np.array_equal(o.init_b(n, 16, seed, col0=100), B[:, 100:116])
    assert not o.init_x0(n, d, seed, o.X0_ZERO).any()
    Xs = o.init_x0(n, d, seed, o.X0_SHARED_NORMAL, std=0.1)
    assert np.all(Xs == Xs[0]) and abs(Xs[0].std() - 0.1) < 0.005
    Xp = o.init_x0(n, d, seed, o.X0_PER_NODE_NORMAL, std=2.0)
    assert not np.array_equal(Xp[0], Xp[1]) and abs(Xp.std() - 2.0) < 0.05
    assert abs(np.corrcoef(Xp[0], B[0])[0, 1]) < 0.06          # separate streams


def test_aga_period_update_worked_example():
    # Algorithm 2: during warm-up F_init <- (F_init + F)/2; afterwards H <- ceil(F_init/F * H_init)
    F_init, H = 0.0, 4
    F_init, H = o.aga_update(3, 10, 4, 2.0, F_init, H)
    assert (F_init, H) == (1.0, 4)
    F_init, H = o.aga_update(7, 10, 4, 3.0, F_init, H)
    assert (F_init, H) == (2.0, 4)
    F_init, H = o.aga_update(11, 10, 4, 0.5, F_init, H)
    assert (F_init, H) == (2.0, 16)
    F_init, H = o.aga_update(27, 10, 4, 0.6, F_init, H)
    assert (F_init, H) == (2.0, 14)          # ceil(13.33)


def test_vector_box_muller_and_mean_loss_helpers():
    rng = np.random.default_rng(0)
    a = rng.integers(0, 2**32, 50, dtype=np.uint64).astype(np.uint32)
    b = rng.integers(0, 2**32, 50, dtype=np.uint64).astype(np.uint32)
    z = o.box_muller_many(a, b)
    for t in range(50):
        assert np.array_equal(z[t], o.box_muller(int(a[t]), int(b[t])))
    X = rng.standard_normal((3, 4))
    B = rng.standard_normal((3, 4))
    assert abs(o.quadratic_mean_loss(X, B) - 0.5 * np.linalg.norm(X - B, "fro") ** 2 / 3) < 1e-13


def test_metropolis_weights_are_doubly_stochastic_and_mix_like_dense_w():
    rng = np.random.default_rng(12)
    n = 9
    adj = rng.uniform(size=(n, n)) < 0.35
    adj = np.triu(adj, 1)
    adj = adj | adj.T
    adj[np.arange(n), (np.arange(n) + 1) % n] = True          # keep it connected: add a ring
    adj = adj | adj.T
    W = o.metropolis_w(adj)
    assert (W >= 0).all() and np.allclose(W, W.T)
    assert np.allclose(W.sum(0), 1, atol=1e-15) and np.allclose(W.sum(1), 1, atol=1e-15)
    assert np.array_equal(W > 0, adj | np.eye(n, dtype=bool))   # w_ij > 0 exactly on neighbours and i = j
    assert np.linalg.norm(W - np.full((n, n), 1.0 / n), 2) < 1.0  # beta < 1: connected graph (Assumption 3)
    B = rng.standard_normal((n, 6))
    X = rng.standard_normal((n, 6))
    p = o.Problem(o.TOPO_SPARSE, 3, 0.2, 4, sigma=0.3, data=B, W=W)
    for k in range(5):
        a, b = o.step_f64(p, X, k, dense=False), o.step_f64(p, X, k, dense=True)
        assert np.allclose(a, b, rtol=1e-12, atol=1e-13)
        assert np.allclose(a.mean(0), o.quadratic_half_step(X, B, 0.2, 0.3, 4, k).mean(0), atol=1e-13)
        X = a


def test_counter_layout_of_the_noise_generator():
    # the documented keying: counter = (column group q, node i, iteration k, stream id),
    # key = (seed low word, seed high word); (z0,z1) from words 0,1 and (z2,z3) from words 2,3
    seed, stream, k, i, q = (0x89ABCDEF << 32) | 0x01234567, 3, 1000, 17, 123456
    w = o.philox4x32_10([q, i, k, stream], [0x01234567, 0x89ABCDEF])
    want = np.concatenate([o.box_muller(int(w[0]), int(w[1])), o.box_muller(int(w[2]), int(w[3]))])
    assert np.array_equal(o.normal4(seed, stream, k, i, q), want)
