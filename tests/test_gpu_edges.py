"""Edge cases and invariants of the CUDA path: extreme node counts, counters at the end of their
range, structural properties the paper's setting fixes (checked on the GPU results themselves)."""
import numpy as np
import pytest

import paper_2105_09080_b200 as pkg
from oracle import gpga_oracle as o
from paper_2105_09080_b200.inputs import logistic_inputs, quadratic_inputs
from test_gpu_parity import TOL_RUN, TOL_STEP, TOPO, close, make_quadratic

pytestmark = pytest.mark.gpu


def _torch():
    import torch
    return torch


@pytest.mark.parametrize("topo,n,d", [("ring", 4096, 8), ("exp", 4096, 12), ("ring", 4097, 8), ("ring", 5000, 5),
                                      ("exp", 8192, 4), ("static_exp", 1024, 8), ("grid", 4096, 4)])
def test_many_nodes_few_columns(topo, n, d):
    """n at and beyond what the shared-memory tile holds (4096 rows): both kernel families."""
    X0, B = quadratic_inputs(n, d, n + d, x0="per_node")
    for H, k in ((0, 3), (2, 1)):
        g, p = make_quadratic(n, d, topo, H, 0.3, 5, 0.2, X0, B)
        if topo == "grid":
            p.grid_cols = 64
        g.step(k)
        ok, worst = close(g.get_x().cpu().numpy(), o.step(p, X0, k), TOL_STEP)
        assert ok, (H, k, worst)
        xi = o.consensus_distance(o.step(p, X0, k))
        assert abs(g.consensus_distance() - xi) <= 1e-5 * xi + 1e-9
        g.close()


def test_counters_at_the_end_of_their_range():
    """Largest iteration index, a seed using all 64 bits, the largest column offset."""
    n, d = 4, 64
    X0, B = quadratic_inputs(n, d, 3, x0="per_node")
    seed = 0xFEDCBA9876543210
    k = 2**32 - 1
    col0 = 2**34 - 64 - 4
    g, p = make_quadratic(n, d, "exp", 0, 0.1, seed, 1.0, X0, B, col0=col0)
    g.step(k)
    ok, worst = close(g.get_x().cpu().numpy(), o.step(p, X0, k), TOL_STEP)
    assert ok, worst
    # a wide state keyed far into the column range goes through the streaming kernels
    d2 = 19_004
    X0, B = quadratic_inputs(n, d2, 4, x0="per_node")
    col0 = 2**34 - d2 - 4
    g, p = make_quadratic(n, d2, "ring", 0, 0.1, seed, 1.0, X0, B, col0=col0)
    g.step(k)
    ok, worst = close(g.get_x().cpu().numpy(), o.step(p, X0, k), TOL_STEP)
    assert ok, worst


@pytest.mark.parametrize("topo,d", [("ring", 1 << 18), ("exp", 1 << 18), ("grid", 20_000), ("ring", 1024)])
def test_mixing_preserves_the_node_mean_on_the_gpu(topo, d):
    """W is doubly stochastic: with no gradient step the column means do not move (Section 3)."""
    n = 16
    X0, B = quadratic_inputs(n, d, 11, x0="per_node")
    g, _ = make_quadratic(n, d, topo, 0, 0.0, 1, 0.0, X0, B)
    before = X0.astype(np.float64).mean(0)
    g.run(5)
    after = g.get_x().cpu().numpy().astype(np.float64).mean(0)
    assert np.abs(after - before).max() <= 5e-7
    assert g.consensus_distance() < o.consensus_distance(X0)


def test_ring_contracts_by_lambda2_on_the_gpu():
    """No gradient, no noise, state on the second eigenvector: each ring step multiplies it by
    lambda_2 = (1 + 2 cos(2 pi / n)) / 3 (Appendix A: ||(W - J)^k|| <= beta^k with equality here)."""
    n, d = 32, 1 << 16
    lam = (1 + 2 * np.cos(2 * np.pi / n)) / 3
    rng = np.random.default_rng(0)
    X0 = (np.cos(2 * np.pi * np.arange(n) / n)[:, None] * rng.standard_normal((1, d))).astype(np.float32)
    g, _ = make_quadratic(n, d, "ring", 0, 0.0, 1, 0.0, X0, np.zeros_like(X0))
    xi_prev = g.consensus_distance()
    for _ in range(6):
        g.run(1)
        xi = g.consensus_distance()
        assert abs(np.sqrt(xi / xi_prev) - lam) < 1e-5
        xi_prev = xi


def test_period_one_is_parallel_sgd():
    """H = 1: W = (1/n) 1 1^T every step, all rows identical after every iteration (Section 3)."""
    n, d = 8, 32_768
    X0, B = quadratic_inputs(n, d, 12)
    g, p = make_quadratic(n, d, "exp", 1, 0.1, 9, 0.3, X0, B)
    want = X0
    for k in range(5):
        g.step(k)
        want = o.step(p, want, k)
        got = g.get_x().cpu().numpy()
        assert np.all(got == got[0])
        assert g.consensus_distance() == 0.0
    ok, worst = close(got, want, TOL_RUN)
    assert ok, worst


def test_step_size_schedule_and_period_change_between_steps():
    """gamma halved mid-run (the convex experiment's schedule) and H changed on the fly."""
    n, d = 8, 20_004
    X0, B = quadratic_inputs(n, d, 13)
    g, p = make_quadratic(n, d, "ring", 4, 0.2, 9, 0.1, X0, B)
    g.run(6)
    want = o.run(p, X0, 0, 6)
    g.set_gamma(0.1)
    g.set_period(2)
    p.gamma, p.H = 0.1, 2
    g.run(6)
    want = o.run(p, want, 6, 6)
    ok, worst = close(g.get_x().cpu().numpy(), want, TOL_RUN)
    assert ok, worst
    assert g.get_k() == 12


def test_adaptive_period_with_the_logistic_objective():
    torch = _torch()
    n, m, d, batch, K, H_init, warm = 8, 256, 64, 32, 40, 2, 6
    A, y = logistic_inputs(n, m, d, 21)
    X0 = np.zeros((n, d), dtype=np.float32)
    g = pkg.Gpga(n, d, pkg.GPGA_TOPO_RING, 0, 0.5, 7)
    g.set_objective(pkg.GPGA_OBJ_LOGISTIC, l2=1e-3, m=m, batch=batch)
    xa = torch.from_numpy(X0).cuda()
    g.bind(xa, torch.empty_like(xa), torch.from_numpy(A).cuda(), torch.from_numpy(y).cuda())
    periods = g.run_adaptive(K, H_init, warm)
    p = o.Problem(o.TOPO_RING, 0, 0.5, 7, objective="logistic", data=A, labels=y, l2=1e-3, batch=batch)
    X, H, C, F_init, want_periods = X0, H_init, 0, 0.0, []
    for k in range(K):
        C += 1
        glob = C == H
        if glob:   # Algorithm 2: mean over nodes of the mini-batch loss of this iteration at x^(k)
            F = np.mean([o.logistic_loss(A[i][o.batch_indices(7, k, i, batch, m)],
                                         y[i][o.batch_indices(7, k, i, batch, m)], X[i], 1e-3) for i in range(n)])
        p.H = 1 if glob else 0
        X = o.step(p, X, k)
        if glob:
            want_periods.append(H)
            C = 0
            F_init, H = o.aga_update(k, warm, H_init, F, F_init, H)
    assert periods == want_periods
    ok, worst = close(g.get_x().cpu().numpy(), X, TOL_RUN)
    assert ok, worst


def test_logistic_with_padded_state_rows():
    torch = _torch()
    n, m, d, ld, batch = 4, 64, 32, 48, 16
    A, y = logistic_inputs(n, m, d, 22)
    rng = np.random.default_rng(2)
    X0 = (0.2 * rng.standard_normal((n, d))).astype(np.float32)
    g = pkg.Gpga(n, d, pkg.GPGA_TOPO_EXP, 3, 0.3, 7)
    g.set_objective(pkg.GPGA_OBJ_LOGISTIC, l2=1e-3, m=m, batch=batch)
    g.set_row_stride(ld)
    bufs = [torch.full((n, ld), -7.0, dtype=torch.float32, device="cuda") for _ in range(2)]
    bufs[0][:, :d] = torch.from_numpy(X0).cuda()
    g.bind(bufs[0], bufs[1], torch.from_numpy(A).cuda(), torch.from_numpy(y).cuda())
    g.run(7)
    p = o.Problem(o.TOPO_EXP, 3, 0.3, 7, objective="logistic", data=A, labels=y, l2=1e-3, batch=batch)
    want = o.run(p, X0, 0, 7)
    out = g.get_x().cpu().numpy()
    ok, worst = close(out[:, :d], want, TOL_RUN)
    assert ok, worst
    assert np.all(out[:, d:] == -7.0)
    f = o.global_logistic_loss(A, y, want.astype(np.float64).mean(0), 1e-3)
    assert abs(g.global_loss() - f) <= 1e-4 * f


@pytest.mark.parametrize("topo,n,d,H", [("ring", 8, 65_536, 4), ("exp", 32, 4096, 8), ("ring", 7, 1031, 3),
                                        ("grid", 12, 520, 5), ("static_exp", 16, 64, 0), ("none", 5, 36, 2),
                                        ("ring", 1, 8, 2), ("exp", 2, 20_004, 1), ("ring", 600, 24, 4)])
def test_multi_iteration_launch_equals_single_iterations(topo, n, d, H):
    """gpga_run keeps a small state in shared memory across iterations (one launch for many
    iterations); the result is bit-identical to stepping one launch per iteration."""
    X0, B = quadratic_inputs(n, d, 31 + n, x0="shared", x0_std=0.5)
    K = 13
    g, p = make_quadratic(n, d, topo, H, 0.1, 17, 0.2, X0, B)
    if topo == "grid":
        p.grid_cols = 4
    g.run(K)
    assert g.launch_count() == 1 and g.get_k() == K
    fused = g.get_x().cpu().numpy().copy()
    g2, _ = make_quadratic(n, d, topo, H, 0.1, 17, 0.2, X0, B)
    for k in range(K):
        g2.step(k)
    assert g2.launch_count() == K
    assert np.array_equal(fused, g2.get_x().cpu().numpy())
    ok, worst = close(fused, o.run(p, X0, 0, K), TOL_RUN)
    assert ok, worst
    # continuing from the middle of a period gives the same as one long run
    g3, _ = make_quadratic(n, d, topo, H, 0.1, 17, 0.2, X0, B)
    g3.run(5)
    g3.run(K - 5)
    assert np.array_equal(fused, g3.get_x().cpu().numpy())


# row-streaming kernels (wide d, scalar tail included), the shared-memory tile kernel (narrow d and
# the grid / static exponential / W = I mixes) and the multi-iteration launch
@pytest.mark.parametrize("topo,n,d,H", [("ring", 8, 40_000, 3), ("exp", 16, 24_004, 2), ("ring", 2, 30_001, 2),
                                        ("exp", 8, 20_003, 0), ("ring", 7, 1031, 3), ("grid", 12, 520, 5),
                                        ("static_exp", 16, 64, 0), ("none", 5, 36, 2), ("exp", 32, 4096, 8)])
def test_in_place_update_equals_the_double_buffered_one(topo, n, d, H):
    """Binding the same buffer as x_a and x_b overwrites X^(k) with X^(k+1); every element must come
    out exactly as with two buffers, stepping one launch per iteration and through gpga_run."""
    torch = _torch()
    X0, B = quadratic_inputs(n, d, 77 + n, x0="shared", x0_std=0.5)
    K = 6
    g, p = make_quadratic(n, d, topo, H, 0.1, 23, 0.2, X0, B)
    if topo == "grid":
        p.grid_cols = 4               # the library's default for n = 12
    for k in range(K):
        g.step(k)
    want = g.get_x().cpu().numpy().copy()
    for stepwise in (True, False):
        h = pkg.Gpga(n, d, TOPO[topo][0], H, 0.1, 23)
        h.set_objective(pkg.GPGA_OBJ_QUADRATIC, sigma=0.2)
        x = torch.from_numpy(X0).cuda()
        h.bind(x, x, torch.from_numpy(B).cuda())
        if stepwise:
            for k in range(K):
                h.step(k)
        else:
            h.run(K)
        assert h.get_k() == K
        assert np.array_equal(x.cpu().numpy(), want), (topo, stepwise)
        h.close()
    ok, worst = close(want, o.run(p, X0, 0, K), TOL_RUN)
    assert ok, worst


def test_in_place_update_with_the_logistic_objective():
    torch = _torch()
    n, m, d, batch, K = 8, 128, 256, 48, 7
    A, y = logistic_inputs(n, m, d, 5)
    rng = np.random.default_rng(4)
    X0 = (0.2 * rng.standard_normal((n, d))).astype(np.float32)
    outs = []
    for in_place in (False, True):
        g = pkg.Gpga(n, d, pkg.GPGA_TOPO_RING, 3, 0.3, 9)
        g.set_objective(pkg.GPGA_OBJ_LOGISTIC, l2=1e-3, m=m, batch=batch)
        xa = torch.from_numpy(X0).cuda()
        g.bind(xa, xa if in_place else torch.empty_like(xa), torch.from_numpy(A).cuda(), torch.from_numpy(y).cuda())
        g.run(K)
        outs.append(g.get_x().cpu().numpy().copy())
        g.close()
    assert np.array_equal(outs[0], outs[1])
    p = o.Problem(o.TOPO_RING, 3, 0.3, 9, objective="logistic", data=A, labels=y, l2=1e-3, batch=batch)
    ok, worst = close(outs[1], o.run(p, X0, 0, K), TOL_RUN)
    assert ok, worst


def test_partly_overlapping_state_buffers_are_rejected():
    torch = _torch()
    n, d = 4, 64
    g = pkg.Gpga(n, d, pkg.GPGA_TOPO_RING, 2, 0.1, 1)
    big = torch.zeros(2 * n * d, dtype=torch.float32, device="cuda")
    data = torch.zeros(n * d, dtype=torch.float32, device="cuda")
    scratch = torch.empty(g.scratch_bytes(), dtype=torch.uint8, device="cuda")
    with pytest.raises(pkg.GpgaError) as err:
        g.bind_raw(big.data_ptr(), big.data_ptr() + 64, data.data_ptr(), None, scratch.data_ptr(), scratch.numel())
    assert err.value.status == pkg.GPGA_ERR_INVALID_ARG
    g.bind_raw(big.data_ptr(), big.data_ptr() + n * d * 4, data.data_ptr(), None, scratch.data_ptr(), scratch.numel())


@pytest.mark.parametrize("topo,n,d,H,fused", [("exp", 16, 1_500_004, 8, True), ("ring", 32, 600_000, 5, True),
                                              ("ring", 64, 300_000, 4, True), ("ring", 100, 200_000, 3, True),
                                              ("ring", 200, 100_000, 4, True), ("exp", 256, 80_000, 0, True),
                                              ("ring", 300, 70_000, 4, False), ("ring", 16, 1_200_000, 2, True),
                                              ("ring", 16, 1_200_000, 1, True)])
def test_long_runs_with_few_nodes_take_the_multi_iteration_launch_at_any_size(topo, n, d, H, fused):
    """Above 64 MB of state gpga_run still advances many iterations per launch when n <= 256 (one cell
    per thread) and the run has at least 8 iterations (the on-chip arithmetic is then faster than
    streaming the state from HBM every iteration, also with a global average every iteration); wider
    n keeps one launch per iteration.  Either way the result is bit-identical to stepping, and within
    tolerance of the oracle on a slice of columns."""
    X0, B = quadratic_inputs(n, d, 5 + n, x0="shared", x0_std=0.5)
    assert 12 * n * d > 64 << 20
    K = 40
    g, _ = make_quadratic(n, d, topo, H, 0.05, 29, 0.1, X0, B)
    g.run(K)
    assert g.launch_count() == (1 if fused else K)
    got = g.get_x().cpu().numpy().copy()
    g2, _ = make_quadratic(n, d, topo, H, 0.05, 29, 0.1, X0, B)
    for k in range(K):
        g2.step(k)
    assert np.array_equal(got, g2.get_x().cpu().numpy())
    g3, _ = make_quadratic(n, d, topo, H, 0.05, 29, 0.1, X0, B)
    g3.run(K - 7)                      # fewer than 8 left after the first call: falls back to stepping
    l0 = g3.launch_count()
    g3.run(7)
    assert g3.launch_count() - l0 == (7 if 12 * n * d > 64 << 20 else 1)
    assert np.array_equal(got, g3.get_x().cpu().numpy())
    c0, w = (d // 2) // 4 * 4, 2048
    p = o.Problem(TOPO[topo][1], H, 0.05, 29, sigma=0.1, data=np.ascontiguousarray(B[:, c0:c0 + w]), col0=c0)
    ok, worst = close(got[:, c0:c0 + w], o.run(p, np.ascontiguousarray(X0[:, c0:c0 + w]), 0, K), TOL_RUN)
    assert ok, worst


def test_multi_iteration_launch_is_chunked_for_long_runs():
    n, d, K = 4, 256, 2500            # more than one launch worth of iterations
    X0, B = quadratic_inputs(n, d, 5)
    g, p = make_quadratic(n, d, "ring", 16, 0.05, 3, 0.1, X0, B)
    g.run(K)
    assert g.launch_count() == 3 and g.get_k() == K
    ok, worst = close(g.get_x().cpu().numpy(), o.run(p, X0, 0, K), TOL_RUN)
    assert ok, worst


@pytest.mark.parametrize("n,d", [(9, 40), (30, 1030), (16, 20_004)])
def test_general_sparse_weight_matrix(n, d):
    """Topology SPARSE: Metropolis weights of a random connected graph, given in CSR form."""
    torch = _torch()
    rng = np.random.default_rng(n)
    adj = np.triu(rng.uniform(size=(n, n)) < 0.3, 1)
    adj[np.arange(n - 1), np.arange(1, n)] = True
    adj = adj | adj.T
    W = o.metropolis_w(adj)
    row_ptr, col, val = [0], [], []
    for i in range(n):
        nz = np.nonzero(W[i])[0]
        col += list(nz)
        val += list(W[i, nz])
        row_ptr.append(len(col))
    X0, B = quadratic_inputs(n, d, 77, x0="per_node")
    for H, K in ((0, 1), (3, 7)):
        g = pkg.Gpga(n, d, pkg.GPGA_TOPO_SPARSE, H, 0.2, 5)
        g.set_objective(pkg.GPGA_OBJ_QUADRATIC, sigma=0.3)
        xa = torch.from_numpy(X0).cuda()
        g.bind(xa, torch.empty_like(xa), torch.from_numpy(B).cuda())
        with pytest.raises(pkg.GpgaError):
            g.step(0)                                   # no weight matrix yet
        g.set_weight_matrix(torch.tensor(row_ptr, dtype=torch.int32, device="cuda"),
                            torch.tensor(col, dtype=torch.int32, device="cuda"),
                            torch.tensor(val, dtype=torch.float32, device="cuda"))
        p = o.Problem(o.TOPO_SPARSE, H, 0.2, 5, sigma=0.3, data=B, W=W)
        if K == 1:
            g.step(0)
        else:
            g.run(K)
        ok, worst = close(g.get_x().cpu().numpy(), o.run(p, X0, 0, K), TOL_STEP if K == 1 else TOL_RUN)
        assert ok, (H, K, worst)
        g.close()


def test_bounded_wait_gives_up_and_reports_timeout():
    """A wait inside a kernel that can never be satisfied ends by itself and surfaces as
    GPGA_ERR_TIMEOUT at the next synchronising call; the GPU context stays usable."""
    n, d = 4, 64
    X0, B = quadratic_inputs(n, d, 1)
    g, _ = make_quadratic(n, d, "ring", 0, 0.1, 1, 0.0, X0, B)
    assert g.consensus_distance() == 0.0
    g.selftest_bounded_wait()
    with pytest.raises(pkg.GpgaError) as err:
        g.consensus_distance()
    assert err.value.status == pkg.GPGA_ERR_TIMEOUT
    with pytest.raises(pkg.GpgaError) as err:       # sticky
        g.step(0)
    assert err.value.status == pkg.GPGA_ERR_TIMEOUT
    g.close()
    # another handle on the same device works as before
    g2, p = make_quadratic(n, d, "ring", 0, 0.1, 1, 0.2, X0, B)
    g2.step(0)
    ok, worst = close(g2.get_x().cpu().numpy(), o.step(p, X0, 0), TOL_STEP)
    assert ok, worst
