"""Configuration-level parity: the benchmark configurations run through the C ABI and
compared with the oracle -- fully where the oracle finishes in seconds, on sampled column
blocks (columns evolve independently under the quadratic objective) at full size."""
import numpy as np
import pytest

import paper_2105_09080_b200 as pkg
from oracle import gpga_oracle as o
from paper_2105_09080_b200.inputs import logistic_inputs, quadratic_inputs
from test_gpu_parity import TOL_RUN, TOL_STEP, TOPO, close, make_quadratic

pytestmark = pytest.mark.gpu

SEED = 20210509


def _torch():
    import torch
    return torch


def test_config_1_ring_h4_full_run():
    # n=8, d=65536, ring, H=4, gamma=0.1, sigma=0.1, K=32, x0 = 0
    n, d, H, gamma, sigma, K = 8, 65536, 4, 0.1, 0.1, 32
    X0, B = quadratic_inputs(n, d, SEED)
    g, p = make_quadratic(n, d, "ring", H, gamma, SEED, sigma, X0, B)
    want = X0
    for k in range(K):
        g.step(k)
        want = o.step(p, want, k)
        ok, worst = close(g.get_x().cpu().numpy(), want, TOL_STEP if k == 0 else TOL_RUN)
        assert ok, (k, worst)
        if (k + 1) % H == 0:
            assert g.consensus_distance() == 0.0        # rows identical after a global average
        elif k % 5 == 0:
            xi = o.consensus_distance(want)
            assert abs(g.consensus_distance() - xi) <= 1e-5 * xi + n * d * (2.0**-22 * 8) ** 2
    # the run ends on a global average: K = 32, H = 4
    got = g.get_x().cpu().numpy()
    assert np.all(got == got[0])


def test_config_2_exp_h8_full_run():
    # n=32, d=2^20, one-peer exponential, H=8, gamma=0.05, sigma=0.1, K=64
    n, d, H, gamma, sigma, K = 32, 1 << 20, 8, 0.05, 0.1, 64
    X0, B = quadratic_inputs(n, d, SEED + 1)
    g, p = make_quadratic(n, d, "exp", H, gamma, SEED, sigma, X0, B)
    g.step(0)
    want1 = o.step(p, X0, 0)
    ok, worst = close(g.get_x().cpu().numpy(), want1, TOL_STEP)
    assert ok, worst
    g.run(K - 1)
    want = o.run(p, want1, 1, K - 1)
    ok, worst = close(g.get_x().cpu().numpy(), want, TOL_RUN)
    assert ok, worst
    xi = o.consensus_distance(want)
    assert abs(g.consensus_distance() - xi) <= 1e-5 * xi + n * d * (2.0**-22 * 8) ** 2


def test_config_2_exact_consensus_after_log2n_mixing_steps():
    # gamma = 0, sigma = 0, random per-node X0: five hops 1,2,4,8,16 give the exact average
    n, d = 32, 1 << 20
    X0, B = quadratic_inputs(n, d, SEED + 2, x0="per_node")
    g, p = make_quadratic(n, d, "exp", 0, 0.0, SEED, 0.0, X0, B)
    xi0 = g.consensus_distance()
    assert abs(xi0 - o.consensus_distance(X0)) <= 1e-5 * xi0
    g.run(4)
    assert g.consensus_distance() > 1e-3 * xi0            # not yet
    g.run(1)
    assert g.consensus_distance() <= 1e-12 * xi0          # float32 storage: exact up to rounding
    got = g.get_x().cpu().numpy()
    mean = X0.astype(np.float64).mean(0)
    assert np.abs(got - mean[None, :]).max() <= 1e-6


def test_init_from_seed_matches_oracle_streams():
    torch = _torch()
    n, d, c0 = 6, 4104, 8192
    for kind, okind, std, shift in ((pkg.GPGA_X0_ZERO, o.X0_ZERO, 1.0, 0.0),
                                    (pkg.GPGA_X0_SHARED_NORMAL, o.X0_SHARED_NORMAL, 0.1, 0.5),
                                    (pkg.GPGA_X0_PER_NODE_NORMAL, o.X0_PER_NODE_NORMAL, 1.0, 0.0)):
        g = pkg.Gpga(n, d, pkg.GPGA_TOPO_RING, 0, 0.1, SEED)
        g.set_column_offset(c0)
        xa, xb, b = g.allocate()
        g.init_from_seed(kind, std, shift)
        # seeded inputs are N(0,1)-scale numbers; the fast device Box-Muller is within 2.5e-5
        assert np.abs(b.cpu().numpy() - o.init_b(n, d, SEED, shift, c0)).max() <= 3e-5
        assert np.abs(xa.cpu().numpy() - o.init_x0(n, d, SEED, okind, std, c0)).max() <= 3e-5 * std
        if kind == pkg.GPGA_X0_SHARED_NORMAL:
            x = xa.cpu().numpy()
            assert np.all(x == x[0])
        g.close()
    # ragged d (scalar path)
    g = pkg.Gpga(3, 1031, pkg.GPGA_TOPO_RING, 0, 0.1, SEED)
    xa, xb, b = g.allocate()
    g.init_from_seed(pkg.GPGA_X0_PER_NODE_NORMAL, 2.0, 0.25)
    assert np.abs(b.cpu().numpy() - o.init_b(3, 1031, SEED, 0.25)).max() <= 3e-5
    assert np.abs(xa.cpu().numpy() - o.init_x0(3, 1031, SEED, o.X0_PER_NODE_NORMAL, 2.0)).max() <= 6e-5


def test_run_host_equals_device_run():
    torch = _torch()
    n, d, K = 8, 65536, 6
    X0, B = quadratic_inputs(n, d, SEED + 3)
    g, _ = make_quadratic(n, d, "ring", 4, 0.1, SEED, 0.1, X0, B)
    g.run(K)
    dev = g.get_x().cpu().numpy()
    g2, _ = make_quadratic(n, d, "ring", 4, 0.1, SEED, 0.1, np.zeros_like(X0), np.zeros_like(B))
    out = torch.empty((n, d), dtype=torch.float32).pin_memory()
    g2.run_host(torch.from_numpy(X0).pin_memory(), torch.from_numpy(B).pin_memory(), K, out)
    assert np.array_equal(out.numpy(), dev)
    # X0 = NULL means X^(0) = 0, filled on the device: the same run (X0 is zero here), whatever the
    # device buffers held before
    g2.x_bufs[0].fill_(7.0)
    g2.x_bufs[1].fill_(-3.0)
    out.fill_(float("nan"))
    g2.run_host(None, torch.from_numpy(B).pin_memory(), K, out)
    assert np.array_equal(out.numpy(), dev)


def test_run_host_zero_start_through_the_chunked_pipeline():
    """A state above 64 MB moves through the host entry as column chunks; with X0 = NULL every chunk
    of X^(0) is zeroed on the device instead of uploaded.  Same result as the resident run from zeros."""
    torch = _torch()
    n, d, K = 8, 3_000_000, 5
    B = np.random.default_rng(SEED).standard_normal((n, d), dtype=np.float32)
    X0 = np.zeros((n, d), dtype=np.float32)
    g, _ = make_quadratic(n, d, "exp", 3, 0.05, SEED, 0.1, X0, B)
    g.run(K)
    dev = g.get_x().cpu().numpy()
    g.x_bufs[0].fill_(1.5)
    g.x_bufs[1].fill_(2.5)
    out = torch.full((n, d), float("nan"), dtype=torch.float32).pin_memory()
    g.run_host(None, torch.from_numpy(B).pin_memory(), K, out)
    assert np.array_equal(out.numpy(), dev)
    assert np.array_equal(g.get_x().cpu().numpy(), dev)
    g.close()


# ------------------------------------------------------------------ logistic objective
def _make_logistic(n, m, d, batch, topo, H, gamma, l2, seed, A, y, X0):
    torch = _torch()
    g = pkg.Gpga(n, d, TOPO[topo][0], H, gamma, seed)
    g.set_objective(pkg.GPGA_OBJ_LOGISTIC, l2=l2, m=m, batch=batch)
    xa = torch.from_numpy(X0).cuda()
    g.bind(xa, torch.empty_like(xa), torch.from_numpy(A).cuda(), torch.from_numpy(y).cuda())
    p = o.Problem(TOPO[topo][1], H, gamma, seed, objective="logistic", data=A, labels=y, l2=l2,
                  batch=batch)
    return g, p


@pytest.mark.parametrize("topo", ["ring", "exp"])
# d <= 1024: rows staged by bulk asynchronous copies, one pipeline per warp, rows through registers
# once (d = 4: one lane busy; d = 260: ragged over the lanes); d <= 8192: staged in two alternating
# tiles, a thread owns 2 / 4 / 8 groups of four columns (d = 1028, 2052: ragged over the threads;
# 4096 and 8192: full); wider: plain loads; d >= 18944: gradient buffer + row-streaming step kernels
# instead of the tile kernel
@pytest.mark.parametrize("n,m,d,batch", [(4, 64, 32, 8), (8, 256, 1024, 128), (2, 100, 260, 50), (4, 20, 4, 33),
                                         (2, 64, 1028, 40), (4, 40, 2052, 70), (4, 24, 4096, 40),
                                         (2, 16, 8192, 8), (2, 16, 8196, 8), (2, 16, 20000, 33)])
def test_logistic_steps(topo, n, m, d, batch):
    A, y = logistic_inputs(n, m, d, SEED + n)
    rng = np.random.default_rng(0)
    X0 = (0.1 * rng.standard_normal((n, d))).astype(np.float32)
    g, p = _make_logistic(n, m, d, batch, topo, 4, 0.1, 1e-4, SEED, A, y, X0)
    g.step(0)
    want = o.step(p, X0, 0)
    ok, worst = close(g.get_x().cpu().numpy(), want, TOL_STEP)
    assert ok, worst
    g.run(11)
    want = o.run(p, want, 1, 11)
    ok, worst = close(g.get_x().cpu().numpy(), want, TOL_RUN)
    assert ok, worst
    # mini-batch loss of the next iteration's batch, at each node's own iterate
    k = g.get_k()
    f = np.mean([o.logistic_loss(A[i][o.batch_indices(SEED, k, i, batch, m)],
                                 y[i][o.batch_indices(SEED, k, i, batch, m)], want[i], 1e-4)
                 for i in range(n)])
    assert abs(g.mean_loss() - f) <= 1e-4 * abs(f)
    # global loss of problem (1) at the node average, over every local sample
    f_glob = o.global_logistic_loss(A, y, want.astype(np.float64).mean(0), 1e-4)
    assert abs(g.global_loss() - f_glob) <= 1e-4 * abs(f_glob)


@pytest.fixture(scope="module")
def c5_data():
    """The convex workload's data set (n = 64 nodes, m = 4096 samples of d = 1024 features) once
    for all sweep points: fp32 for the GPU, and the same values widened to fp64 once for the
    oracle (which otherwise converts all of A on every iteration)."""
    torch = _torch()
    n, m, d = 64, 4096, 1024
    A, y = logistic_inputs(n, m, d, SEED)
    return dict(n=n, m=m, d=d, A=A, y=y, A64=A.astype(np.float64), y64=y.astype(np.float64),
                A_dev=torch.from_numpy(A).cuda(), y_dev=torch.from_numpy(y).cuda())


# the ten (topology, H) points of the sweep; H = 0 encodes H = infinity (pure gossip)
C5_POINTS = [(topo, H) for topo in ("ring", "exp") for H in (1, 4, 16, 64, 0)]
# (501 and 1502 fall between global averages for every finite H > 1 of the sweep)
C5_CHECKPOINTS = (200, 501, 1000, 1502, 2000)


@pytest.mark.parametrize("topo,H", C5_POINTS)
def test_config_5_logistic_sweep_full_length(c5_data, topo, H):
    """Every point of the sweep for its whole K = 2000 iterations (batch 128, l2 = 1e-4,
    gamma = 0.1, X0 = 0) against the oracle, with the state, the consensus distance and the global
    loss f(xbar) of problem (1) compared at k = 0, 200, 501, 1000, 1502 and 2000."""
    torch = _torch()
    c = c5_data
    n, m, d, batch, l2, gamma = c["n"], c["m"], c["d"], 128, 1e-4, 0.1
    g = pkg.Gpga(n, d, TOPO[topo][0], H, gamma, SEED)
    g.set_objective(pkg.GPGA_OBJ_LOGISTIC, l2=l2, m=m, batch=batch)
    xa = torch.zeros((n, d), dtype=torch.float32, device="cuda")
    g.bind(xa, torch.empty_like(xa), c["A_dev"], c["y_dev"])
    p = o.Problem(TOPO[topo][1], H, gamma, SEED, objective="logistic", data=c["A64"], labels=c["y64"], l2=l2,
                  batch=batch)
    want = np.zeros((n, d), dtype=np.float32)
    f0 = o.global_logistic_loss(c["A64"], c["y64"], np.zeros(d), l2)
    assert abs(f0 - np.log(2.0)) < 1e-12                     # loss at x = 0
    assert abs(g.global_loss() - f0) <= 1e-6 * f0
    k = 0
    losses = [f0]
    for k_next in C5_CHECKPOINTS:
        g.run(k_next - k)
        want = o.run(p, want, k, k_next - k)
        k = k_next
        got = g.get_x().cpu().numpy()
        ok, worst = close(got, want, TOL_RUN)
        assert ok, (topo, H, k, worst)
        # the consensus-distance kernel against the oracle on the very state the GPU holds
        xi_gpu = g.consensus_distance()
        xi_same = o.consensus_distance(got)
        assert abs(xi_gpu - xi_same) <= 1e-5 * xi_same, (topo, H, k, xi_gpu, xi_same)
        # and against the oracle's own trajectory: sqrt(Xi) is the norm ||X - Xbar||_F, so the two
        # differ by at most the norm of the difference of the states
        xi_traj = o.consensus_distance(want)
        gap = np.linalg.norm(got.astype(np.float64) - want.astype(np.float64))
        assert abs(np.sqrt(xi_gpu) - np.sqrt(xi_traj)) <= gap * (1 + 1e-6) + 1e-12, (topo, H, k, xi_gpu, xi_traj)
        if H and k % H == 0:
            assert xi_gpu == 0.0 and xi_traj == 0.0           # rows identical after a global average
        else:
            assert xi_traj > 0.0 and xi_gpu > 0.0
        f = o.global_logistic_loss(c["A64"], c["y64"], want.astype(np.float64).mean(0), l2)
        assert abs(g.global_loss() - f) <= 1e-5 * f, (topo, H, k)
        losses.append(f)
    assert all(b < a for a, b in zip(losses, losses[1:]))     # the loss at the average keeps falling
    g.close()


# ------------------------------------------------------------------ Gossip-AGA
def test_adaptive_run_takes_gossip_stretches_in_one_launch_and_equals_single_steps():
    """Between two global averages Gossip-AGA's iterations are plain gossip steps; a stretch of 8 or
    more goes through the multi-iteration launch.  Periods and state must equal those of single steps
    driven from the host with the same rule."""
    n, d, K, H_init, warm = 16, 1_200_000, 90, 4, 8
    X0, B = quadratic_inputs(n, d, SEED + 6, x0="shared", x0_std=3.0)
    g, _ = make_quadratic(n, d, "exp", 0, 0.1, SEED, 0.05, X0, B)
    l0 = g.launch_count()
    periods = g.run_adaptive(K, H_init, warm)
    launches = g.launch_count() - l0
    assert max(periods) >= 9                                   # some stretch is long enough for one launch
    assert launches < K + 2 * len(periods)                     # fewer than one launch per iteration + the losses
    g2, _ = make_quadratic(n, d, "exp", 0, 0.1, SEED, 0.05, X0, B)
    H, count, F_init, want_periods = H_init, 0, 0.0, []
    for k in range(K):
        count += 1
        glob = count == H
        F = g2.mean_loss() if glob else 0.0
        g2.set_period(1 if glob else 0)
        g2.step(k)
        if glob:
            want_periods.append(H)
            count = 0
            F_init, H = o.aga_update(k, warm, H_init, F, F_init, H)
    assert periods == want_periods
    assert np.array_equal(g.get_x().cpu().numpy().view(np.uint32), g2.get_x().cpu().numpy().view(np.uint32))
    g.close()
    g2.close()


def test_adaptive_period_sequence_matches_oracle_driven_loop():
    n, d, K, H_init, warm = 8, 4096, 60, 2, 6
    X0, B = quadratic_inputs(n, d, SEED + 5, x0="shared", x0_std=3.0)
    g, p = make_quadratic(n, d, "ring", 0, 0.1, SEED, 0.05, X0, B)
    periods = g.run_adaptive(K, H_init, warm)
    # the same loop driven by the oracle (Algorithm 2)
    X, H, C, F_init, want_periods = X0, H_init, 0, 0.0, []
    for k in range(K):
        C += 1
        glob = C == H
        F = o.quadratic_mean_loss(X, B) if glob else 0.0
        p.H = 1 if glob else 0
        X = o.step(p, X, k)
        if glob:
            want_periods.append(H)
            C = 0
            F_init, H = o.aga_update(k, warm, H_init, F, F_init, H)
    assert periods == want_periods
    assert len(set(periods)) > 1 and periods[-1] > periods[0]      # the period grows as the loss falls
    ok, worst = close(g.get_x().cpu().numpy(), X, TOL_RUN)
    assert ok, worst
    assert abs(g.mean_loss() - o.quadratic_mean_loss(X, B)) <= 1e-5 * o.quadratic_mean_loss(X, B)
    xbar = np.repeat(X.astype(np.float64).mean(0, keepdims=True), n, axis=0)
    f_glob = o.quadratic_mean_loss(xbar, B)         # (1/n) sum_i 1/2 ||xbar - b_i||^2
    assert abs(g.global_loss() - f_glob) <= 1e-5 * f_glob
