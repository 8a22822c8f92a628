"""The paper's convex experiment (Section 5.1): logistic regression with d = 10 features (padded to
12 columns), M = 8000 samples per node drawn as h ~ N(0, 10 I) with Bernoulli labels, step size 0.2
halved every 1000 iterations.  Parity with the oracle at the experiment's own shape, parity of the
batched-trials form (T independent copies of the network as one block-diagonal problem), and the
qualitative ordering the section reports."""
import numpy as np
import pytest

import paper_2105_09080_b200 as pkg
from oracle import gpga_oracle as o
from paper_2105_09080_b200 import convex_experiment as ce
from paper_2105_09080_b200 import topologies
from paper_2105_09080_b200.inputs import convex_experiment_inputs
from test_gpu_parity import TOL_RUN, close

pytestmark = pytest.mark.gpu

SEED = 20210509


def _torch():
    import torch
    return torch


@pytest.mark.parametrize("topo,H", [("ring", 16), ("ring", 0), ("ring", 1)])
def test_experiment_shape_2000_iterations_with_a_step_size_halving(topo, H):
    """n = 20, M = 8000, batch 8 on the ring: Gossip-PGA with H = 16, Gossip SGD and parallel SGD over
    2000 iterations (the step size halves at iteration 1000) against the oracle."""
    torch = _torch()
    n, m, batch, K = 20, 8000, 8, 2000
    A, y = convex_experiment_inputs(n, m, 10, seed=1020)
    d = A.shape[2]
    assert d == 12
    g = pkg.Gpga(n, d, pkg.GPGA_TOPO_RING, H, 0.2, SEED)
    g.set_objective(pkg.GPGA_OBJ_LOGISTIC, l2=0.0, m=m, batch=batch)
    xa = torch.zeros((n, d), device="cuda")
    g.bind(xa, torch.empty_like(xa), torch.from_numpy(A).cuda(), torch.from_numpy(y).cuda())
    A64, y64 = A.astype(np.float64), y.astype(np.float64)
    p = o.Problem(o.TOPO_RING, H, 0.2, SEED, objective="logistic", data=A64, labels=y64, l2=0.0, batch=batch)
    want = np.zeros((n, d), dtype=np.float32)
    for seg, gamma in ((0, 0.2), (1000, 0.1)):
        g.set_gamma(gamma)
        g.run(1000)
        p.gamma = gamma
        want = o.run(p, want, seg, 1000)
        got = g.get_x().cpu().numpy()
        ok, worst = close(got, want, TOL_RUN)
        assert ok, (topo, H, seg, worst)
        assert not got[:, 10:].any()                      # padded weights receive zero gradient and stay 0
        xi = o.consensus_distance(got)
        assert abs(g.consensus_distance() - xi) <= 1e-5 * xi
        f = o.global_logistic_loss(A64, y64, want.astype(np.float64).mean(0), 0.0)
        assert abs(g.global_loss() - f) <= 1e-5 * f
    g.close()


@pytest.mark.parametrize("method,topology", [("gossip_pga", "ring"), ("local_sgd", "ring"), ("gossip_sgd", "grid"),
                                             ("parallel_sgd", "ring"), ("gossip_pga", "static_exp")])
def test_batched_trials_equal_the_oracle_on_the_block_diagonal_problem(method, topology):
    """Three copies of a 20-node network as one 60-node problem with a block-diagonal W: the run
    equals the oracle driven with the same matrices (gossip matrix, and the per-copy average on
    the iterations with mod(k + 1, H) = 0), and every copy's diagnostics are its own."""
    torch = _torch()
    n, T, m, batch, period, iters, every, halve = 20, 3, 600, 8, 16, 330, 110, 150
    parts = [convex_experiment_inputs(n, m, 10, seed=50 + t) for t in range(T)]
    A = np.concatenate([q[0] for q in parts])
    y = np.concatenate([q[1] for q in parts])
    bt = ce.BatchedTrials(torch.from_numpy(A).cuda(), torch.from_numpy(y).cuda(), n, topology, batch, SEED,
                          halve_every=halve)
    marks, loss, cons = bt.run(method, period, iters, every)
    assert marks == [0, 110, 220, 330] and loss.shape == (4, T)
    got = bt.g.get_x().cpu().numpy()
    # the oracle on the same 60-node problem
    gossip_name, periodic = ce.METHODS[method]
    W_gossip = topologies.dense(gossip_name or topology, n, T)
    W_avg = topologies.dense("average", n, T)
    for W in (W_gossip, W_avg):
        assert np.allclose(W.sum(0), 1.0, atol=1e-6) and np.allclose(W.sum(1), 1.0, atol=1e-6)
    A64, y64 = A.astype(np.float64), y.astype(np.float64)
    p = o.Problem(o.TOPO_SPARSE, 0, 0.2, SEED, objective="logistic", data=A64, labels=y64, l2=0.0, batch=batch)
    X = np.zeros((n * T, A.shape[2]), dtype=np.float32)
    H = period if periodic else 0
    for k in range(iters):
        p.gamma = 0.2 * 0.5 ** (k // halve)
        p.W = W_avg if (H and (k + 1) % H == 0) else W_gossip
        X = o.step(p, X, k)
    ok, worst = close(got, X, TOL_RUN)
    assert ok, (method, topology, worst)
    for t in range(T):
        rows = slice(t * n, (t + 1) * n)
        f = o.global_logistic_loss(A64[rows], y64[rows], X[rows].astype(np.float64).mean(0), 0.0)
        assert abs(loss[-1, t] - f) <= 1e-5 * f
        xi = o.consensus_distance(got[rows])
        assert abs(cons[-1, t] - xi) <= 1e-5 * xi + 1e-30
    if method == "parallel_sgd":
        assert np.all(cons == 0.0)                          # every copy is averaged on every iteration
    bt.close()


def test_ordering_of_the_methods_on_the_ring():
    """What Section 5.1 reports, at a reduced size: periodic global averaging keeps the nodes closer
    to consensus than plain gossip, Local SGD with the same period drifts further apart than
    Gossip-PGA, and every method lowers the loss at the average."""
    res = ce.run_size(20, 6, 1200, 200, 8, 2000, False, "ring", 16, list(ce.METHODS))
    cons = {name: r[2][1:].mean() for name, r in res.items()}
    assert cons["parallel_sgd"] == 0.0
    assert cons["gossip_pga"] < cons["gossip_sgd"]
    assert cons["gossip_pga"] < cons["local_sgd"]
    for name, (marks, loss, _) in res.items():
        assert marks[-1] == 1200 and loss.shape == (7, 6)
        assert loss[-1].mean() < loss[0].mean()
    stage = {name: ce.transient_stage(res[name][0], res[name][1], res["parallel_sgd"][1]) for name in res}
    assert stage["parallel_sgd"] == 0
