"""gpga_run on the logistic objective (narrow states): many iterations in one launch, x_i resident
on chip, neighbours' half-step rows exchanged through global memory as (value, iteration tag)
words.  Every sum is formed in the order of the one-iteration kernels, so a run must equal the same
number of gpga_step calls bit for bit; parity with the oracle is checked on top.  (With H = 1 or 2
gpga_run keeps to single steps unless there are many nodes: they are faster there.)"""
import numpy as np
import pytest

import paper_2105_09080_b200 as pkg
from oracle import gpga_oracle as o
from paper_2105_09080_b200.inputs import logistic_inputs
from test_gpu_parity import TOL_RUN, TOPO, close

pytestmark = pytest.mark.gpu

SEED = 20210509


def _pair(n, m, d, batch, topo, H, X0, A, y, gamma=0.1, l2=1e-4):
    import torch
    out = []
    dA, dy = torch.from_numpy(A).cuda(), torch.from_numpy(y).cuda()
    for _ in range(2):
        g = pkg.Gpga(n, d, TOPO[topo][0], H, gamma, SEED)
        g.set_objective(pkg.GPGA_OBJ_LOGISTIC, l2=l2, m=m, batch=batch)
        xa = torch.from_numpy(X0).cuda()
        g.bind(xa, torch.empty_like(xa), dA, dy)
        out.append(g)
    return out


# (n, m, d, batch): full-size rows and batch; ragged batch (last chunk short, idle warps); rows ragged
# over the lanes and an odd number of column groups (unequal halves); one lane busy; n = 1 and 2
# (a node is its own neighbour); n not a power of two with a column-mean tail of 1, 2, 3 rows
SHAPES = [(8, 256, 1024, 128), (16, 64, 512, 100), (5, 100, 260, 50), (4, 20, 4, 33), (1, 40, 36, 7),
          (2, 40, 64, 128), (6, 30, 20, 9), (7, 30, 12, 40), (64, 128, 1024, 128)]


@pytest.mark.parametrize("n,m,d,batch", SHAPES)
@pytest.mark.parametrize("topo,H", [("ring", 4), ("ring", 0), ("ring", 3), ("exp", 3), ("exp", 0), ("exp", 5)])
def test_resident_run_equals_single_steps(topo, H, n, m, d, batch):
    if topo == "exp" and n & (n - 1):
        pytest.skip("the one-peer exponential graph needs n to be a power of two")
    A, y = logistic_inputs(n, m, d, SEED + n + d)
    rng = np.random.default_rng(n * 1000 + d)
    X0 = (0.1 * rng.standard_normal((n, d))).astype(np.float32)
    run, stepped = _pair(n, m, d, batch, topo, H, X0, A, y)
    K = 9
    launches0 = run.launch_count()
    run.run(K)
    assert run.launch_count() - launches0 == 1, "the run was not taken by the one-launch kernel"
    for k in range(K):
        stepped.step(k)
    a, b = run.get_x().cpu().numpy(), stepped.get_x().cpu().numpy()
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32)), float(np.abs(a - b).max())
    assert run.get_k() == K
    # a second run continues from the first (odd then even number of iterations: both buffers)
    run.run(6)
    for k in range(K, K + 6):
        stepped.step(k)
    a, b = run.get_x().cpu().numpy(), stepped.get_x().cpu().numpy()
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32))
    assert run.consensus_distance() == stepped.consensus_distance()
    run.close()
    stepped.close()


@pytest.mark.parametrize("topo,H,n,one_launch", [("ring", 1, 64, True), ("exp", 2, 64, True), ("ring", 2, 32, True),
                                                 ("ring", 1, 32, False), ("exp", 2, 16, False)])
def test_short_averaging_periods_take_one_launch_only_with_many_nodes(topo, H, n, one_launch):
    """With a global average every iteration or every other one the one-launch kernel is taken only
    where it is faster than single steps (n >= 48 for H = 1, n >= 24 for H = 2); either way the result
    equals single steps bit for bit."""
    m, d, batch, K = 64, 1024, 128, 10
    A, y = logistic_inputs(n, m, d, SEED + n)
    rng = np.random.default_rng(n + H)
    X0 = (0.1 * rng.standard_normal((n, d))).astype(np.float32)
    run, stepped = _pair(n, m, d, batch, topo, H, X0, A, y)
    launches0 = run.launch_count()
    run.run(K)
    assert (run.launch_count() - launches0 == 1) == one_launch
    for k in range(K):
        stepped.step(k)
    a, b = run.get_x().cpu().numpy(), stepped.get_x().cpu().numpy()
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32)), float(np.abs(a - b).max())
    run.close()
    stepped.close()


@pytest.mark.parametrize("topo,H", [("ring", 4), ("exp", 0)])
def test_resident_run_matches_oracle(topo, H):
    n, m, d, batch, K = 8, 128, 256, 64, 25
    A, y = logistic_inputs(n, m, d, SEED)
    X0 = np.zeros((n, d), dtype=np.float32)
    run, _ = _pair(n, m, d, batch, topo, H, X0, A, y)
    p = o.Problem(TOPO[topo][1], H, 0.1, SEED, objective="logistic", data=A, labels=y, l2=1e-4, batch=batch)
    run.run(K)
    want = o.run(p, X0, 0, K)
    ok, worst = close(run.get_x().cpu().numpy(), want, TOL_RUN)
    assert ok, worst


def test_resident_run_in_place_and_long():
    """x_a == x_b (update in place) and a run long enough to wrap every buffer and barrier phase
    many times; compared with single steps on the double buffer."""
    import torch
    n, m, d, batch, K = 16, 512, 1024, 128, 301
    A, y = logistic_inputs(n, m, d, SEED + 3)
    X0 = np.zeros((n, d), dtype=np.float32)
    dA, dy = torch.from_numpy(A).cuda(), torch.from_numpy(y).cuda()
    g = pkg.Gpga(n, d, pkg.GPGA_TOPO_EXP, 8, 0.1, SEED)
    g.set_objective(pkg.GPGA_OBJ_LOGISTIC, l2=1e-4, m=m, batch=batch)
    x = torch.from_numpy(X0).cuda()
    g.bind(x, x, dA, dy)
    g.run(K)
    ref = pkg.Gpga(n, d, pkg.GPGA_TOPO_EXP, 8, 0.1, SEED)
    ref.set_objective(pkg.GPGA_OBJ_LOGISTIC, l2=1e-4, m=m, batch=batch)
    xa = torch.from_numpy(X0).cuda()
    ref.bind(xa, torch.empty_like(xa), dA, dy)
    for k in range(K):
        ref.step(k)
    a, b = g.get_x().cpu().numpy(), ref.get_x().cpu().numpy()
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32)), float(np.abs(a - b).max())
    assert g.consensus_distance() == ref.consensus_distance()


def test_resident_run_is_cut_into_launches_of_16384_iterations():
    """A longer run takes two launches (the tags restart with each launch, its buffers are cleared
    before it); still bit-identical to single steps."""
    n, m, d, batch, K = 4, 64, 64, 8, (1 << 14) + 10
    A, y = logistic_inputs(n, m, d, SEED + 9)
    X0 = np.zeros((n, d), dtype=np.float32)
    run, stepped = _pair(n, m, d, batch, "ring", 4, X0, A, y, gamma=0.05)
    run.run(K)
    assert run.launch_count() == 2 and run.get_k() == K
    for k in range(K):
        stepped.step(k)
    a, b = run.get_x().cpu().numpy(), stepped.get_x().cpu().numpy()
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32)), float(np.abs(a - b).max())


def test_waits_between_blocks_give_up_and_report_timeout():
    """Node 0's pair of blocks launched alone with wait limits of a few thousand polls: its
    neighbours' rows never appear, so its waits run out, the error word is raised, both blocks
    of the pair leave, and the next synchronising call returns GPGA_ERR_TIMEOUT.  Nothing hangs
    or faults: the device runs the next problem as before."""
    import time
    import torch
    n, m, d, batch = 2, 64, 256, 64
    A, y = logistic_inputs(n, m, d, SEED)
    X0 = np.zeros((n, d), dtype=np.float32)
    run, stepped = _pair(n, m, d, batch, "ring", 0, X0, A, y)
    run.run(4)                                           # the kernel itself works on this problem
    for k in range(4):
        stepped.step(k)
    assert np.array_equal(run.get_x().cpu().numpy(), stepped.get_x().cpu().numpy())
    assert run.consensus_distance() >= 0.0
    t0 = time.perf_counter()
    run.selftest_run_wait()
    with pytest.raises(pkg.GpgaError) as err:
        run.consensus_distance()
    assert err.value.status == pkg.GPGA_ERR_TIMEOUT
    assert time.perf_counter() - t0 < 5.0                # milliseconds of polling, not the seconds of the defaults
    with pytest.raises(pkg.GpgaError) as err:           # sticky
        run.run(2)
    assert err.value.status == pkg.GPGA_ERR_TIMEOUT
    run.close()
    torch.cuda.synchronize()
    # a handle that the kernel does not take is turned away
    with pytest.raises(pkg.GpgaError) as err:
        stepped_exp = _pair(2, m, d, batch, "exp", 0, X0, A, y)[0]
        stepped_exp.selftest_run_wait()
    assert err.value.status == pkg.GPGA_ERR_UNSUPPORTED
    # the device is as before: a fresh pair of handles agrees again
    run2, stepped2 = _pair(n, m, d, batch, "ring", 3, X0, A, y)
    run2.run(7)
    for k in range(7):
        stepped2.step(k)
    assert np.array_equal(run2.get_x().cpu().numpy(), stepped2.get_x().cpu().numpy())
