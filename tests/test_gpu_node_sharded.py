"""Node-sharded Gossip-PGA on ONE device: the n nodes are split into shards of consecutive rows,
each shard a handle of its own; per iteration every shard exports what its neighbours need,
the messages are delivered by one device-to-device copy each, and every shard steps.  The result
must equal the unsharded run of the same problem bit for bit -- ring, every hop of the one-peer
exponential graph (hops inside a shard and hops that span shards) and the global average -- and
match the oracle within the parity tolerances."""
import numpy as np
import pytest

import paper_2105_09080_b200 as pkg
from oracle import gpga_oracle as o
from paper_2105_09080_b200 import node_sharded as ns
from paper_2105_09080_b200.inputs import quadratic_inputs
from test_gpu_parity import TOL_RUN, TOL_STEP, TOPO, close, make_quadratic

pytestmark = pytest.mark.gpu

SEED = 20210509


def _sharded_run(n, d, topo, H, gamma, sigma, X0, B, shards, K, col0=0, check_first=None, mode="whole"):
    import torch
    n_l = n // shards
    parts = []
    for s in range(shards):
        sh = ns.NodeShard(n, d, TOPO[topo][0], H, gamma, SEED, shards, s, sigma=sigma, col0=col0)
        rows = slice(s * n_l, (s + 1) * n_l)
        xa = torch.from_numpy(np.ascontiguousarray(X0[rows])).cuda()
        sh.bind(xa, torch.empty_like(xa), torch.from_numpy(np.ascontiguousarray(B[rows])).cuda())
        parts.append(sh)
    if mode == "direct":   # the send fused into the export kernel: no copy between the shards at all
        if check_first is not None:
            ns.run_local_direct(parts, 1)
            check_first(np.concatenate([sh.get_x().cpu().numpy() for sh in parts]))
            ns.run_local_direct(parts, K - 1, k0=1)
        else:
            ns.run_local_direct(parts, K)
    for k in range(K if mode != "direct" else 0):
        for sh in parts:
            sh.export(k)
        if mode == "whole":
            ns.exchange_local(parts, k)
            for sh in parts:
                sh.step(k)
        else:
            # the step in two parts; "early": the rows that need nothing received are formed BEFORE the
            # messages are delivered (they must not depend on them)
            if mode == "split":
                ns.exchange_local(parts, k)
            for sh in parts:
                sh.step_interior(k)
            if mode == "early":
                ns.exchange_local(parts, k)
            for sh in parts:
                sh.step_boundary(k)
        if check_first is not None and k == 0:
            check_first(np.concatenate([sh.get_x().cpu().numpy() for sh in parts]))
    out = np.concatenate([sh.get_x().cpu().numpy() for sh in parts])
    assert all(sh.g.get_k() == K for sh in parts)
    for sh in parts:
        sh.close()
    return out


# d = 4104: the unsharded run goes through the shared-memory tile kernel; d = 19456: through the
# row-streaming kernels; d = 1031: the scalar path (rows neither aligned nor whole groups)
@pytest.mark.parametrize("d", [4104, 19456, 1031])
@pytest.mark.parametrize("topo,H,n,shards", [("ring", 4, 16, 2), ("ring", 0, 16, 4), ("ring", 3, 8, 1), ("ring", 5, 24, 3),
                                             ("exp", 3, 16, 2), ("exp", 0, 16, 4), ("exp", 5, 32, 4), ("exp", 4, 8, 1),
                                             ("exp", 0, 8, 2)])
def test_sharded_run_is_bit_identical_to_the_unsharded_run(topo, H, n, shards, d):
    gamma, sigma, K = 0.1, 0.3, 13          # 13 iterations: every hop of the exponential graph, several global averages
    X0, B = quadratic_inputs(n, d, SEED + n + d, x0="per_node")
    g, p = make_quadratic(n, d, topo, H, gamma, SEED, sigma, X0, B)
    first = {}

    def one_step(x):
        first["x"] = x

    got = _sharded_run(n, d, topo, H, gamma, sigma, X0, B, shards, K, check_first=one_step)
    g.step(0)
    assert np.array_equal(first["x"].view(np.uint32), g.get_x().cpu().numpy().view(np.uint32))
    ok, worst = close(first["x"], o.step(p, X0, 0), TOL_STEP)
    assert ok, worst
    for k in range(1, K):
        g.step(k)
    want = g.get_x().cpu().numpy()
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), float(np.abs(got - want).max())
    ok, worst = close(got, o.run(p, X0, 0, K), TOL_RUN)
    assert ok, worst
    if H and K % H == 0:
        assert np.all(got == got[0])
    g.close()


@pytest.mark.parametrize("mode", ["split", "early"])
@pytest.mark.parametrize("topo,H,n,shards,d", [("ring", 4, 16, 2, 4104), ("ring", 0, 16, 4, 1031), ("ring", 3, 8, 1, 4104),
                                               ("ring", 5, 8, 2, 64), ("exp", 3, 16, 2, 4104), ("exp", 0, 32, 4, 1031),
                                               ("exp", 5, 8, 1, 19456), ("exp", 0, 8, 2, 64)])
def test_two_part_step_equals_the_whole_step(topo, H, n, shards, d, mode):
    """gpga_shard_step_interior + gpga_shard_step_boundary (the form that lets the exchange overlap
    the arithmetic) against the unsharded run, bit for bit; in the "early" order the interior rows are
    formed while the receive buffers still hold the previous iteration's messages."""
    gamma, sigma, K = 0.1, 0.3, 11
    X0, B = quadratic_inputs(n, d, SEED + n + d + 1, x0="per_node")
    g, _ = make_quadratic(n, d, topo, H, gamma, SEED, sigma, X0, B)
    for k in range(K):
        g.step(k)
    want = g.get_x().cpu().numpy()
    got = _sharded_run(n, d, topo, H, gamma, sigma, X0, B, shards, K, mode=mode)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), float(np.abs(got - want).max())
    g.close()


@pytest.mark.parametrize("d", [4104, 19456, 1031])
@pytest.mark.parametrize("topo,H,n,shards", [("ring", 4, 16, 2), ("ring", 0, 16, 4), ("ring", 3, 8, 1), ("ring", 5, 24, 3),
                                             ("exp", 3, 16, 2), ("exp", 0, 16, 4), ("exp", 5, 32, 4), ("exp", 4, 8, 1),
                                             ("exp", 0, 8, 2)])
def test_export_with_the_send_fused_in_is_bit_identical_to_the_unsharded_run(topo, H, n, shards, d):
    """gpga_shard_export_to: the export kernel stores every outgoing row, and the column sums of a
    global average, straight into the other shards' receive areas (two per shard, alternating with
    the parity of k); no copy is made between the shards.  Against the unsharded run bit for bit and
    against the oracle within tolerance, first iteration and whole run."""
    gamma, sigma, K = 0.1, 0.3, 13
    X0, B = quadratic_inputs(n, d, SEED + n + d + 2, x0="per_node")
    g, p = make_quadratic(n, d, topo, H, gamma, SEED, sigma, X0, B)
    first = {}
    got = _sharded_run(n, d, topo, H, gamma, sigma, X0, B, shards, K, check_first=lambda x: first.update(x=x),
                       mode="direct")
    g.step(0)
    assert np.array_equal(first["x"].view(np.uint32), g.get_x().cpu().numpy().view(np.uint32))
    ok, worst = close(first["x"], o.step(p, X0, 0), TOL_STEP)
    assert ok, worst
    for k in range(1, K):
        g.step(k)
    want = g.get_x().cpu().numpy()
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), float(np.abs(got - want).max())
    ok, worst = close(got, o.run(p, X0, 0, K), TOL_RUN)
    assert ok, worst
    g.close()


@pytest.mark.parametrize("n,shards,d", [(16, 4, 4104), (32, 2, 1031), (8, 2, 19456)])
def test_fused_export_without_a_kept_copy(n, shards, d):
    """With no keep buffer the step of a hop that exported every local row forms the half-step again
    instead of reading the exported rows: same result, bit for bit."""
    import torch
    gamma, sigma, K, H = 0.1, 0.3, 9, 0
    X0, B = quadratic_inputs(n, d, SEED + n + d + 3, x0="per_node")
    g, _ = make_quadratic(n, d, "exp", H, gamma, SEED, sigma, X0, B)
    for k in range(K):
        g.step(k)
    want = g.get_x().cpu().numpy()
    n_l, parts = n // shards, []
    for s in range(shards):
        sh = ns.NodeShard(n, d, TOPO["exp"][0], H, gamma, SEED, shards, s, sigma=sigma)
        xa = torch.from_numpy(np.ascontiguousarray(X0[s * n_l:(s + 1) * n_l])).cuda()
        sh.bind(xa, torch.empty_like(xa), torch.from_numpy(np.ascontiguousarray(B[s * n_l:(s + 1) * n_l])).cuda())
        parts.append(sh)
    ns.run_local_direct(parts, K, keep=False)
    got = np.concatenate([sh.get_x().cpu().numpy() for sh in parts])
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), float(np.abs(got - want).max())
    for sh in parts:
        sh.close()
    g.close()


@pytest.mark.parametrize("topo,n,shards,d", [("ring", 8, 2, 4096), ("exp", 16, 4, 1031), ("ring", 16, 4, 19456)])
def test_adaptive_period_on_shards_equals_the_unsharded_adaptive_run(topo, n, shards, d):
    """Gossip-AGA (Algorithm 2) on node shards -- the mean loss is the mean of the shards' mean
    losses, the period rule is the library's gpga_aga_update -- takes the period sequence of the
    unsharded gpga_run_adaptive and of the loop driven by the oracle, and ends in the same state."""
    import torch
    gamma, sigma, K, H_init, warm = 0.1, 0.05, 60, 2, 6
    X0, B = quadratic_inputs(n, d, SEED + 5, x0="shared", x0_std=3.0)
    g, p = make_quadratic(n, d, topo, 0, gamma, SEED, sigma, X0, B)
    want_periods = g.run_adaptive(K, H_init, warm)
    want = g.get_x().cpu().numpy()
    n_l, parts = n // shards, []
    for s in range(shards):
        sh = ns.NodeShard(n, d, TOPO[topo][0], 0, gamma, SEED, shards, s, sigma=sigma)
        xa = torch.from_numpy(np.ascontiguousarray(X0[s * n_l:(s + 1) * n_l])).cuda()
        sh.bind(xa, torch.empty_like(xa), torch.from_numpy(np.ascontiguousarray(B[s * n_l:(s + 1) * n_l])).cuda())
        parts.append(sh)
    periods = ns.run_local_adaptive(parts, K, H_init, warm)
    assert periods == want_periods and len(set(periods)) > 1
    got = np.concatenate([sh.get_x().cpu().numpy() for sh in parts])
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), float(np.abs(got - want).max())
    # the oracle's loop
    X, H, count, F_init, oracle_periods = X0, H_init, 0, 0.0, []
    for k in range(K):
        count += 1
        glob = count == H
        F = o.quadratic_mean_loss(X, B) if glob else 0.0
        p.H = 1 if glob else 0
        X = o.step(p, X, k)
        if glob:
            oracle_periods.append(H)
            count = 0
            F_init, H = o.aga_update(k, warm, H_init, F, F_init, H)
    assert periods == oracle_periods
    ok, worst = close(got, X, TOL_RUN)
    assert ok, worst
    for sh in parts:
        sh.close()
    g.close()


@pytest.mark.parametrize("kind", ["shared", "per_node"])
def test_seeded_fill_of_the_shards_is_the_whole_problems(kind):
    """gpga_init_from_seed on a shard handle fills local row i as node shard * n + i: the shards
    together hold bit for bit what the unsharded handle's fill holds, and a run from there agrees."""
    import torch
    n, d, shards, K = 16, 4104, 4, 6
    x0_kind = pkg.GPGA_X0_SHARED_NORMAL if kind == "shared" else pkg.GPGA_X0_PER_NODE_NORMAL
    g = pkg.Gpga(n, d, TOPO["ring"][0], 3, 0.1, SEED)
    g.set_objective(pkg.GPGA_OBJ_QUADRATIC, sigma=0.2)
    xa = torch.empty((n, d), device="cuda")
    b = torch.empty_like(xa)
    g.bind(xa, torch.empty_like(xa), b)
    g.init_from_seed(x0_kind, 0.3, 0.5)
    x0_full, b_full = g.get_x().cpu().numpy().copy(), b.cpu().numpy().copy()
    n_l, parts, bs = n // shards, [], []
    for s in range(shards):
        sh = ns.NodeShard(n, d, TOPO["ring"][0], 3, 0.1, SEED, shards, s, sigma=0.2)
        x = torch.empty((n_l, d), device="cuda")
        bb = torch.empty_like(x)
        sh.bind(x, torch.empty_like(x), bb)
        sh.init_from_seed(x0_kind, 0.3, 0.5)
        parts.append(sh)
        bs.append(bb)
    assert np.array_equal(np.concatenate([sh.get_x().cpu().numpy() for sh in parts]), x0_full)
    assert np.array_equal(np.concatenate([t.cpu().numpy() for t in bs]), b_full)
    assert len(np.unique(b_full[:, 0])) == n                          # every node has its own b
    for k in range(K):
        g.step(k)
        for sh in parts:
            sh.export(k)
        ns.exchange_local(parts, k)
        for sh in parts:
            sh.step(k)
    assert np.array_equal(np.concatenate([sh.get_x().cpu().numpy() for sh in parts]), g.get_x().cpu().numpy())
    for sh in parts:
        sh.close()
    g.close()


@pytest.mark.parametrize("topo,H,n,shards,d", [("ring", 0, 16, 4, 4104), ("exp", 5, 16, 2, 1031), ("ring", 3, 8, 1, 19456)])
def test_whole_problem_diagnostics_from_the_shards_parts(topo, H, n, shards, d):
    """Consensus distance and global loss of the whole problem, each the sum of the shards' parts
    (column sums all-gathered, mean over all nodes formed on every shard), against the oracle's values
    of the same state and against the unsharded handle's diagnostics."""
    import torch
    gamma, sigma, K = 0.1, 0.3, 7
    X0, B = quadratic_inputs(n, d, SEED + n + d + 4, x0="per_node")
    g, _ = make_quadratic(n, d, topo, H, gamma, SEED, sigma, X0, B)
    n_l, parts = n // shards, []
    for s in range(shards):
        sh = ns.NodeShard(n, d, TOPO[topo][0], H, gamma, SEED, shards, s, sigma=sigma)
        xa = torch.from_numpy(np.ascontiguousarray(X0[s * n_l:(s + 1) * n_l])).cuda()
        sh.bind(xa, torch.empty_like(xa), torch.from_numpy(np.ascontiguousarray(B[s * n_l:(s + 1) * n_l])).cuda())
        parts.append(sh)
    for k in range(K):
        g.step(k)
        for sh in parts:
            sh.export(k)
        ns.exchange_local(parts, k)
        for sh in parts:
            sh.step(k)
        if k in (0, 3, K - 1):
            X = np.concatenate([sh.get_x().cpu().numpy() for sh in parts])
            xi, loss = ns.diagnostics_local(parts)
            xi_want = o.consensus_distance(X)
            xbar = np.repeat(X.astype(np.float64).mean(0, keepdims=True), n, axis=0)
            loss_want = o.quadratic_mean_loss(xbar, B)                 # (1/n) sum_i 1/2 ||xbar - b_i||^2
            assert xi_want > 0 and abs(xi - xi_want) <= 1e-5 * xi_want, (k, xi, xi_want)
            assert abs(loss - loss_want) <= 1e-5 * loss_want, (k, loss, loss_want)
            assert abs(xi - g.consensus_distance()) <= 1e-5 * xi_want
            assert abs(loss - g.global_loss()) <= 1e-9 * loss_want
    for sh in parts:
        sh.close()
    g.close()


def test_whole_problem_diagnostics_of_logistic_shards():
    import torch
    from paper_2105_09080_b200.inputs import logistic_inputs
    topo, H, n, shards, m, d, batch, gamma, l2, K = "ring", 4, 8, 2, 64, 256, 40, 0.1, 1e-3, 6
    A, y = logistic_inputs(n, m, d, SEED + n)
    X0 = (0.1 * np.random.default_rng(n + d).standard_normal((n, d))).astype(np.float32)
    g = pkg.Gpga(n, d, TOPO[topo][0], H, gamma, SEED)
    g.set_objective(pkg.GPGA_OBJ_LOGISTIC, l2=l2, m=m, batch=batch)
    xa = torch.from_numpy(X0).cuda()
    g.bind(xa, torch.empty_like(xa), torch.from_numpy(A).cuda(), torch.from_numpy(y).cuda())
    n_l, parts = n // shards, []
    for s in range(shards):
        rows = slice(s * n_l, (s + 1) * n_l)
        sh = ns.NodeShard(n, d, TOPO[topo][0], H, gamma, SEED, shards, s, logistic=dict(l2=l2, m=m, batch=batch))
        x = torch.from_numpy(np.ascontiguousarray(X0[rows])).cuda()
        sh.bind(x, torch.empty_like(x), torch.from_numpy(np.ascontiguousarray(A[rows])).cuda(),
                torch.from_numpy(np.ascontiguousarray(y[rows])).cuda())
        parts.append(sh)
    for k in range(K):
        g.step(k)
        for sh in parts:
            sh.export(k)
        if k == 2:      # between export and step: the step forms the gradient again, the result must not change
            ns.diagnostics_local(parts, own_buffers=True)
        ns.exchange_local(parts, k)
        for sh in parts:
            sh.step(k)
        X = np.concatenate([sh.get_x().cpu().numpy() for sh in parts])
        assert np.array_equal(X.view(np.uint32), g.get_x().cpu().numpy().view(np.uint32))
        xi, loss = ns.diagnostics_local(parts)
        xi_want = o.consensus_distance(X)
        loss_want = o.global_logistic_loss(A.astype(np.float64), y.astype(np.float64), X.astype(np.float64).mean(0), l2)
        if (k + 1) % H:
            assert xi_want > 0 and abs(xi - xi_want) <= 1e-5 * xi_want, (k, xi, xi_want)
        else:
            assert xi <= 1e-12
        assert abs(loss - loss_want) <= 1e-5 * loss_want, (k, loss, loss_want)
        assert abs(loss - g.global_loss()) <= 1e-6 * loss_want
    for sh in parts:
        sh.close()
    g.close()


def test_fused_export_argument_checks():
    import ctypes as C
    import torch
    L = pkg.lib()
    n, d, shards = 8, 64, 2
    sh = ns.NodeShard(n, d, TOPO["ring"][0], 4, 0.1, SEED, shards, 0)
    X0, B = quadratic_inputs(n // shards, d, 3, x0="per_node")
    xa = torch.from_numpy(X0).cuda()
    sh.bind(xa, torch.empty_like(xa), torch.from_numpy(B).cuda())
    good = sh.recv.data_ptr()
    two = (C.c_void_p * 2)(good, good + 512)
    one = (C.c_void_p * 1)(good)
    odd = (C.c_void_p * 2)(good, good + 4)
    null = (C.c_void_p * 2)(good, None)
    h = sh.g._h
    assert L.gpga_shard_export_to(h, 0, None, one, 1, None) == pkg.GPGA_ERR_INVALID_ARG      # the ring sends two messages
    assert L.gpga_shard_export_to(h, 0, None, odd, 2, None) == pkg.GPGA_ERR_INVALID_ARG      # misaligned destination
    assert L.gpga_shard_export_to(h, 0, None, null, 2, None) == pkg.GPGA_ERR_INVALID_ARG     # NULL destination
    assert L.gpga_shard_export_to(h, 0, None, None, 2, None) == pkg.GPGA_ERR_INVALID_ARG
    assert L.gpga_shard_export_to(h, 3, None, one, 1, None) == pkg.GPGA_ERR_INVALID_ARG      # k = 3, H = 4: one slot per shard
    assert L.gpga_shard_export_to(h, 0, None, two, 2, None) == pkg.GPGA_OK
    assert L.gpga_shard_export_to(h, 3, None, two, 2, None) == pkg.GPGA_OK
    torch.cuda.synchronize()
    sh.close()


def test_sharded_run_with_a_column_offset_and_no_noise():
    n, d, shards, K = 16, 2052, 4, 6
    X0, B = quadratic_inputs(n, d, 5, x0="per_node")
    for sigma, col0 in ((0.0, 0), (0.2, 8192)):
        g, _ = make_quadratic(n, d, "exp", 3, 0.05, SEED, sigma, X0, B, col0=col0)
        g.run(K)
        got = _sharded_run(n, d, "exp", 3, 0.05, sigma, X0, B, shards, K, col0=col0)
        assert np.array_equal(got, g.get_x().cpu().numpy())
        g.close()


def test_plan_and_argument_checks():
    L = pkg.lib()
    # two shards of 8 nodes, 16-node exponential graph: hops 1, 2, 4 stay next door, hop 8 is one shard ahead
    for k, hop, rows in ((0, 1, 1), (1, 2, 2), (2, 4, 4), (3, 8, 8), (4, 1, 1)):
        plan = ns.shard_plan(pkg.GPGA_TOPO_EXP, 0, 16, 2, 0, 40, k)
        assert (plan.kind, plan.hop, plan.messages) == (ns.GPGA_SHARD_EXP, hop, 1)
        assert plan.bytes[0] == rows * 40 * 4 and plan.send_to[0] == 1 and plan.recv_from[0] == 1
    # eight shards of 4 nodes, 32 nodes: hop 16 is four shards ahead, hop 2 is the next shard
    plan = ns.shard_plan(pkg.GPGA_TOPO_EXP, 0, 32, 8, 1, 8, 4)
    assert plan.hop == 16 and plan.recv_from[0] == 5 and plan.send_to[0] == 5 and plan.bytes[0] == 4 * 8 * 4
    plan = ns.shard_plan(pkg.GPGA_TOPO_EXP, 0, 32, 8, 1, 8, 1)
    assert plan.hop == 2 and plan.recv_from[0] == 2 and plan.send_to[0] == 0 and plan.bytes[0] == 2 * 8 * 4
    # ring: first row up, last row down; d = 10 travels as 12 floats
    plan = ns.shard_plan(pkg.GPGA_TOPO_RING, 4, 12, 3, 0, 10, 0)
    assert (plan.kind, plan.messages) == (ns.GPGA_SHARD_RING, 2)
    assert list(plan.send_to) == [2, 1] and list(plan.recv_from) == [2, 1]
    assert list(plan.bytes) == [48, 48] and list(plan.send_offset) == [0, 48] and list(plan.dst_offset) == [48, 0]
    plan = ns.shard_plan(pkg.GPGA_TOPO_RING, 4, 12, 3, 0, 10, 3)          # mod(k + 1, H) = 0
    assert plan.kind == ns.GPGA_SHARD_GLOBAL and plan.messages == 0 and plan.gather_bytes == 12 * 8
    with pytest.raises(pkg.GpgaError):
        ns.shard_plan(pkg.GPGA_TOPO_EXP, 0, 16, 3, 0, 8, 0)               # 3 shards of a 16-node exponential graph
    with pytest.raises(pkg.GpgaError):
        ns.shard_plan(pkg.GPGA_TOPO_GRID, 0, 16, 2, 0, 8, 0)
    # a shard of several holds a multiple of four nodes
    with pytest.raises(pkg.GpgaError) as err:
        ns.NodeShard(12, 64, pkg.GPGA_TOPO_RING, 4, 0.1, 1, 2, 0)
    assert err.value.status == pkg.GPGA_ERR_UNSUPPORTED
    # the two-part step needs the double buffer
    import torch
    sh = ns.NodeShard(8, 64, pkg.GPGA_TOPO_RING, 4, 0.1, 1, 2, 0)
    x = torch.zeros((4, 64), device="cuda")
    sh.bind(x, x, torch.zeros((4, 64), device="cuda"))
    sh.export(0)
    with pytest.raises(pkg.GpgaError) as err:
        sh.step_interior(0)
    assert err.value.status == pkg.GPGA_ERR_UNSUPPORTED
    sh.step(0)                                              # the whole step works in place
    sh.close()


@pytest.mark.parametrize("topo,H,n,shards,m,d,batch", [("ring", 4, 8, 2, 64, 256, 40), ("exp", 3, 16, 4, 32, 1024, 128),
                                                         ("ring", 0, 12, 3, 40, 2052, 33), ("exp", 0, 8, 2, 24, 64, 8),
                                                         ("ring", 3, 8, 1, 64, 256, 40)])
def test_logistic_objective_sharded_by_nodes(topo, H, n, shards, m, d, batch):
    """The logistic workload split by nodes (every shard binds its own nodes' samples and labels;
    mini-batch draws keyed by the global node index): bit-identical to the unsharded steps, and within
    tolerance of the oracle."""
    import torch
    from paper_2105_09080_b200.inputs import logistic_inputs
    gamma, l2, K = 0.1, 1e-4, 9
    A, y = logistic_inputs(n, m, d, SEED + n)
    rng = np.random.default_rng(n + d)
    X0 = (0.1 * rng.standard_normal((n, d))).astype(np.float32)
    g = pkg.Gpga(n, d, TOPO[topo][0], H, gamma, SEED)
    g.set_objective(pkg.GPGA_OBJ_LOGISTIC, l2=l2, m=m, batch=batch)
    xa = torch.from_numpy(X0).cuda()
    g.bind(xa, torch.empty_like(xa), torch.from_numpy(A).cuda(), torch.from_numpy(y).cuda())
    for k in range(K):
        g.step(k)
    want = g.get_x().cpu().numpy()
    n_l = n // shards
    parts = []
    for s in range(shards):
        rows = slice(s * n_l, (s + 1) * n_l)
        sh = ns.NodeShard(n, d, TOPO[topo][0], H, gamma, SEED, shards, s, logistic=dict(l2=l2, m=m, batch=batch))
        x = torch.from_numpy(np.ascontiguousarray(X0[rows])).cuda()
        sh.bind(x, torch.empty_like(x), torch.from_numpy(np.ascontiguousarray(A[rows])).cuda(),
                torch.from_numpy(np.ascontiguousarray(y[rows])).cuda())
        parts.append(sh)
    for k in range(K):
        for sh in parts:
            sh.export(k)
        ns.exchange_local(parts, k)
        for sh in parts:
            if k % 2:
                sh.step(k)
            else:                       # the two-part form as well
                sh.step_interior(k)
                sh.step_boundary(k)
    got = np.concatenate([sh.get_x().cpu().numpy() for sh in parts])
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), float(np.abs(got - want).max())
    p = o.Problem(TOPO[topo][1], H, gamma, SEED, objective="logistic", data=A.astype(np.float64),
                  labels=y.astype(np.float64), l2=l2, batch=batch)
    ok, worst = close(got, o.run(p, X0, 0, K), TOL_RUN)
    assert ok, worst
    # K more iterations with the send fused into the export kernel, against K more single steps
    ns.run_local_direct(parts, K, k0=K)
    for k in range(K, 2 * K):
        g.step(k)
    got, want = np.concatenate([sh.get_x().cpu().numpy() for sh in parts]), g.get_x().cpu().numpy()
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), float(np.abs(got - want).max())
    for sh in parts:
        sh.close()
    g.close()
