"""The exchange schedule of node-sharded Gossip-PGA over ranks: world_size 2 (and 4), gloo on CPU.
Each rank holds a shard of consecutive nodes and computes with the oracle; what is under test is
the plan (who sends which rows to whom at which iteration: the ring's two neighbours, the partner
shard of every hop of the one-peer exponential graph, the all-gather of the global average) and
the torch.distributed delivery of the messages.  A wrong neighbour, offset or hop changes the
result by O(1); the comparison with the unsharded oracle run allows only the fp32 rounding of the
exchanged rows."""
import os
import socket

import numpy as np
import pytest

import paper_2105_09080_b200 as pkg
from oracle import gpga_oracle as o
from paper_2105_09080_b200 import node_sharded as ns
from paper_2105_09080_b200.inputs import quadratic_inputs

TOPOLOGY = {"ring": (pkg.GPGA_TOPO_RING, o.TOPO_RING), "exp": (pkg.GPGA_TOPO_EXP, o.TOPO_EXP)}


class OracleShard:
    """A shard whose arithmetic is the oracle's: exported rows are the fp64 half-step rounded to the
    fp32 the messages carry; the mix uses the received rows where the neighbour is not local."""

    def __init__(self, n_total, d, topo, H, gamma, sigma, seed, shards, shard, X0, B):
        import torch
        self.n_total, self.d, self.topology, self.H = n_total, d, TOPOLOGY[topo][0], H
        self.topo, self.gamma, self.sigma, self.seed = topo, gamma, sigma, seed
        self.shards, self.shard, self.n = shards, shard, n_total // shards
        rows = slice(shard * self.n, (shard + 1) * self.n)
        self.X, self.B = X0[rows].astype(np.float32), B[rows].astype(np.float64)
        self.q4 = (d + 3) // 4 * 4
        nbytes = max(max(self.n, 2) * self.q4 * 4, shards * self.q4 * 8)
        self.send = torch.zeros(nbytes, dtype=torch.uint8)
        self.recv = torch.zeros(nbytes, dtype=torch.uint8)

    def plan(self, k):
        return ns.shard_plan(self.topology, self.H, self.n_total, self.shards, self.shard, self.d, k)

    def set_period(self, H):
        self.H = H

    def state_sums(self, out=None):
        sums = np.zeros(self.q4)
        sums[:self.d] = self.X.astype(np.float64).sum(0)
        (self.send if out is None else out)[:self.q4 * 8] = _bytes(sums)

    def diagnostics(self, gathered=None):
        buf = (self.recv if gathered is None else gathered).numpy()[:self.shards * self.q4 * 8]
        total = np.frombuffer(buf.tobytes(), dtype=np.float64).reshape(self.shards, self.q4).sum(0)[:self.d]
        xbar = total / self.n_total
        X = self.X.astype(np.float64)
        return float(((X - xbar) ** 2).sum()), float(0.5 * ((xbar - self.B) ** 2).sum() / self.n_total)

    def mean_loss(self):
        return o.quadratic_mean_loss(self.X, self.B)

    def _half_step(self, k):
        """fp64 half-step of the local rows: the rows sit at their global positions of a full-height
        matrix so that the oracle keys the noise by the global node index."""
        full_x = np.zeros((self.n_total, self.d))
        full_b = np.zeros((self.n_total, self.d))
        rows = slice(self.shard * self.n, (self.shard + 1) * self.n)
        full_x[rows], full_b[rows] = self.X, self.B
        return o.quadratic_half_step(full_x, full_b, self.gamma, self.sigma, self.seed, k)[rows]

    def export(self, k):
        plan, Y = self.plan(k), self._half_step(k)
        self.Y = Y
        if plan.kind == ns.GPGA_SHARD_GLOBAL:
            sums = np.zeros(self.q4)
            sums[:self.d] = Y.sum(0)
            self.send[:self.q4 * 8] = _bytes(sums)
            return
        if plan.kind == ns.GPGA_SHARD_RING:
            out = Y[[0, self.n - 1]]
        else:
            out = Y[:min(plan.hop, self.n)]
        msg = np.zeros((out.shape[0], self.q4), dtype=np.float32)
        msg[:, :self.d] = out
        self.send[:msg.nbytes] = _bytes(msg)

    def step(self, k):
        plan, Y, n, d = self.plan(k), self.Y, self.n, self.d
        if plan.kind == ns.GPGA_SHARD_GLOBAL:
            parts = np.frombuffer(self.recv.numpy()[:self.shards * self.q4 * 8].tobytes(), dtype=np.float64)
            total = parts.reshape(self.shards, self.q4).sum(0)[:d]
            Z = np.repeat((total / self.n_total)[None, :], n, axis=0)
        else:
            rows = 2 if plan.kind == ns.GPGA_SHARD_RING else min(plan.hop, n)
            got = np.frombuffer(self.recv.numpy()[:rows * self.q4 * 4].tobytes(), dtype=np.float32)
            got = got.reshape(rows, self.q4)[:, :d].astype(np.float64)
            if plan.kind == ns.GPGA_SHARD_RING:
                ext = np.concatenate([got[:1], Y, got[1:]])          # row above, local rows, row below
                Z = (ext[:-2] + ext[1:-1] + ext[2:]) / 3.0
            else:
                he = rows
                partner = np.concatenate([Y[he:], got]) if he < n else got
                Z = (Y + partner) / 2.0
        self.X = Z.astype(np.float32)


def _bytes(a):
    import torch
    return torch.frombuffer(bytearray(np.ascontiguousarray(a).tobytes()), dtype=torch.uint8)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _oracle_adaptive(topo, n, d, K, H_init, warm, gamma, sigma, seed, X0, B):
    """Algorithm 2 driven by the oracle on the unsharded problem: (periods, X^(K))."""
    p = o.Problem(TOPOLOGY[topo][1], 0, gamma, seed, sigma=sigma, data=B)
    X, H, count, F_init, periods = X0, H_init, 0, 0.0, []
    for k in range(K):
        count += 1
        glob = count == H
        F = o.quadratic_mean_loss(X, B) if glob else 0.0
        p.H = 1 if glob else 0
        X = o.step(p, X, k)
        if glob:
            periods.append(H)
            count = 0
            F_init, H = o.aga_update(k, warm, H_init, F, F_init, H)
    return periods, X


def _adaptive_worker(rank, world, port, topo, n, d, K, H_init, warm, out_dir):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    X0, B = quadratic_inputs(n, d, 7, x0="shared", x0_std=3.0)
    shard = OracleShard(n, d, topo, 0, 0.1, 0.05, 11, world, rank, X0, B)
    periods = ns.run_dist_adaptive(shard, K, H_init, warm)
    gathered = [None] * world
    dist.all_gather_object(gathered, (rank, shard.X, periods))
    if rank == 0:
        assert all(g[2] == periods for g in gathered)       # every rank took the same periods
        np.save(os.path.join(out_dir, "full.npy"), np.concatenate([x for _, x, _ in sorted(gathered, key=lambda t: t[0])]))
        np.save(os.path.join(out_dir, "periods.npy"), np.array(periods, dtype=np.int64))
    dist.barrier()
    dist.destroy_process_group()


def _diag_worker(rank, world, port, n, d, K, out_dir):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    X0, B = quadratic_inputs(n, d, 7, x0="per_node")
    shard = OracleShard(n, d, "ring", 0, 0.1, 0.4, 11, world, rank, X0, B)
    ns.run_dist(shard, K)
    xi, loss = ns.diagnostics_dist(shard)
    gathered = [None] * world
    dist.all_gather_object(gathered, (rank, shard.X, xi, loss))
    if rank == 0:
        assert all(g[2] == xi and g[3] == loss for g in gathered)     # every rank holds the same totals
        np.save(os.path.join(out_dir, "full.npy"), np.concatenate([x for _, x, _, _ in sorted(gathered, key=lambda t: t[0])]))
        np.save(os.path.join(out_dir, "diag.npy"), np.array([xi, loss]))
    dist.barrier()
    dist.destroy_process_group()


def _worker(rank, world, port, topo, H, n, d, K, out_dir, tags=True):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    X0, B = quadratic_inputs(n, d, 7, x0="per_node")
    shard = OracleShard(n, d, topo, H, 0.1, 0.4, 11, world, rank, X0, B)
    ns.run_dist(shard, K, tags=tags)
    gathered = [None] * world
    dist.all_gather_object(gathered, (rank, shard.X))
    if rank == 0:
        np.save(os.path.join(out_dir, "full.npy"), np.concatenate([x for _, x in sorted(gathered, key=lambda t: t[0])]))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("topo,H,n,world", [("ring", 4, 8, 2), ("exp", 3, 16, 2), ("exp", 0, 16, 4), ("ring", 0, 12, 3)])
def test_ranks_exchange_the_right_rows(tmp_path, topo, H, n, world):
    import torch.multiprocessing as mp
    d, K = 10, 9
    mp.spawn(_worker, args=(world, _free_port(), topo, H, n, d, K, str(tmp_path)), nprocs=world, join=True)
    X0, B = quadratic_inputs(n, d, 7, x0="per_node")
    want = o.run(o.Problem(TOPOLOGY[topo][1], H, 0.1, 11, sigma=0.4, data=B), X0, 0, K)
    got = np.load(tmp_path / "full.npy")
    assert got.shape == want.shape
    # the exchanged half-step rows travel as fp32: a relative 6e-8 per exchanged row and iteration
    assert np.abs(got - want).max() <= 2e-6 * (1 + np.abs(want).max())


def test_two_shard_ring_without_tags(tmp_path):
    """Both neighbours of a shard are the same rank in a ring of two shards; a backend without message
    tags pairs sends and receives by posting order alone.  With every tag forced to 0 the run must
    still be right."""
    import torch.multiprocessing as mp
    n, d, K, world = 8, 10, 7, 2
    mp.spawn(_worker, args=(world, _free_port(), "ring", 3, n, d, K, str(tmp_path), False), nprocs=world, join=True)
    X0, B = quadratic_inputs(n, d, 7, x0="per_node")
    want = o.run(o.Problem(o.TOPO_RING, 3, 0.1, 11, sigma=0.4, data=B), X0, 0, K)
    got = np.load(tmp_path / "full.npy")
    assert np.abs(got - want).max() <= 2e-6 * (1 + np.abs(want).max())


def test_one_process_delivery_matches_the_plan():
    """exchange_local with four oracle shards in this process, ring and exponential graph."""
    n, d, K, shards = 16, 6, 7, 4
    X0, B = quadratic_inputs(n, d, 3, x0="per_node")
    for topo, H in (("ring", 3), ("exp", 0), ("exp", 4)):
        parts = [OracleShard(n, d, topo, H, 0.2, 0.1, 5, shards, s, X0, B) for s in range(shards)]
        for k in range(K):
            for sh in parts:
                sh.export(k)
            ns.exchange_local(parts, k)
            for sh in parts:
                sh.step(k)
        got = np.concatenate([sh.X for sh in parts])
        want = o.run(o.Problem(TOPOLOGY[topo][1], H, 0.2, 5, sigma=0.1, data=B), X0, 0, K)
        assert np.abs(got - want).max() <= 2e-6 * (1 + np.abs(want).max()), (topo, H)


def test_plan_is_consistent_for_every_shape():
    """Host logic only, exhaustively over small shapes: every message a shard sends is one its
    destination expects (same size, landing where the destination reads it), and the rows a shard
    receives are the rows its local nodes' neighbours live in."""
    row = lambda d: (d + 3) // 4 * 16
    for d in (8, 10):
        for n in (4, 8, 16, 32, 64):
            for shards in (1, 2, 4, 8, 16):
                if n % shards or (n // shards) % 4 and shards > 1:
                    continue
                n_l = n // shards
                for k in range(0, 14):
                    plans = [ns.shard_plan(pkg.GPGA_TOPO_EXP, 0, n, shards, g, d, k) for g in range(shards)]
                    hop = plans[0].hop
                    assert hop == 1 << (k % max(1, n.bit_length() - 1))
                    he = min(hop, n_l)
                    for g, p in enumerate(plans):
                        assert (p.kind, p.messages, p.bytes[0]) == (ns.GPGA_SHARD_EXP, 1, he * row(d))
                        src = p.recv_from[0]
                        assert plans[src].send_to[0] == g and plans[src].bytes[0] == p.bytes[0]
                        # local node i = n_l - he + c (the last he rows) has its partner (i + hop) mod n at row c of `src`
                        for c in range(he):
                            partner = (g * n_l + n_l - he + c + hop) % n
                            assert partner == src * n_l + c, (n, shards, k, g, c)
                        # and every other local node's partner is local
                        for i in range(n_l - he):
                            assert g * n_l <= (g * n_l + i + hop) % n < (g + 1) * n_l
        for n, shards in ((8, 1), (8, 2), (12, 3), (64, 4), (64, 16), (20, 5)):
            n_l = n // shards
            plans = [ns.shard_plan(pkg.GPGA_TOPO_RING, 4, n, shards, g, d, 0) for g in range(shards)]
            for g, p in enumerate(plans):
                assert (p.kind, p.messages) == (ns.GPGA_SHARD_RING, 2)
                assert p.recv_from[0] == (g - 1) % shards and p.recv_from[1] == (g + 1) % shards
                for m in (0, 1):
                    dst = plans[p.send_to[m]]
                    assert dst.recv_from[1 - m] == g                      # my first row is my upper neighbour's "row below"
                    assert p.dst_offset[m] == dst.recv_offset[1 - m] and p.bytes[m] == row(d)
                # the row above local row 0 is the last row of shard g-1; the row below the last is row 0 of shard g+1
                assert (g * n_l - 1) % n == ((g - 1) % shards) * n_l + n_l - 1
                assert ((g + 1) * n_l) % n == ((g + 1) % shards) * n_l
            glob = ns.shard_plan(pkg.GPGA_TOPO_RING, 4, n, shards, 0, d, 3)
            assert glob.kind == ns.GPGA_SHARD_GLOBAL and glob.gather_bytes == (d + 3) // 4 * 4 * 8


def test_direct_destinations_land_where_the_copies_land():
    """Host logic of the fused export (the kernel stores its messages straight into the receivers'
    areas): in a flat fake address space, writing every shard's send buffer to the addresses
    direct_destinations gives must leave every receive area exactly as exchange_local's copies do --
    ring, every hop of the exponential graph, the all-gather of a global average."""
    import torch
    d = 10
    for topo, H, n, shards in (("ring", 4, 16, 4), ("ring", 0, 8, 2), ("ring", 3, 4, 1), ("exp", 3, 16, 2), ("exp", 0, 32, 8),
                               ("exp", 5, 16, 4), ("exp", 2, 4, 1)):
        rng = np.random.default_rng(n + shards)
        X0, B = quadratic_inputs(n, d, 3, x0="per_node")
        parts = [OracleShard(n, d, topo, H, 0.2, 0.1, 5, shards, s, X0, B) for s in range(shards)]
        area = parts[0].recv.numel()
        for k in range(12):
            for sh in parts:   # messages with contents that identify (shard, k, byte)
                sh.send[:] = torch.from_numpy(rng.integers(0, 256, area, dtype=np.uint8))
                sh.recv[:] = 0
            ns.exchange_local(parts, k)
            memory = np.zeros(shards * area, dtype=np.uint8)
            for sh in parts:
                plan = sh.plan(k)
                dests = ns.direct_destinations(plan, sh.shard, shards, lambda s: s * area)
                if plan.kind == ns.GPGA_SHARD_GLOBAL:
                    assert len(dests) == shards
                    for a in dests:
                        memory[a:a + plan.gather_bytes] = sh.send.numpy()[:plan.gather_bytes]
                else:
                    assert len(dests) == plan.messages
                    for m, a in enumerate(dests):
                        lo, nb = plan.send_offset[m], plan.bytes[m]
                        assert a % 16 == 0 and a // area == plan.send_to[m] and a % area + nb <= area
                        memory[a:a + nb] = sh.send.numpy()[lo:lo + nb]
            for s, sh in enumerate(parts):
                assert np.array_equal(memory[s * area:(s + 1) * area], sh.recv.numpy()), (topo, H, n, shards, k, s)


def test_library_period_rule_equals_the_oracles():
    """gpga_aga_update (host arithmetic of the library) against the oracle's Algorithm 2 rule wherever
    the rule is defined (F > 0, F_init > 0); the library's guards for the degenerate cases apart."""
    rng = np.random.default_rng(4)
    for _ in range(2000):
        k, warm, H_init = int(rng.integers(0, 50)), int(rng.integers(0, 30)), int(rng.integers(1, 9))
        F = float(rng.choice([1e-9, rng.uniform(1e-3, 10.0)]))
        F_init, H = float(rng.uniform(1e-3, 10.0)), int(rng.integers(1, 40))
        assert ns.aga_update(k, warm, H_init, F, F_init, H) == o.aga_update(k, warm, H_init, F, F_init, H)
    assert ns.aga_update(9, 5, 4, 0.0, 2.0, 7) == (2.0, 7)         # F = 0: the ratio is undefined, the period stays
    assert ns.aga_update(9, 5, 4, 1.0, 0.0, 7) == (0.0, 1)         # ceil(0) = 0: a period is at least 1
    assert ns.aga_update(9, 5, 4, 1e-9, 1e10, 7)[1] == int(9.0e15)       # beyond int64: clamped
    assert ns.aga_update(9, 5, 4, 1e-300, 1e300, 7)[1] == 7            # an infinite ratio: the period stays
    assert pkg.lib().gpga_aga_update(0, 0, 0, 1.0, None, None) == pkg.GPGA_ERR_INVALID_ARG


@pytest.mark.parametrize("topo,n,shards", [("ring", 16, 4), ("exp", 16, 2), ("ring", 8, 1)])
def test_adaptive_period_on_shards_of_one_process(topo, n, shards):
    """Gossip-AGA on node shards (the mean loss is the mean of the shards' mean losses): the period
    sequence and the final state equal those of Algorithm 2 driven by the oracle on the whole problem."""
    d, K, H_init, warm = 12, 60, 2, 6
    X0, B = quadratic_inputs(n, d, 7, x0="shared", x0_std=3.0)
    parts = [OracleShard(n, d, topo, 0, 0.1, 0.05, 11, shards, s, X0, B) for s in range(shards)]
    periods = ns.run_local_adaptive(parts, K, H_init, warm)
    want_periods, want = _oracle_adaptive(topo, n, d, K, H_init, warm, 0.1, 0.05, 11, X0, B)
    assert periods == want_periods and len(set(periods)) > 1 and periods[-1] > periods[0]
    got = np.concatenate([sh.X for sh in parts])
    assert np.abs(got - want).max() <= 2e-6 * (1 + np.abs(want).max())


def test_adaptive_period_across_ranks(tmp_path):
    """The same with one shard per gloo rank: the loss is all-reduced, every rank takes the same periods."""
    import torch.multiprocessing as mp
    topo, n, d, K, H_init, warm, world = "ring", 8, 12, 40, 2, 6, 2
    mp.spawn(_adaptive_worker, args=(world, _free_port(), topo, n, d, K, H_init, warm, str(tmp_path)), nprocs=world, join=True)
    X0, B = quadratic_inputs(n, d, 7, x0="shared", x0_std=3.0)
    want_periods, want = _oracle_adaptive(topo, n, d, K, H_init, warm, 0.1, 0.05, 11, X0, B)
    assert np.load(tmp_path / "periods.npy").tolist() == want_periods
    got = np.load(tmp_path / "full.npy")
    assert np.abs(got - want).max() <= 2e-6 * (1 + np.abs(want).max())


def test_whole_problem_diagnostics_across_ranks(tmp_path):
    """diagnostics_dist: column sums all-gathered in rank order, the two parts all-reduced; against the
    oracle's consensus distance and global loss of the assembled state."""
    import torch.multiprocessing as mp
    n, d, K, world = 12, 10, 5, 3
    mp.spawn(_diag_worker, args=(world, _free_port(), n, d, K, str(tmp_path)), nprocs=world, join=True)
    X = np.load(tmp_path / "full.npy")
    xi, loss = np.load(tmp_path / "diag.npy")
    _, B = quadratic_inputs(n, d, 7, x0="per_node")
    xi_want = o.consensus_distance(X)
    xbar = np.repeat(X.astype(np.float64).mean(0, keepdims=True), n, axis=0)
    assert xi_want > 0 and abs(xi - xi_want) <= 1e-9 * xi_want
    assert abs(loss - o.quadratic_mean_loss(xbar, B)) <= 1e-9 * loss
