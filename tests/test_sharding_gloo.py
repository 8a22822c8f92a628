"""Column sharding over ranks, world_size 2, gloo on CPU.  The compute on each rank is the
oracle (no GPU here); what is under test is the shard arithmetic and the scalar reduction."""
import os
import socket

import numpy as np
import pytest

from paper_2105_09080_b200 import sharding


def test_split_columns_covers_range_with_aligned_starts():
    for d, w in ((40, 2), (41, 2), (7, 4), (25_557_032, 8), (3, 2), (1024, 3)):
        parts = sharding.split_columns(d, w)
        assert len(parts) == w
        assert parts[0][0] == 0 and sum(p[1] for p in parts) == d
        for (c0, width), nxt in zip(parts, parts[1:] + [(d, 0)]):
            assert c0 % 4 == 0 or width == 0
            assert c0 + width == nxt[0] or nxt[1] == 0
    assert sharding.weak_shard_offset(3, 25_557_032) == 3 * 25_557_032
    assert sharding.weak_shard_offset(2, 1031) == 2 * 1032


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, n, d_total, K, out_dir):
    import torch
    import torch.distributed as dist
    from oracle import gpga_oracle as o
    from paper_2105_09080_b200.inputs import quadratic_inputs
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    X0, B = quadratic_inputs(n, d_total, 7)
    c0, width = sharding.split_columns(d_total, world)[rank]
    p = o.Problem(o.TOPO_EXP, 3, 0.1, 11, sigma=0.4, data=B[:, c0:c0 + width], col0=c0)
    X = o.run(p, X0[:, c0:c0 + width], 0, K)
    xi = sharding.all_reduce_sum(o.consensus_distance(X))
    gathered = [None] * world
    dist.all_gather_object(gathered, (c0, X))
    if rank == 0:
        full = np.concatenate([x for _, x in sorted(gathered, key=lambda t: t[0])], axis=1)
        np.save(os.path.join(out_dir, "full.npy"), full)
        np.save(os.path.join(out_dir, "xi.npy"), np.array([xi]))
    dist.barrier()
    dist.destroy_process_group()


def test_sharded_run_equals_unsharded_run(tmp_path):
    import torch.multiprocessing as mp
    from oracle import gpga_oracle as o
    from paper_2105_09080_b200.inputs import quadratic_inputs
    n, d_total, K, world = 8, 78, 7, 2
    mp.spawn(_worker, args=(world, _free_port(), n, d_total, K, str(tmp_path)), nprocs=world, join=True)
    X0, B = quadratic_inputs(n, d_total, 7)
    want = o.run(o.Problem(o.TOPO_EXP, 3, 0.1, 11, sigma=0.4, data=B), X0, 0, K)
    got = np.load(tmp_path / "full.npy")
    assert np.array_equal(got, want)
    xi = float(np.load(tmp_path / "xi.npy")[0])
    assert abs(xi - o.consensus_distance(want)) <= 1e-12 * xi


def test_convex_experiment_inputs_follow_the_recipe():
    from paper_2105_09080_b200.inputs import convex_experiment_inputs
    A, y = convex_experiment_inputs(6, 2000, 10, seed=1)
    assert A.shape == (6, 2000, 12) and not A[:, :, 10:].any()           # zero padding to a multiple of 4
    assert abs(A[:, :, :10].std() - np.sqrt(10)) < 0.05
    assert set(np.unique(y)) == {-1.0, 1.0}
    A2, y2 = convex_experiment_inputs(6, 2000, 10, seed=1, iid=True)
    assert A2.shape == A.shape and abs(y2.mean()) < 0.1
