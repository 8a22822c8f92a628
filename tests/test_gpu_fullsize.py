"""Full-size configurations (ResNet-50- and BERT-Large-sized parameter counts) in the
launch configuration the benchmark times, checked on sampled column blocks.

Under the quadratic objective W acts on rows only and the gradient and noise are
element-wise, so every column evolves independently: the oracle run on a block of columns
(keyed by the block's global column offset) gives exactly the values a full run would.
Both sides fill b and X0 from the seed by their own implementation of the same streams;
nothing computed on the GPU is fed to the oracle."""
import numpy as np
import pytest

import paper_2105_09080_b200 as pkg
from oracle import gpga_oracle as o
from test_gpu_parity import TOL_RUN, TOL_STEP, TOPO, close

pytestmark = pytest.mark.gpu

SEED = 20210509
BLOCK = 1024            # columns per sampled block = columns per 256-thread CTA


def _torch():
    import torch
    return torch


def _blocks(d, count, rng):
    """Column offsets (multiples of 4): first block, last (ragged end), blocks straddling
    CTA boundaries, and random ones."""
    offs = {0, (d - BLOCK) // 4 * 4, BLOCK // 2, 148 * BLOCK - 512, (d // 2) // BLOCK * BLOCK + 508}
    while len(offs) < count:
        offs.add(int(rng.integers(0, (d - BLOCK) // 4)) * 4)
    return sorted(offs)


def _gpu_block(x, c0, width):
    return x[:, c0:c0 + width].cpu().numpy()


def _free_gib():
    torch = _torch()
    free, _ = torch.cuda.mem_get_info()
    return free / 2**30


def _oracle_xi_of_device_state(x, d, chunk=1 << 20):
    """Consensus distance of the state the GPU holds, recomputed by the oracle: X is downloaded in
    column chunks and the oracle's value of every chunk is added up (the distance
    sum_j sum_i (x_ij - xbar_j)^2 of Section 4 is a sum over columns)."""
    total = 0.0
    for c0 in range(0, d, chunk):
        total += o.consensus_distance(x[:, c0:min(d, c0 + chunk)].cpu().numpy())
    return total


def _run_case(bufs, n, d, topo, H, gamma, sigma, K, x0_kind, x0_std, b_shift, offs, one_step_ks, ld=None,
              check_xi=False, stepped=False):
    xa, xb, b, scratch = bufs
    ld = ld or d
    xa, xb, b = (t.view(-1)[:n * ld].view(n, ld) for t in (xa, xb, b))
    okind = {pkg.GPGA_X0_ZERO: o.X0_ZERO, pkg.GPGA_X0_SHARED_NORMAL: o.X0_SHARED_NORMAL}[x0_kind]
    g = pkg.Gpga(n, d, TOPO[topo][0], H, gamma, SEED)
    g.set_objective(pkg.GPGA_OBJ_QUADRATIC, sigma=sigma)
    g.set_row_stride(ld)
    g.bind(xa, xb, b, scratch=scratch)
    width = lambda c0: min(BLOCK, d - c0)
    ora = {}
    for c0 in offs:
        w = width(c0)
        B = o.init_b(n, w, SEED, b_shift, c0).astype(np.float32)
        X0 = o.init_x0(n, w, SEED, okind, x0_std, c0).astype(np.float32)
        ora[c0] = (X0, o.Problem(TOPO[topo][1], H, gamma, SEED, sigma=sigma, data=B, col0=c0))
    # single iterations at chosen k, each from the initial state
    for k in one_step_ks:
        g.init_from_seed(x0_kind, x0_std, b_shift)
        g.step(k)
        x = g.get_x()
        for c0 in offs:
            X0, p = ora[c0]
            ok, worst = close(_gpu_block(x, c0, width(c0)), o.step(p, X0, k), TOL_STEP)
            assert ok, (topo, H, "k", k, "col0", c0, worst)
    # the K-iteration run
    # (stepped: one launch of the row-streaming kernels per iteration, the loop the benchmark times;
    # otherwise gpga_run, which takes a run of 8 or more iterations through the multi-iteration launch)
    g.init_from_seed(x0_kind, x0_std, b_shift)
    launches0 = g.launch_count()
    if stepped:
        for k in range(K):
            g.step(k)
        assert g.launch_count() - launches0 == K
    else:
        g.run(K)
    x = g.get_x()
    for c0 in offs:
        X0, p = ora[c0]
        ok, worst = close(_gpu_block(x, c0, width(c0)), o.run(p, X0, 0, K), TOL_RUN)
        assert ok, (topo, H, "run col0", c0, worst)
    xi = g.consensus_distance()
    assert np.isfinite(xi) and xi >= 0.0
    if H and K % H == 0:
        assert xi == 0.0            # ended on a global average: rows bit-identical
    elif check_xi:
        # the whole n x d state through the oracle: the kernel's strided pass over all column
        # groups and its 64-bit element offsets, on a state whose rows differ
        want = _oracle_xi_of_device_state(x, d)
        assert want > 0.0
        assert abs(xi - want) <= 1e-5 * want, (topo, H, xi, want)
    g.close()


def test_config_3_resnet50_sized():
    torch = _torch()
    n, d, gamma, sigma, K = 64, 25_557_032, 0.01, 0.01, 50
    if _free_gib() < 3 * n * d * 4 / 2**30 + 2:
        pytest.skip("not enough free device memory")
    ld = (d + 31) // 32 * 32          # the benchmark's layout: rows padded to 128 bytes
    xa = torch.empty((n, ld), dtype=torch.float32, device="cuda")
    xb = torch.empty_like(xa)
    b = torch.empty_like(xa)
    scratch = torch.empty(4 << 20, dtype=torch.uint8, device="cuda")   # >= gpga_scratch_bytes at these sizes
    offs = _blocks(d, 64, np.random.default_rng(3))
    assert d % 128 == 40 and offs[-1] + BLOCK == d
    for topo in ("ring", "exp"):
        for H in (4, 16, 0):
            ks = [0]
            if H == 4:
                ks = [0, 3] if topo == "ring" else [0, 1, 2, 3, 4, 5]   # hops 1..32; k=3 is global
            # K = 50 ends between global averages for H = 16 and for pure gossip
            # (H = 4: one launch of the row-streaming kernels per iteration, the loop the benchmark times;
            # the other periods through gpga_run's multi-iteration launch)
            _run_case((xa, xb, b, scratch), n, d, topo, H, gamma, sigma, K,
                      pkg.GPGA_X0_SHARED_NORMAL, 0.1, 0.5, offs, ks, ld=ld,
                      check_xi=(topo, H) in (("ring", 16), ("exp", 0)), stepped=(H == 4))
    # the dense layout (row stride d, rows not 128-byte aligned) once as well
    _run_case((xa, xb, b, scratch), n, d, "ring", 4, gamma, sigma, 8, pkg.GPGA_X0_SHARED_NORMAL, 0.1, 0.5,
              offs, [0], ld=d)
    del xa, xb, b
    torch.cuda.empty_cache()


def test_config_3_through_the_host_pipeline():
    """The ResNet-50-sized job through the host entry (pinned X0 and b in, X^(K) out, moved as
    column chunks on three streams): bit-identical to the resident run on sampled blocks, and
    within tolerance of the oracle on blocks that straddle chunk boundaries."""
    torch = _torch()
    n, d, gamma, sigma, K, H = 64, 25_557_032, 0.01, 0.01, 8, 4
    if _free_gib() < 3 * n * d * 4 / 2**30 + 2:
        pytest.skip("not enough free device memory")
    ld = (d + 31) // 32 * 32
    try:
        host = [torch.empty((n, d), dtype=torch.float32, pin_memory=True) for _ in range(3)]
    except RuntimeError:
        pytest.skip("cannot pin 3 x 6.5 GB of host memory")
    x0_h, b_h, out_h = host
    g = pkg.Gpga(n, d, pkg.GPGA_TOPO_RING, H, gamma, SEED)
    g.set_objective(pkg.GPGA_OBJ_QUADRATIC, sigma=sigma)
    g.set_row_stride(ld)
    xa, xb, b = g.allocate()
    g.init_from_seed(pkg.GPGA_X0_SHARED_NORMAL, 0.1, 0.5)
    x0_h.copy_(xa[:, :d])
    b_h.copy_(b[:, :d])
    torch.cuda.synchronize()
    chunks = -(-n * d * 4 // (128 << 20))                 # the library's rule at this size: 128 MB of one buffer per chunk
    width = -(-(-(-d // chunks)) // 32) * 32
    assert chunks == 49 and width == 521_600
    rng = np.random.default_rng(8)
    offs = sorted({0, (d - BLOCK) // 4 * 4, width - 512, 2 * width - 4, 48 * width - 1020} |
                  {int(rng.integers(0, (d - BLOCK) // 4)) * 4 for _ in range(27)})
    g.run(K)
    resident = {c0: _gpu_block(g.get_x(), c0, min(BLOCK, d - c0)) for c0 in offs}
    out_h.fill_(float("nan"))
    g.run_host(x0_h, b_h, K, out_h)
    assert g.get_k() == K
    out = out_h.numpy()
    assert not np.isnan(out[:, ::4099]).any()
    for c0 in offs:
        w = min(BLOCK, d - c0)
        assert np.array_equal(out[:, c0:c0 + w], resident[c0]), c0
        assert np.array_equal(_gpu_block(g.get_x(), c0, w), resident[c0]), c0
    for c0 in (width - 512, 2 * width - 4, 48 * width - 1020):      # across chunk boundaries
        w = min(BLOCK, d - c0)
        B = o.init_b(n, w, SEED, 0.5, c0).astype(np.float32)
        X0 = o.init_x0(n, w, SEED, o.X0_SHARED_NORMAL, 0.1, c0).astype(np.float32)
        p = o.Problem(o.TOPO_RING, H, gamma, SEED, sigma=sigma, data=B, col0=c0)
        ok, worst = close(out[:, c0:c0 + w], o.run(p, X0, 0, K), TOL_RUN)
        assert ok, (c0, worst)
    g.close()
    del xa, xb, b, host, x0_h, b_h, out_h
    torch.cuda.empty_cache()


def test_config_4_bert_large_sized():
    torch = _torch()
    n, d, gamma, sigma, K, H = 16, 335_141_888, 0.01, 0.01, 20, 4
    if _free_gib() < 3 * n * d * 4 / 2**30 + 2:
        pytest.skip("not enough free device memory")
    assert n * d > 2**32            # element indices need 64 bits
    xa = torch.empty((n, d), dtype=torch.float32, device="cuda")
    xb = torch.empty_like(xa)
    b = torch.empty_like(xa)
    scratch = torch.empty(4 << 20, dtype=torch.uint8, device="cuda")   # >= gpga_scratch_bytes at these sizes
    offs = _blocks(d, 48, np.random.default_rng(4))
    # the configuration's K = 20 iterations with one launch of the row-streaming kernels each (the loop the
    # benchmark times)
    _run_case((xa, xb, b, scratch), n, d, "exp", H, gamma, sigma, K, pkg.GPGA_X0_ZERO, 1.0, 0.0,
              offs, [0, 1, 2, 3], stepped=True)
    # K = 18 ends two gossip steps after a global average: a non-zero consensus distance over
    # n d > 2^32 elements, recomputed by the oracle from the downloaded state
    _run_case((xa, xb, b, scratch), n, d, "exp", H, gamma, sigma, 18, pkg.GPGA_X0_ZERO, 1.0, 0.0,
              offs[::6], [], check_xi=True, stepped=True)
    # gpga_run takes 8 or more iterations through the multi-iteration launch: 10.5 M strips of 8 column groups
    _run_case((xa, xb, b, scratch), n, d, "exp", H, gamma, sigma, K, pkg.GPGA_X0_ZERO, 1.0, 0.0,
              offs[::2], [])
    del xa, xb, b
    torch.cuda.empty_cache()


def test_config_4_sharded_by_nodes_on_one_device():
    """The BERT-Large-sized problem as two node shards of eight nodes each on one device (a shard's
    state has 2.7e9 elements: 64-bit offsets in the shard kernels), filled from the seed by each shard
    for its own nodes, five iterations -- hops 1, 2, 4 inside a shard or across, hop 8 where every row
    crosses, then a global average -- with one copy per message between the shards; sampled column
    blocks against the oracle's run of all sixteen nodes."""
    torch = _torch()
    from paper_2105_09080_b200 import node_sharded as ns
    n, d, gamma, sigma, K, H, shards = 16, 335_141_888, 0.01, 0.01, 5, 5, 2
    n_l = n // shards
    if _free_gib() < shards * 5 * n_l * d * 4 / 2**30 + 4:
        pytest.skip("not enough free device memory")
    parts = []
    for s in range(shards):
        sh = ns.NodeShard(n, d, pkg.GPGA_TOPO_EXP, H, gamma, SEED, shards, s, sigma=sigma)
        xa = torch.empty((n_l, d), dtype=torch.float32, device="cuda")
        sh.bind(xa, torch.empty_like(xa), torch.empty_like(xa))
        sh.init_from_seed(pkg.GPGA_X0_PER_NODE_NORMAL, 0.1, 0.5)
        parts.append(sh)
    offs = _blocks(d, 12, np.random.default_rng(6))
    # the shards' fills are the whole problem's rows (keyed by the global node index)
    for c0 in offs[:4]:
        want = o.init_x0(n, BLOCK, SEED, o.X0_PER_NODE_NORMAL, 0.1, c0)
        got = np.concatenate([_gpu_block(sh.get_x(), c0, BLOCK) for sh in parts])
        assert np.abs(got - want).max() <= 1e-5
    for k in range(K):
        for sh in parts:
            sh.export(k)
        ns.exchange_local(parts, k)
        for sh in parts:
            sh.step(k)
    for c0 in offs:
        w = min(BLOCK, d - c0)
        B = o.init_b(n, w, SEED, 0.5, c0).astype(np.float32)
        X0 = o.init_x0(n, w, SEED, o.X0_PER_NODE_NORMAL, 0.1, c0).astype(np.float32)
        p = o.Problem(o.TOPO_EXP, H, gamma, SEED, sigma=sigma, data=B, col0=c0)
        got = np.concatenate([_gpu_block(sh.get_x(), c0, w) for sh in parts])
        ok, worst = close(got, o.run(p, X0, 0, K), TOL_RUN)
        assert ok, ("col0", c0, worst)
        assert np.all(got == got[0])        # K = H = 5: the run ends on a global average
    for sh in parts:
        sh.close()
    del parts, sh, xa
    torch.cuda.empty_cache()
