"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element,
on the same seeded inputs.  Tolerances: |gpu - oracle| <= 1e-6 (1 + |oracle|) after one
iteration, 1e-4 (1 + |oracle|) after a K-iteration run, consensus distance 1e-5 relative."""
import numpy as np
import pytest

import paper_2105_09080_b200 as pkg
from oracle import gpga_oracle as o
from paper_2105_09080_b200 import binding
from paper_2105_09080_b200.inputs import logistic_inputs, quadratic_inputs

pytestmark = pytest.mark.gpu

TOL_STEP = 1e-6
TOL_RUN = 1e-4

TOPO = {"ring": (pkg.GPGA_TOPO_RING, o.TOPO_RING), "exp": (pkg.GPGA_TOPO_EXP, o.TOPO_EXP),
        "grid": (pkg.GPGA_TOPO_GRID, o.TOPO_GRID),
        "static_exp": (pkg.GPGA_TOPO_STATIC_EXP, o.TOPO_STATIC_EXP),
        "none": (pkg.GPGA_TOPO_NONE, o.TOPO_NONE)}


def _torch():
    import torch
    return torch


def close(got, want, tol):
    err = np.abs(got.astype(np.float64) - want.astype(np.float64))
    bound = tol * (1 + np.abs(want.astype(np.float64)))
    worst = float((err / bound).max()) if err.size else 0.0
    return worst <= 1.0, worst


def make_quadratic(n, d, topo, H, gamma, seed, sigma, X0, B, col0=0, grid_cols=0):
    torch = _torch()
    g = pkg.Gpga(n, d, TOPO[topo][0], H, gamma, seed)
    g.set_objective(pkg.GPGA_OBJ_QUADRATIC, sigma=sigma)
    if col0:
        g.set_column_offset(col0)
    if grid_cols:
        g.set_grid_cols(grid_cols)
    xa = torch.from_numpy(X0).cuda()
    g.bind(xa, torch.empty_like(xa), torch.from_numpy(B).cuda())
    p = o.Problem(TOPO[topo][1], H, gamma, seed, sigma=sigma, data=B, col0=col0, grid_cols=grid_cols)
    return g, p


# ------------------------------------------------------------------ generator
def test_device_philox_known_answers_and_random_counters():
    torch = _torch()
    from pathlib import Path
    rows = [l.split() for l in (Path(__file__).parent / "golden" / "philox4x32_10_kat.txt")
            .read_text().splitlines() if l.strip() and not l.startswith("#")]
    for row in rows:
        v = [int(t, 16) for t in row]
        ctr = torch.tensor(np.array([v[0:4]], dtype=np.uint32).view(np.int32), device="cuda")
        out = binding.philox_words(ctr, v[4], v[5]).cpu().numpy().view(np.uint32)[0]
        assert [int(x) for x in out] == v[6:10]
    rng = np.random.default_rng(1)
    ctr = rng.integers(0, 2**32, (4096, 4), dtype=np.uint64).astype(np.uint32)
    out = binding.philox_words(torch.tensor(ctr.view(np.int32), device="cuda"), 0xDEADBEEF, 0x1234567)
    out = out.cpu().numpy().view(np.uint32)
    for t in range(0, 4096, 37):
        assert np.array_equal(out[t], o.philox4x32_10(ctr[t], [0xDEADBEEF, 0x1234567]))


# The normals enter the state as gamma * sigma * z, so an error dz costs gamma sigma dz.  The
# largest gamma * sigma of the benchmark configurations is 0.01; keeping that contribution
# below a quarter of the one-step tolerance needs |dz| <= 2.5e-5.
DZ_MAX = 2.5e-5


def test_device_box_muller_exhaustive_radius_and_angle():
    torch = _torch()
    m = np.arange(2**24, dtype=np.uint32)
    words = torch.tensor((m << 8).view(np.int32), device="cuda")
    # every value of u1, at angles 0 (z = (r, 0)) and pi/2 + a bit
    for bword in (0, (2**22 + 12345) << 8):
        bw = torch.full_like(words, bword)
        z = binding.box_muller_words(words, bw).cpu().numpy()
        want = o.box_muller_many(m << 8, np.full(m.shape, bword, dtype=np.uint32))
        assert np.abs(z - want).max() <= DZ_MAX
    # every value of u2, at a small, a typical and the largest radius
    for aword in ((2**24 - 2) << 8, 0x7FFFFF00, 0):
        aw = torch.full_like(words, np.array([aword], dtype=np.uint32).view(np.int32)[0])
        z = binding.box_muller_words(aw, words).cpu().numpy()
        want = o.box_muller_many(np.full(m.shape, aword, dtype=np.uint32), m << 8)
        assert np.abs(z - want).max() <= DZ_MAX


def test_device_normal_fill_matches_oracle_keying():
    seed = (0xABCDEF12 << 32) | 0x3456789A
    z = binding.normal_fill(seed, 0, 7, 3, 1000, 257).cpu().numpy()
    for t in (0, 1, 100, 256):
        assert np.abs(z[t] - o.normal4(seed, 0, 7, 3, 1000 + t)).max() <= DZ_MAX
    assert abs(z.mean()) < 0.2 and abs(z.std() - 1) < 0.1


# ------------------------------------------------------------------ one step, every kernel
# below 148 * 32 column groups (d < 18944) a step goes through the tile kernel, above it through
# the row-streaming kernels: both ranges, with 128-bit and scalar (d % 4 != 0) shapes
SHAPES = [(1, 4), (2, 8), (3, 12), (4, 132), (5, 1028), (8, 4100), (16, 1024 + 40), (7, 6), (3, 1),
          (6, 1031), (64, 520),
          (1, 20004), (2, 20008), (3, 19000), (4, 24580), (5, 20007), (7, 19001), (9, 32772), (64, 19004)]


@pytest.mark.parametrize("n,d", SHAPES)
@pytest.mark.parametrize("sigma", [0.0, 0.3])
def test_ring_and_global_one_step(n, d, sigma):
    X0, B = quadratic_inputs(n, d, 100 + n, x0="per_node")
    for H, k in ((0, 5), (3, 2)):           # gossip step; global-average step (mod(k+1,H)=0)
        g, p = make_quadratic(n, d, "ring", H, 0.25, 77, sigma, X0, B)
        g.step(k)
        want = o.step(p, X0, k)
        ok, worst = close(g.get_x().cpu().numpy(), want, TOL_STEP)
        assert ok, (H, k, worst)
        if H:
            got = g.get_x().cpu().numpy()
            assert np.all(got == got[0])    # rows bit-identical after a global average
        g.close()


@pytest.mark.parametrize("n", [1, 2, 4, 8, 32, 64])
@pytest.mark.parametrize("d", [4, 7, 1028, 4096 + 8, 20004, 19003])
def test_exp_one_step_every_hop(n, d):
    X0, B = quadratic_inputs(n, d, 200 + n, x0="per_node")
    tau = max(1, int(np.log2(n)))
    for k in range(tau + 1):
        g, p = make_quadratic(n, d, "exp", 0, 0.1, 5, 0.2, X0, B)
        g.step(k)
        ok, worst = close(g.get_x().cpu().numpy(), o.step(p, X0, k), TOL_STEP)
        assert ok, (k, worst)
        g.close()


@pytest.mark.parametrize("topo,n,gc", [("grid", 12, 4), ("grid", 16, 0), ("grid", 6, 1),
                                       ("static_exp", 8, 0), ("static_exp", 64, 0), ("none", 5, 0)])
@pytest.mark.parametrize("d", [8, 1030])
def test_tile_topologies_one_step(topo, n, gc, d):
    X0, B = quadratic_inputs(n, d, 300 + n, x0="per_node")
    g, p = make_quadratic(n, d, topo, 0, 0.2, 9, 0.4, X0, B, grid_cols=gc)
    if topo == "grid" and gc == 0:
        p.grid_cols = 4                      # library default: most square torus
    g.step(3)
    ok, worst = close(g.get_x().cpu().numpy(), o.step(p, X0, 3), TOL_STEP)
    assert ok, worst
    g.close()


@pytest.mark.parametrize("topo,H,k", [("ring", 0, 1), ("exp", 0, 2), ("ring", 2, 1), ("grid", 0, 0)])
@pytest.mark.parametrize("d,ld", [(1000, 1024), (1030, 1056), (7, 9), (1026, 1027), (20000, 20032), (19002, 19003)])
def test_padded_row_stride(topo, H, k, d, ld):
    """Rows padded to ld floats: same results as the dense layout; padding is never touched."""
    torch = _torch()
    n = 8
    X0, B = quadratic_inputs(n, d, 500 + d, x0="per_node")
    g = pkg.Gpga(n, d, TOPO[topo][0], H, 0.2, 13)
    g.set_objective(pkg.GPGA_OBJ_QUADRATIC, sigma=0.3)
    g.set_row_stride(ld)
    sentinel = -12345.0
    bufs = [torch.full((n, ld), sentinel, dtype=torch.float32, device="cuda") for _ in range(3)]
    bufs[0][:, :d] = torch.from_numpy(X0).cuda()
    bufs[2][:, :d] = torch.from_numpy(B).cuda()
    g.bind(*bufs)
    g.step(k)
    p = o.Problem(TOPO[topo][1], H, 0.2, 13, sigma=0.3, data=B, grid_cols=4 if topo == "grid" else 0)
    want = o.step(p, X0, k)
    out = g.get_x().cpu().numpy()
    ok, worst = close(out[:, :d], want, TOL_STEP)
    assert ok, worst
    assert np.all(out[:, d:] == sentinel)
    xi = o.consensus_distance(want)
    assert abs(g.consensus_distance() - xi) <= 1e-5 * xi + n * d * (2.0**-22 * 8) ** 2
    assert abs(g.mean_loss() - o.quadratic_mean_loss(out[:, :d], B)) <= 1e-6 * o.quadratic_mean_loss(want, B)
    xbar = np.repeat(want.astype(np.float64).mean(0, keepdims=True), n, axis=0)
    assert abs(g.global_loss() - o.quadratic_mean_loss(xbar, B)) <= 1e-5 * o.quadratic_mean_loss(xbar, B)
    g.init_from_seed(pkg.GPGA_X0_PER_NODE_NORMAL, 1.0, 0.5)
    assert np.abs(bufs[2].cpu().numpy()[:, :d] - o.init_b(n, d, 13, 0.5)).max() <= 3e-5
    assert np.all(bufs[2].cpu().numpy()[:, d:] == sentinel)
    assert np.all(bufs[0].cpu().numpy()[:, d:] == sentinel)
    g.close()


def test_run_host_with_padded_rows():
    torch = _torch()
    n, d, ld, K = 4, 1000, 1024, 5
    X0, B = quadratic_inputs(n, d, 9)
    g, _ = make_quadratic(n, d, "ring", 2, 0.1, 3, 0.2, X0, B)
    g.run(K)
    want = g.get_x().cpu().numpy()
    g2 = pkg.Gpga(n, d, pkg.GPGA_TOPO_RING, 2, 0.1, 3)
    g2.set_objective(pkg.GPGA_OBJ_QUADRATIC, sigma=0.2)
    g2.set_row_stride(ld)
    g2.allocate()
    out = torch.empty((n, d), dtype=torch.float32).pin_memory()
    g2.run_host(torch.from_numpy(X0).pin_memory(), torch.from_numpy(B).pin_memory(), K, out)
    assert np.array_equal(out.numpy(), want)


@pytest.mark.parametrize("topo,H", [("ring", 3), ("exp", 2)])
def test_run_host_in_column_chunks_equals_the_device_run(topo, H):
    """A state too large for one chunk goes through the host entry as a pipeline of column chunks
    (upload, K iterations, download on three streams); every element must come out exactly as from
    the unchunked run on resident buffers.  384 MB per buffer = 16 chunks, the last one ragged."""
    torch = _torch()
    n, d, K = 8, 12_000_040, 5
    rng = np.random.default_rng(17)
    X0 = rng.standard_normal((n, d), dtype=np.float32)
    B = rng.standard_normal((n, d), dtype=np.float32)
    ld = (d + 31) // 32 * 32
    outs = []
    for host in (False, True):
        g = pkg.Gpga(n, d, TOPO[topo][0], H, 0.1, 5)
        g.set_objective(pkg.GPGA_OBJ_QUADRATIC, sigma=0.3)
        g.set_row_stride(ld)
        xa, _, data = g.allocate()
        if host:
            out = torch.empty((n, d), dtype=torch.float32).pin_memory()
            out.fill_(float("nan"))
            g.run_host(torch.from_numpy(X0).pin_memory(), torch.from_numpy(B).pin_memory(), K, out)
            assert g.get_k() == K
            assert np.array_equal(g.get_x()[:, :d].cpu().numpy(), out.numpy())   # the device state is whole too
            outs.append(out.numpy())
        else:
            xa[:, :d] = torch.from_numpy(X0).cuda()
            data[:, :d] = torch.from_numpy(B).cuda()
            g.run(K)
            outs.append(g.get_x()[:, :d].cpu().numpy())
        g.close()
        del xa, data
    assert np.array_equal(outs[0], outs[1])


def test_column_offset_keys_the_noise():
    n, d, c0 = 4, 64, 4096
    X0, B = quadratic_inputs(n, d, 1)
    g, p = make_quadratic(n, d, "ring", 0, 0.1, 3, 1.0, X0, B, col0=c0)
    g.step(0)
    ok, worst = close(g.get_x().cpu().numpy(), o.step(p, X0, 0), TOL_STEP)
    assert ok, worst
    g0, p0 = make_quadratic(n, d, "ring", 0, 0.1, 3, 1.0, X0, B)
    g0.step(0)
    assert not np.array_equal(g0.get_x().cpu().numpy(), g.get_x().cpu().numpy())


def test_step_is_a_pure_function_and_resume_is_exact():
    n, d = 8, 2052
    X0, B = quadratic_inputs(n, d, 2)
    g, _ = make_quadratic(n, d, "exp", 4, 0.1, 11, 0.1, X0, B)
    g.run(10)
    full = g.get_x().cpu().numpy().copy()
    g2, _ = make_quadratic(n, d, "exp", 4, 0.1, 11, 0.1, X0, B)
    g2.run(6)
    mid = g2.get_x().cpu().numpy().copy()
    g3, _ = make_quadratic(n, d, "exp", 4, 0.1, 11, 0.1, mid, B)
    g3.set_k(6)
    g3.run(4)
    assert np.array_equal(g3.get_x().cpu().numpy(), full)
    assert g.get_k() == 10


# ------------------------------------------------------------------ consensus distance
# (8, 1_300_000) and (3, 1_250_003): more column groups than 1184 blocks of 256 threads cover in one
# pass (d > 1.21 M), so every thread strides to a second group -- 128-bit and scalar paths
@pytest.mark.parametrize("n,d", [(1, 8), (2, 5), (8, 4100), (64, 777), (16, 100000), (8, 1_300_000),
                                 (3, 1_250_003)])
def test_consensus_distance(n, d):
    X0, B = quadratic_inputs(n, d, 400 + n, x0="per_node")
    g, _ = make_quadratic(n, d, "ring", 0, 0.1, 1, 0.0, X0, B)
    want = o.consensus_distance(X0)
    assert abs(g.consensus_distance() - want) <= 1e-5 * want + 1e-300
    # nearly consensual rows: one row differs in the last bits
    X1 = np.repeat(X0[:1], n, axis=0).copy()
    if n > 1:
        X1[n - 1] = np.nextafter(X1[n - 1], np.float32(10))
    g, _ = make_quadratic(n, d, "ring", 0, 0.1, 1, 0.0, X1, B)
    want = o.consensus_distance(X1)
    assert abs(g.consensus_distance() - want) <= 1e-5 * want
    g.close()
