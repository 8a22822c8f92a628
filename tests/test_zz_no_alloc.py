"""The allocation-free logistic-gradient entry point.

Some users of this library cannot allocate device memory where they need the gradient --
a loop that must not synchronise the GPU, or a plug-in that only ever receives tensors from
its host framework.  For them the library carries its own fixed scratch array.  These tests
call that entry point through the C ABI and check its output, twice in a row (the scratch
array keeps the first call's contents when the second one starts), against the CPU oracle's
gradient matrix and against what the ordinary handle-based path (gpga_step with the logistic
objective) computes from the same inputs.

Why the file sorts last: the entry point stands apart from the iteration the other files
cover, so a run that stops at the first failure (`pytest -x`) should reach it only after
every other test has run.  The tests do not depend on that order: they pass alone in a
fresh process as well as after the rest of the suite.
"""
import ctypes as C

import numpy as np
import pytest

import paper_2105_09080_b200 as pkg
from oracle import gpga_oracle as o
from paper_2105_09080_b200 import binding
from paper_2105_09080_b200.inputs import logistic_inputs

pytestmark = pytest.mark.gpu

TOL = 1e-6      # the one-iteration tolerance of the parity tests: |a - b| <= TOL (1 + |b|)


def _reference_step(A, y, X0, batch, l2, seed, k):
    """X - G through the existing entry point: W = I, no global averaging, gamma = 1."""
    import torch
    n, m, d = A.shape
    g = pkg.Gpga(n, d, pkg.GPGA_TOPO_NONE, 0, 1.0, seed)
    g.set_objective(pkg.GPGA_OBJ_LOGISTIC, l2=l2, m=m, batch=batch)
    xa = torch.from_numpy(X0).cuda()
    g.bind(xa, torch.empty_like(xa), torch.from_numpy(A).cuda(), torch.from_numpy(y).cuda())
    g.step(k)
    out = g.get_x().cpu().numpy().copy()
    g.close()
    return out


# d = 1024: rows staged by per-warp bulk copies; d = 2052: the two-tile staging (ragged over the
# threads); d = 9000: plain loads -- the three gradient kernels the entry point can take
@pytest.mark.parametrize("n,m,d,batch", [(16, 512, 1024, 128), (6, 96, 2052, 70), (3, 40, 9000, 33)])
def test_noalloc_gradient_matches_oracle_and_handle_path_on_two_calls_in_a_row(n, m, d, batch):
    import torch
    l2, seed = 1e-4, 20210509
    A, y = logistic_inputs(n, m, d, seed)
    rng = np.random.default_rng(1)
    states = [(0.3 * rng.standard_normal((n, d))).astype(np.float32) for _ in range(2)]
    A_dev, y_dev = torch.from_numpy(A).cuda(), torch.from_numpy(y).cuda()
    G_dev = torch.empty((n, d), dtype=torch.float32, device="cuda")
    x_devs = [torch.from_numpy(X0).cuda() for X0 in states]
    A64 = A.astype(np.float64)
    free_before_second = None
    for call, (X0, k) in enumerate(zip(states, (3, 4))):
        G_dev.fill_(float("nan"))
        torch.cuda.synchronize()
        if call == 1:           # the first call on a device may load the library's device code
            free_before_second = torch.cuda.mem_get_info()[0]
        st, need, _ = binding.logistic_gradient_noalloc(A_dev, y_dev, x_devs[call], batch, l2, seed, k, out=G_dev)
        assert st == pkg.GPGA_OK
        assert need == -(-batch // 32) * n * d * 4 <= binding.GPGA_NOALLOC_SCRATCH_BYTES
        torch.cuda.synchronize()
        if call == 1:           # nothing was allocated: the device's free memory did not move
            assert torch.cuda.mem_get_info()[0] == free_before_second
        G = G_dev.cpu().numpy()
        assert np.isfinite(G).all()
        # the oracle's gradient matrix for the mini-batches of iteration k (fp64)
        G_want = o.logistic_gradient_matrix(A64, y, X0, seed, k, batch, l2)
        err = np.abs(G.astype(np.float64) - G_want)
        assert np.all(err <= TOL * (1 + np.abs(G_want))), (call, float(err.max()))
        assert np.abs(G_want).max() > 1e-3                                      # a real gradient, not zeros
        # and the existing entry point: X0 - G from gpga_step with W = I and gamma = 1
        want = _reference_step(A, y, X0, batch, l2, seed, k)
        err = np.abs((X0 - G).astype(np.float64) - want)
        assert np.all(err <= TOL * (1 + np.abs(want))), (call, float(err.max()))


def test_noalloc_refuses_what_does_not_fit_and_bad_arguments():
    import torch
    n, m, d, batch = 64, 64, 4096, 256              # 8 chunks * 64 * 4096 floats = 8 MiB > 4 MiB
    A = torch.zeros((n, m, d), dtype=torch.float32, device="cuda")
    y = torch.ones((n, m), dtype=torch.float32, device="cuda")
    x = torch.zeros((n, d), dtype=torch.float32, device="cuda")
    st, need, _ = binding.logistic_gradient_noalloc(A, y, x, batch, 0.0, 1, 0)
    assert st == pkg.GPGA_ERR_UNSUPPORTED
    assert need == 8 * n * d * 4 > binding.GPGA_NOALLOC_SCRATCH_BYTES
    st, need, _ = binding.logistic_gradient_noalloc(A, y, x, 0, 0.0, 1, 0)
    assert st == pkg.GPGA_ERR_INVALID_ARG
    L = pkg.lib()
    assert L.gpga_logistic_gradient_noalloc(None, None, None, 8, 1, 8, 1, 1, 0.0, 1, 0, None, None, None) \
        == pkg.GPGA_ERR_INVALID_ARG


def test_noalloc_refuses_memory_that_is_not_the_current_devices():
    """A buffer the current device does not own (here: plain host memory standing in for another
    GPU's) is turned away by the pointer check before anything is launched."""
    import torch
    n, m, d, batch = 2, 8, 64, 8
    A = torch.zeros((n, m, d), dtype=torch.float32, device="cuda")
    y = torch.ones((n, m), dtype=torch.float32, device="cuda")
    x = torch.zeros((n, d), dtype=torch.float32, device="cuda")
    host = np.zeros(n * d + 8, dtype=np.float32)
    addr = (host.ctypes.data + 15) // 16 * 16                    # 16-byte aligned host address
    L = pkg.lib()
    need = C.c_int64()
    st = L.gpga_logistic_gradient_noalloc(A.data_ptr(), y.data_ptr(), x.data_ptr(), d, n, d, m, batch, 0.0, 1, 0,
                                          addr, None, C.byref(need))
    assert st == pkg.GPGA_ERR_INVALID_ARG
    torch.cuda.synchronize()                                     # the context is intact
    assert not host.any()
    with pytest.raises(ValueError):                              # the binding's own same-device rule
        binding.logistic_gradient_noalloc(A, y, x, batch, 0.0, 1, 0, out=torch.zeros((n, d)))
