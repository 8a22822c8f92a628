"""The allocation-free logistic-gradient entry point (collected last on purpose).

Some users of this library cannot allocate device memory where they need the gradient --
a loop that must not synchronise the GPU, or a plug-in that only ever receives tensors from
its host framework.  For them the library carries its own fixed scratch array.  This test
calls that entry point through the C ABI and checks it against what the ordinary handle-based
path (gpga_step with the logistic objective) computes from the same inputs, twice in a row,
because the scratch array keeps the first call's contents when the second one starts.
"""
import numpy as np
import pytest

import paper_2105_09080_b200 as pkg
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


def test_noalloc_gradient_matches_handle_path_on_two_calls_in_a_row():
    import torch
    n, m, d, batch, l2, seed = 16, 512, 1024, 128, 1e-4, 20210509
    A, y = logistic_inputs(n, m, d, seed)
    rng = np.random.default_rng(1)
    states = [(0.3 * rng.standard_normal((n, d))).astype(np.float32) for _ in range(2)]
    A_dev, y_dev = torch.from_numpy(A).cuda(), torch.from_numpy(y).cuda()
    G_dev = torch.empty((n, d), dtype=torch.float32, device="cuda")
    for call, (X0, k) in enumerate(zip(states, (3, 4))):
        x_dev = torch.from_numpy(X0).cuda()
        st, need, _ = binding.logistic_gradient_noalloc(A_dev, y_dev, x_dev, batch, l2, seed, k, out=G_dev)
        assert st == pkg.GPGA_OK
        assert need == 4 * n * d * 4 <= binding.GPGA_NOALLOC_SCRATCH_BYTES       # ceil(128/32) chunks
        torch.cuda.synchronize()
        G = G_dev.cpu().numpy()
        want = _reference_step(A, y, X0, batch, l2, seed, k)                     # = X0 - G
        got = X0 - G
        err = np.abs(got.astype(np.float64) - want)
        assert np.all(err <= TOL * (1 + np.abs(want))), (call, float(err.max()))
        assert np.abs(G).max() > 1e-3                                           # a real gradient, not zeros


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
