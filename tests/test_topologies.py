"""The weight matrices handed to topology SPARSE (paper_2105_09080_b200/topologies.py) against the
oracle's own dense matrices of Section 3, and the properties Section 3 asks of W."""
import numpy as np
import pytest

from oracle import gpga_oracle as o
from paper_2105_09080_b200 import topologies as t


@pytest.mark.parametrize("n", [1, 2, 3, 4, 20, 50])
def test_ring_matches_the_oracles_matrix(n):
    assert np.abs(t.dense("ring", n) - o.dense_w_ring(n)).max() <= 1e-7


def test_grid_and_static_exponential_match_the_oracles_matrices():
    assert np.abs(t.dense("grid", 20) - o.dense_w_grid(4, 5)).max() <= 1e-7          # the most square torus
    assert np.abs(t.dense("grid", 12, grid_cols=6) - o.dense_w_grid(2, 6)).max() <= 1e-7
    for n in (2, 4, 16, 64):
        assert np.abs(t.dense("static_exp", n) - o.dense_w_static_exp(n)).max() <= 1e-7


@pytest.mark.parametrize("name", ["ring", "grid", "static_exp", "none", "average"])
@pytest.mark.parametrize("n,copies", [(1, 1), (2, 3), (20, 2), (50, 1), (100, 2)])
def test_doubly_stochastic_and_block_diagonal(name, n, copies):
    W = t.dense(name, n, copies)
    assert np.allclose(W.sum(0), 1.0, atol=1e-5) and np.allclose(W.sum(1), 1.0, atol=1e-5)
    assert (W >= 0).all()
    for a in range(copies):
        for b in range(copies):
            block = W[a * n:(a + 1) * n, b * n:(b + 1) * n]
            if a == b:
                assert np.abs(block - W[:n, :n]).max() == 0.0          # every copy has the same W
            else:
                assert not block.any()                                 # and no edge leaves a copy
    row_ptr, col, val = t.csr(name, n, copies)
    assert row_ptr[0] == 0 and row_ptr[-1] == len(col) == len(val) and len(row_ptr) == n * copies + 1
    assert all(len(set(col[row_ptr[i]:row_ptr[i + 1]])) == row_ptr[i + 1] - row_ptr[i] for i in range(n * copies))


def test_spectral_gaps_order_the_topologies_as_the_paper_does():
    """beta = second largest eigenvalue magnitude: exponential graph < grid < ring at n = 100, and the
    ring's beta at n = 20, 50, 100 is what Section 5.1 prints (0.967, 0.995, 0.998)."""
    def beta(W):
        ev = np.sort(np.abs(np.linalg.eigvals(W)))[::-1]
        return ev[1]
    b = {name: beta(t.dense(name, 100)) for name in ("static_exp", "grid", "ring")}
    assert b["static_exp"] < b["grid"] < b["ring"] < 1.0
    assert abs(beta(t.dense("average", 30))) < 1e-6 and abs(beta(t.dense("none", 5)) - 1.0) < 1e-12
    for n, printed in ((20, 0.967), (50, 0.995), (100, 0.998)):
        assert printed - 5e-4 <= beta(t.dense("ring", n)) < printed + 1e-3      # three printed digits (100: cut, not rounded)
