"""Weight matrices W of Section 3 as inputs for topology SPARSE (CSR arrays), and their
block-diagonal replication for batches of independent problems.

A caller of the library supplies W; this module only writes down the sparsity patterns and
weights of the graphs the paper's experiments name (ring, grid, static exponential graph,
W = I for Local SGD, the exact average for the global-averaging step).  The mixing itself runs
in the library's kernels.  Every matrix here is symmetric or circulant with rows summing to one,
hence doubly stochastic.
"""
from __future__ import annotations

import numpy as np


def neighbour_lists(topology: str, n: int, grid_cols: int = 0):
    """[(neighbour, weight), ...] for every node i of one n-node graph.

    ring: 1/3 on i-1, i, i+1 (indices mod n; repeated neighbours keep their repeated weight).
    grid: r x c torus, 1/5 on the node and its four neighbours.
    static_exp: 1/(T+1) on i and (i + 2^t) mod n, t < T = ceil(log2 n).
    none: W = I.   average: 1/n on every node (the global-averaging step as a matrix).
    """
    rows = []
    for i in range(n):
        if topology == "ring":
            nb = [((i - 1) % n, 1 / 3), (i, 1 / 3), ((i + 1) % n, 1 / 3)]
        elif topology == "grid":
            c = grid_cols or _square_cols(n)
            r = n // c
            a, b = divmod(i, c)
            nb = [(((a - 1) % r) * c + b, 0.2), (((a + 1) % r) * c + b, 0.2), (a * c + (b - 1) % c, 0.2),
                  (a * c + (b + 1) % c, 0.2), (i, 0.2)]
        elif topology == "static_exp":
            T = max(1, int(np.ceil(np.log2(n)))) if n > 1 else 0
            nb = [(i, 1 / (T + 1))] + [((i + (1 << t)) % n, 1 / (T + 1)) for t in range(T)]
        elif topology == "none":
            nb = [(i, 1.0)]
        elif topology == "average":
            nb = [(j, 1.0 / n) for j in range(n)]
        else:
            raise ValueError(topology)
        rows.append(nb)
    return rows


def _square_cols(n: int) -> int:
    c = int(np.floor(np.sqrt(n)))
    while c > 1 and n % c:
        c -= 1
    return n // c


def csr(topology: str, n: int, copies: int = 1, grid_cols: int = 0):
    """CSR arrays (row_ptr int32, col_idx int32, weights float32) of `copies` disjoint copies of the
    n-node graph: node t * n + i is node i of copy t (a block-diagonal W).  Entries of a row that
    name the same neighbour are merged."""
    base = []
    for nb in neighbour_lists(topology, n, grid_cols):
        merged = {}
        for j, w in nb:
            merged[j] = merged.get(j, 0.0) + w
        base.append(sorted(merged.items()))
    row_ptr, col, val = [0], [], []
    for t in range(copies):
        for nb in base:
            for j, w in nb:
                col.append(t * n + j)
                val.append(w)
            row_ptr.append(len(col))
    return (np.asarray(row_ptr, dtype=np.int32), np.asarray(col, dtype=np.int32),
            np.asarray(val, dtype=np.float32))


def dense(topology: str, n: int, copies: int = 1, grid_cols: int = 0) -> np.ndarray:
    """The same matrix written out (tests, tiny sizes)."""
    row_ptr, col, val = csr(topology, n, copies, grid_cols)
    N = n * copies
    W = np.zeros((N, N))
    for i in range(N):
        for e in range(row_ptr[i], row_ptr[i + 1]):
            W[i, col[e]] += float(val[e])
    return W
