"""Python face of the CPU oracle (TEST INFRASTRUCTURE ONLY).

Wraps ``gpga_oracle.c`` with ctypes and adds the pieces that are easiest to
read in numpy: the dense weight matrices W of Section 3 of the paper and the
driver loop of Algorithm 1.  Nothing here imports, or is imported by, the CUDA
package.  Only tests, the smoke check and the benchmark's CPU-baseline leg may
use this module.

State convention: ``step`` takes and returns float32 state (one rounding per
stored element per iteration, every intermediate fp64); ``step_f64`` never
rounds.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "gpga_oracle.c"
_LIB = _HERE / "libgpga_oracle.so"

TOPO_RING = 0
TOPO_EXP = 1
TOPO_GRID = 2
TOPO_STATIC_EXP = 3
TOPO_NONE = 4
TOPO_SPARSE = 5   # any doubly-stochastic W given explicitly

X0_ZERO = 0
X0_SHARED_NORMAL = 1
X0_PER_NODE_NORMAL = 2


def build(force: bool = False) -> Path:
    """Compile the C oracle with gcc (OpenMP over independent rows/columns only)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               str(_SRC), "-o", str(_LIB), "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def load(path):
    """Load an oracle shared library (the built one, or a deliberately broken copy that a test
    compiled to see whether the pins notice) and declare its signatures."""
    L = C.CDLL(str(path))
    i64, i32, u32, u64, f64 = C.c_int64, C.c_int32, C.c_uint32, C.c_uint64, C.c_double
    P = C.c_void_p
    L.gpga_oracle_philox4x32_10.argtypes = [P, P, P]
    L.gpga_oracle_philox4x32_10.restype = None
    L.gpga_oracle_box_muller.argtypes = [u32, u32, P]
    L.gpga_oracle_box_muller.restype = None
    L.gpga_oracle_normal4.argtypes = [u64, u32, u32, u32, u32, P]
    L.gpga_oracle_normal4.restype = None
    L.gpga_oracle_is_global.argtypes = [i64, i64]
    L.gpga_oracle_is_global.restype = i32
    L.gpga_oracle_exp_hop.argtypes = [i64, i64]
    L.gpga_oracle_exp_hop.restype = i64
    L.gpga_oracle_quadratic_half_step.argtypes = [i64, i64, i64, f64, f64, u64, i64, P, P, P]
    L.gpga_oracle_quadratic_half_step.restype = None
    L.gpga_oracle_gradient_half_step.argtypes = [i64, i64, f64, P, P, P]
    L.gpga_oracle_gradient_half_step.restype = None
    L.gpga_oracle_mix_ring.argtypes = [i64, i64, P, P]
    L.gpga_oracle_mix_ring.restype = None
    L.gpga_oracle_mix_exp.argtypes = [i64, i64, i64, P, P]
    L.gpga_oracle_mix_exp.restype = None
    L.gpga_oracle_mix_global.argtypes = [i64, i64, P, P]
    L.gpga_oracle_mix_global.restype = None
    L.gpga_oracle_mix_grid.argtypes = [i64, i64, i64, P, P]
    L.gpga_oracle_mix_grid.restype = None
    L.gpga_oracle_mix_static_exp.argtypes = [i64, i64, P, P]
    L.gpga_oracle_mix_static_exp.restype = None
    L.gpga_oracle_consensus_distance.argtypes = [i64, i64, P]
    L.gpga_oracle_consensus_distance.restype = f64
    L.gpga_oracle_batch_indices.argtypes = [u64, i64, i64, i64, i64, P]
    L.gpga_oracle_batch_indices.restype = None
    L.gpga_oracle_logistic_loss.argtypes = [i64, i64, P, P, P, f64]
    L.gpga_oracle_logistic_loss.restype = f64
    L.gpga_oracle_logistic_grad.argtypes = [i64, P, P, P, i64, P, f64, P]
    L.gpga_oracle_logistic_grad.restype = None
    L.gpga_oracle_logistic_gradient_matrix.argtypes = [i64, i64, i64, i64, u64, i64, P, P, P,
                                                       f64, P]
    L.gpga_oracle_logistic_gradient_matrix.restype = None
    L.gpga_oracle_init_b.argtypes = [i64, i64, i64, u64, f64, P]
    L.gpga_oracle_init_b.restype = None
    L.gpga_oracle_init_x0.argtypes = [i64, i64, i64, u64, i32, f64, P]
    L.gpga_oracle_init_x0.restype = None
    L.gpga_oracle_aga_update.argtypes = [i64, i64, i64, f64, P, P]
    L.gpga_oracle_aga_update.restype = None
    L.gpga_oracle_box_muller_many.argtypes = [P, P, i64, P]
    L.gpga_oracle_box_muller_many.restype = None
    L.gpga_oracle_quadratic_mean_loss.argtypes = [i64, i64, P, P]
    L.gpga_oracle_quadratic_mean_loss.restype = f64
    return L


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = load(_LIB)
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


# --------------------------------------------------------------------------
# generator
# --------------------------------------------------------------------------
def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    lib().gpga_oracle_philox4x32_10(_p(c), _p(k), _p(out))
    return out


def box_muller(a: int, b: int) -> np.ndarray:
    z = np.zeros(2, dtype=np.float64)
    lib().gpga_oracle_box_muller(int(a), int(b), _p(z))
    return z


def box_muller_many(a, b) -> np.ndarray:
    """Box-Muller of word pairs; returns shape (count, 2) fp64."""
    a = np.ascontiguousarray(a, dtype=np.uint32)
    b = np.ascontiguousarray(b, dtype=np.uint32)
    z = np.empty((a.size, 2), dtype=np.float64)
    lib().gpga_oracle_box_muller_many(_p(a), _p(b), a.size, _p(z))
    return z


def normal4(seed: int, stream: int, k: int, i: int, q: int) -> np.ndarray:
    z = np.zeros(4, dtype=np.float64)
    lib().gpga_oracle_normal4(int(seed), int(stream), int(k), int(i), int(q), _p(z))
    return z


# --------------------------------------------------------------------------
# schedule
# --------------------------------------------------------------------------
def is_global(k: int, H: int) -> bool:
    return bool(lib().gpga_oracle_is_global(int(k), int(H)))


def exp_hop(k: int, n: int) -> int:
    return int(lib().gpga_oracle_exp_hop(int(k), int(n)))


# --------------------------------------------------------------------------
# dense weight matrices (Section 3: doubly stochastic W; tiny n only)
# --------------------------------------------------------------------------
def dense_w_ring(n: int) -> np.ndarray:
    W = np.zeros((n, n))
    for i in range(n):
        for nb in ((i - 1) % n, i, (i + 1) % n):
            W[i, nb] += 1.0 / 3.0
    return W


def dense_w_exp(n: int, hop: int) -> np.ndarray:
    W = np.zeros((n, n))
    for i in range(n):
        W[i, i] += 0.5
        W[i, (i + hop) % n] += 0.5
    return W


def dense_w_global(n: int) -> np.ndarray:
    return np.full((n, n), 1.0 / n)


def dense_w_grid(r: int, c: int) -> np.ndarray:
    n = r * c
    W = np.zeros((n, n))
    for i in range(n):
        a, b = divmod(i, c)
        for nb in (((a - 1) % r) * c + b, ((a + 1) % r) * c + b, a * c + (b - 1) % c,
                   a * c + (b + 1) % c, i):
            W[i, nb] += 0.2
    return W


def dense_w_static_exp(n: int) -> np.ndarray:
    tau = int(np.log2(n))
    W = np.zeros((n, n))
    for i in range(n):
        W[i, i] += 1.0 / (tau + 1)
        for t in range(tau):
            W[i, (i + (1 << t)) % n] += 1.0 / (tau + 1)
    return W


def metropolis_w(adjacency: np.ndarray) -> np.ndarray:
    """Metropolis-Hastings weights of an undirected graph: w_ij = 1 / (1 + max(deg_i, deg_j)) on
    edges, the rest of each row on the diagonal; symmetric, hence doubly stochastic (Section 3)."""
    adj = np.asarray(adjacency, dtype=bool)
    n = adj.shape[0]
    deg = adj.sum(1)
    W = np.zeros((n, n))
    for i in range(n):
        for j in range(n):
            if i != j and adj[i, j]:
                W[i, j] = 1.0 / (1.0 + max(deg[i], deg[j]))
        W[i, i] = 1.0 - W[i].sum()
    return W


def dense_w(topology: int, n: int, k: int, grid_cols: int = 0, W=None) -> np.ndarray:
    if topology == TOPO_SPARSE:
        return np.asarray(W, dtype=np.float64)
    if topology == TOPO_RING:
        return dense_w_ring(n)
    if topology == TOPO_EXP:
        return dense_w_exp(n, exp_hop(k, n))
    if topology == TOPO_GRID:
        return dense_w_grid(n // grid_cols, grid_cols)
    if topology == TOPO_STATIC_EXP:
        return dense_w_static_exp(n)
    if topology == TOPO_NONE:
        return np.eye(n)
    raise ValueError(topology)


# --------------------------------------------------------------------------
# the pieces of Algorithm 1
# --------------------------------------------------------------------------
def quadratic_half_step(X, B, gamma, sigma, seed, k, col0=0) -> np.ndarray:
    X = _f64(X)
    B = _f64(B)
    n, d = X.shape
    Y = np.empty_like(X)
    lib().gpga_oracle_quadratic_half_step(n, d, int(col0), float(gamma), float(sigma), int(seed),
                                          int(k), _p(X), _p(B), _p(Y))
    return Y


def gradient_half_step(X, G, gamma) -> np.ndarray:
    X = _f64(X)
    G = _f64(G)
    Y = np.empty_like(X)
    lib().gpga_oracle_gradient_half_step(X.shape[0], X.shape[1], float(gamma), _p(X), _p(G), _p(Y))
    return Y


def mix(Y, topology: int, k: int, global_step: bool, grid_cols: int = 0, W=None) -> np.ndarray:
    """Sparse-path mixing of the half-step matrix Y (fp64 in, fp64 out)."""
    Y = _f64(Y)
    n, d = Y.shape
    Z = np.empty_like(Y)
    L = lib()
    if topology == TOPO_SPARSE and not global_step:
        # x_i = sum_{j in N_i} w_ij y_j, row by row over the stored neighbours (Algorithm 1)
        Wd = np.asarray(W, dtype=np.float64)
        for i in range(n):
            nb = np.nonzero(Wd[i])[0]
            Z[i] = sum(Wd[i, j] * Y[j] for j in nb)
        return Z
    if global_step:
        L.gpga_oracle_mix_global(n, d, _p(Y), _p(Z))
    elif topology == TOPO_RING:
        L.gpga_oracle_mix_ring(n, d, _p(Y), _p(Z))
    elif topology == TOPO_EXP:
        L.gpga_oracle_mix_exp(n, d, exp_hop(k, n), _p(Y), _p(Z))
    elif topology == TOPO_GRID:
        L.gpga_oracle_mix_grid(n // grid_cols, grid_cols, d, _p(Y), _p(Z))
    elif topology == TOPO_STATIC_EXP:
        L.gpga_oracle_mix_static_exp(n, d, _p(Y), _p(Z))
    elif topology == TOPO_NONE:
        Z[...] = Y
    else:
        raise ValueError(topology)
    return Z


def mix_dense(Y, topology: int, k: int, global_step: bool, grid_cols: int = 0, W=None) -> np.ndarray:
    """Dense-W mixing, X+ = W Y (tiny n only)."""
    Y = _f64(Y)
    n = Y.shape[0]
    Wd = dense_w_global(n) if global_step else dense_w(topology, n, k, grid_cols, W)
    return Wd @ Y


def consensus_distance(X) -> float:
    X = _f64(X)
    return float(lib().gpga_oracle_consensus_distance(X.shape[0], X.shape[1], _p(X)))


# --------------------------------------------------------------------------
# logistic regression
# --------------------------------------------------------------------------
def batch_indices(seed, k, i, batch, m) -> np.ndarray:
    idx = np.zeros(batch, dtype=np.int32)
    lib().gpga_oracle_batch_indices(int(seed), int(k), int(i), int(batch), int(m), _p(idx))
    return idx


def logistic_loss(A_i, y_i, x, l2) -> float:
    A_i = _f64(A_i)
    y_i = _f64(y_i)
    x = _f64(x)
    m, d = A_i.shape
    return float(lib().gpga_oracle_logistic_loss(m, d, _p(A_i), _p(y_i), _p(x), float(l2)))


def logistic_grad(A_i, y_i, rows, x, l2) -> np.ndarray:
    A_i = _f64(A_i)
    y_i = _f64(y_i)
    x = _f64(x)
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    g = np.empty(A_i.shape[1], dtype=np.float64)
    lib().gpga_oracle_logistic_grad(A_i.shape[1], _p(A_i), _p(y_i), _p(rows), rows.size, _p(x),
                                    float(l2), _p(g))
    return g


def logistic_gradient_matrix(A, y, X, seed, k, batch, l2) -> np.ndarray:
    """A: n x m x d, y: n x m, X: n x d  ->  G: n x d for the mini-batches of iteration k."""
    A = _f64(A)
    y = _f64(y)
    X = _f64(X)
    n, m, d = A.shape
    G = np.empty((n, d), dtype=np.float64)
    lib().gpga_oracle_logistic_gradient_matrix(n, d, m, int(batch), int(seed), int(k), _p(A),
                                               _p(y), _p(X), float(l2), _p(G))
    return G


def global_logistic_loss(A, y, x, l2) -> float:
    """(1/n) sum_i f_i(x) at a single point x (problem (1) of the paper)."""
    return float(np.mean([logistic_loss(A[i], y[i], x, l2) for i in range(A.shape[0])]))


# --------------------------------------------------------------------------
# seeded quadratic data
# --------------------------------------------------------------------------
def init_b(n, dloc, seed, shift=0.0, col0=0) -> np.ndarray:
    B = np.empty((n, dloc), dtype=np.float64)
    lib().gpga_oracle_init_b(n, dloc, int(col0), int(seed), float(shift), _p(B))
    return B


def init_x0(n, dloc, seed, kind, std=1.0, col0=0) -> np.ndarray:
    X = np.empty((n, dloc), dtype=np.float64)
    lib().gpga_oracle_init_x0(n, dloc, int(col0), int(seed), int(kind), float(std), _p(X))
    return X


# --------------------------------------------------------------------------
# driver: Algorithm 1
# --------------------------------------------------------------------------
class Problem:
    """Parameters of one run; objective is 'quadratic' (data = B) or 'logistic'
    (data = A of shape n x m x d, labels = y of shape n x m)."""

    def __init__(self, topology, H, gamma, seed, sigma=0.0, objective="quadratic", data=None,
                 labels=None, l2=0.0, batch=0, col0=0, grid_cols=0, W=None):
        self.topology = topology
        self.H = H
        self.gamma = gamma
        self.seed = seed
        self.sigma = sigma
        self.objective = objective
        self.data = data
        self.labels = labels
        self.l2 = l2
        self.batch = batch
        self.col0 = col0
        self.grid_cols = grid_cols
        self.W = W


def step_f64(p: Problem, X, k: int, dense: bool = False) -> np.ndarray:
    """One iteration of Algorithm 1 on fp64 state, no rounding."""
    if p.objective == "quadratic":
        Y = quadratic_half_step(X, p.data, p.gamma, p.sigma, p.seed, k, p.col0)
    else:
        G = logistic_gradient_matrix(p.data, p.labels, X, p.seed, k, p.batch, p.l2)
        Y = gradient_half_step(X, G, p.gamma)
    g = is_global(k, p.H)
    mixer = mix_dense if dense else mix
    return mixer(Y, p.topology, k, g, p.grid_cols, p.W)


def step(p: Problem, X32, k: int, dense: bool = False) -> np.ndarray:
    """One iteration on float32-stored state: fp64 inside, one rounding per element."""
    X32 = np.asarray(X32, dtype=np.float32)
    return step_f64(p, X32.astype(np.float64), k, dense).astype(np.float32)


def run(p: Problem, X32, k0: int, K: int) -> np.ndarray:
    X = np.asarray(X32, dtype=np.float32)
    for k in range(k0, k0 + K):
        X = step(p, X, k)
    return X


def run_f64(p: Problem, X, k0: int, K: int) -> np.ndarray:
    X = _f64(X)
    for k in range(k0, k0 + K):
        X = step_f64(p, X, k)
    return X


def quadratic_mean_loss(X, B) -> float:
    X = _f64(X)
    B = _f64(B)
    return float(lib().gpga_oracle_quadratic_mean_loss(X.shape[0], X.shape[1], _p(X), _p(B)))


def aga_update(k, warmup_iters, H_init, F, F_init, H):
    """Algorithm 2's period update at a global-average iteration; returns (F_init, H)."""
    fi = C.c_double(F_init)
    h = C.c_int64(H)
    lib().gpga_oracle_aga_update(int(k), int(warmup_iters), int(H_init), float(F), C.byref(fi),
                                 C.byref(h))
    return fi.value, h.value


def num_threads() -> int:
    """Threads the C loops use (OpenMP default: OMP_NUM_THREADS or the affinity mask)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env.split(",")[0])
    return len(os.sched_getaffinity(0))
