"""ctypes binding of libgpga: argument marshalling only.

Every step of the Gossip-PGA iteration runs in the library's CUDA kernels; this
module holds no arithmetic of the method.  PyTorch is used for device memory
and streams.  If the shared library is missing or cannot be loaded the import
of ``lib()`` raises -- there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path

PKG = Path(__file__).resolve().parent
LIB_PATH = PKG / "libgpga.so"

GPGA_OK = 0
GPGA_ERR_INVALID_ARG = 1
GPGA_ERR_NOT_READY = 2
GPGA_ERR_CUDA = 3
GPGA_ERR_UNSUPPORTED = 4
GPGA_ERR_TIMEOUT = 5

GPGA_TOPO_RING = 0
GPGA_TOPO_EXP = 1
GPGA_TOPO_GRID = 2
GPGA_TOPO_STATIC_EXP = 3
GPGA_TOPO_NONE = 4
GPGA_TOPO_SPARSE = 5

GPGA_OBJ_QUADRATIC = 0
GPGA_OBJ_LOGISTIC = 1

GPGA_X0_ZERO = 0
GPGA_X0_SHARED_NORMAL = 1
GPGA_X0_PER_NODE_NORMAL = 2

_i32, _i64, _u32, _u64, _f32 = C.c_int32, C.c_int64, C.c_uint32, C.c_uint64, C.c_float
_P = C.c_void_p

# name -> (restype, argtypes); must list every symbol include/gpga.h declares
SIGNATURES = {
    "gpga_create": (_i32, [_i64, _i64, _i32, _i64, _f32, _u64, C.POINTER(_P)]),
    "gpga_set_objective": (_i32, [_P, _i32, _f32, _f32, _i64, _i64]),
    "gpga_set_grid_cols": (_i32, [_P, _i64]),
    "gpga_set_weight_matrix": (_i32, [_P, _P, _P, _P, _i64]),
    "gpga_set_row_stride": (_i32, [_P, _i64]),
    "gpga_set_column_offset": (_i32, [_P, _i64]),
    "gpga_scratch_bytes": (_i64, [_P]),
    "gpga_bind": (_i32, [_P, _P, _P, _P, _P, _P, _i64]),
    "gpga_init_from_seed": (_i32, [_P, _i32, _f32, _f32, _P]),
    "gpga_step": (_i32, [_P, _i64, _P]),
    "gpga_run": (_i32, [_P, _i64, _P]),
    "gpga_run_host": (_i32, [_P, _P, _P, _i64, _P, _P]),
    "gpga_consensus_distance": (_i32, [_P, _P, C.POINTER(C.c_double)]),
    "gpga_mean_loss": (_i32, [_P, _P, C.POINTER(C.c_double)]),
    "gpga_global_loss": (_i32, [_P, _P, C.POINTER(C.c_double)]),
    "gpga_selftest_bounded_wait": (_i32, [_P, _P]),
    "gpga_selftest_run_wait": (_i32, [_P, _P]),
    "gpga_shard_plan": (_i32, [_i32, _i64, _i64, _i64, _i64, _i64, _i64, _P]),
    "gpga_set_node_shard": (_i32, [_P, _i64, _i64]),
    "gpga_shard_exchange_bytes": (_i64, [_P]),
    "gpga_shard_export": (_i32, [_P, _i64, _P, _P]),
    "gpga_shard_export_to": (_i32, [_P, _i64, _P, _P, _i32, _P]),
    "gpga_shard_step": (_i32, [_P, _i64, _P, _P]),
    "gpga_shard_state_sums": (_i32, [_P, _P, _P]),
    "gpga_shard_diagnostics": (_i32, [_P, _P, _P, C.POINTER(C.c_double), C.POINTER(C.c_double)]),
    "gpga_shard_step_interior": (_i32, [_P, _i64, _P]),
    "gpga_shard_step_boundary": (_i32, [_P, _i64, _P, _P]),
    "gpga_run_adaptive": (_i32, [_P, _i64, _i64, _i64, _P, C.POINTER(_i64), _i64, C.POINTER(_i64)]),
    "gpga_get_x": (_i32, [_P, C.POINTER(_P)]),
    "gpga_get_k": (_i32, [_P, C.POINTER(_i64)]),
    "gpga_set_k": (_i32, [_P, _i64]),
    "gpga_set_gamma": (_i32, [_P, _f32]),
    "gpga_set_period": (_i32, [_P, _i64]),
    "gpga_aga_update": (_i32, [_i64, _i64, _i64, C.c_double, C.POINTER(C.c_double), C.POINTER(_i64)]),
    "gpga_launch_count": (_i64, [_P]),
    "gpga_last_error": (C.c_char_p, [_P]),
    "gpga_destroy": (_i32, [_P]),
    "gpga_philox_words": (_i32, [_P, _u32, _u32, _i64, _P, _P]),
    "gpga_box_muller_words": (_i32, [_P, _P, _i64, _P, _P]),
    "gpga_normal_fill": (_i32, [_u64, _u32, _u32, _u32, _u32, _i64, _P, _P]),
    "gpga_logistic_gradient_noalloc": (_i32, [_P, _P, _P, _i64, _i64, _i64, _i64, _i64, _f32, _u64, _i64,
                                              _P, _P, C.POINTER(_i64)]),
}

GPGA_NOALLOC_SCRATCH_BYTES = 4 * 1024 * 1024

_lib = None


def lib():
    """Load libgpga.so (built in-tree by ``build.build_library``).  Fails loudly."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2105_09080_b200.build` "
                "(there is no CPU fallback)")
        L = C.CDLL(str(LIB_PATH))
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


class GpgaError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"gpga status {status}: {message}")
        self.status = status


def _stream_ptr(stream) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


class Gpga:
    """One problem instance.  Methods mirror the C entry points (gpga_<name>).

    Device memory (both X buffers, data, labels, scratch) is torch tensors that this
    object keeps alive; the library only borrows the pointers.
    """

    def __init__(self, n, d, topology, H, gamma, seed):
        self._h = _P()
        self.n, self.d = int(n), int(d)
        self.ld = int(d)
        st = lib().gpga_create(n, d, topology, H, gamma, seed, C.byref(self._h))
        if st != GPGA_OK:
            raise GpgaError(st, lib().gpga_last_error(None).decode())
        self._keep = []
        self.x_bufs = None

    # -- helpers
    def _check(self, st):
        if st != GPGA_OK:
            raise GpgaError(st, lib().gpga_last_error(self._h).decode())

    def _sp(self, stream):
        """Stream pointer for a launch; the handle's device must be the current one (the library
        launches on the current device and never switches it)."""
        dev = getattr(self, "device", None)
        if dev is not None:
            import torch
            if torch.cuda.current_device() != dev.index:
                raise GpgaError(GPGA_ERR_INVALID_ARG,
                                f"buffers live on {dev} but cuda:{torch.cuda.current_device()} is current")
        return _stream_ptr(stream)

    def close(self):
        if self._h:
            lib().gpga_destroy(self._h)
            self._h = _P()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- configuration
    def set_objective(self, objective, sigma=0.0, l2=0.0, m=0, batch=0):
        self._check(lib().gpga_set_objective(self._h, objective, sigma, l2, m, batch))

    def set_grid_cols(self, cols):
        self._check(lib().gpga_set_grid_cols(self._h, cols))

    def set_weight_matrix(self, row_ptr, col_idx, weights):
        """CSR weight matrix as torch CUDA tensors (int32, int32, float32); kept alive by this object."""
        self._w = (row_ptr, col_idx, weights)
        self._check(lib().gpga_set_weight_matrix(self._h, row_ptr.data_ptr(), col_idx.data_ptr(),
                                                 weights.data_ptr(), weights.numel()))

    def set_row_stride(self, ld):
        self._check(lib().gpga_set_row_stride(self._h, ld))
        self.ld = int(ld)

    def set_column_offset(self, col0):
        self._check(lib().gpga_set_column_offset(self._h, col0))

    def scratch_bytes(self) -> int:
        return int(lib().gpga_scratch_bytes(self._h))

    def bind(self, x_a, x_b, data, labels=None, scratch=None):
        """Bind torch CUDA tensors (float32, contiguous)."""
        import torch
        if scratch is None:
            scratch = torch.empty(self.scratch_bytes(), dtype=torch.uint8, device=x_a.device)
        for t in (x_a, x_b, data) + ((labels,) if labels is not None else ()):
            assert t.is_cuda and t.is_contiguous() and t.dtype == torch.float32
            assert t.device == x_a.device, "all buffers of one handle must live on one device"
        assert scratch.device == x_a.device, "all buffers of one handle must live on one device"
        self.device = x_a.device
        self._keep = [x_a, x_b, data, labels, scratch]
        self.x_bufs = (x_a, x_b)
        self._check(lib().gpga_bind(self._h, x_a.data_ptr(), x_b.data_ptr(), data.data_ptr(),
                                    labels.data_ptr() if labels is not None else None,
                                    scratch.data_ptr(), scratch.numel()))

    def bind_raw(self, x_a, x_b, data, labels, scratch, scratch_bytes):
        """Bind raw integer device addresses (argument checks are the library's)."""
        self._check(lib().gpga_bind(self._h, x_a, x_b, data, labels, scratch, scratch_bytes))

    def allocate(self, device="cuda"):
        """Allocate X double buffer, b (n x ld each) and scratch for the quadratic objective and bind."""
        import torch
        xa = torch.empty((self.n, self.ld), dtype=torch.float32, device=device)
        xb = torch.empty_like(xa)
        data = torch.empty_like(xa)
        self.bind(xa, xb, data)
        return xa, xb, data

    # -- the path
    def init_from_seed(self, x0_kind=GPGA_X0_ZERO, x0_std=1.0, b_shift=0.0, stream=None):
        self._check(lib().gpga_init_from_seed(self._h, x0_kind, x0_std, b_shift, self._sp(stream)))

    def step(self, k, stream=None):
        self._check(lib().gpga_step(self._h, k, self._sp(stream)))

    def run(self, K, stream=None):
        self._check(lib().gpga_run(self._h, K, self._sp(stream)))

    def run_host(self, x0_host, data_host, K, x_out_host, stream=None):
        """x0_host, data_host, x_out_host: CPU float32 torch tensors (pinned for speed); x0_host may be
        None for X^(0) = 0."""
        self._check(lib().gpga_run_host(self._h, x0_host.data_ptr() if x0_host is not None else None,
                                        data_host.data_ptr(), K,
                                        x_out_host.data_ptr(), self._sp(stream)))

    def consensus_distance(self, stream=None) -> float:
        out = C.c_double()
        self._check(lib().gpga_consensus_distance(self._h, self._sp(stream), C.byref(out)))
        return out.value

    def mean_loss(self, stream=None) -> float:
        out = C.c_double()
        self._check(lib().gpga_mean_loss(self._h, self._sp(stream), C.byref(out)))
        return out.value

    def global_loss(self, stream=None) -> float:
        out = C.c_double()
        self._check(lib().gpga_global_loss(self._h, self._sp(stream), C.byref(out)))
        return out.value

    def selftest_bounded_wait(self, stream=None):
        self._check(lib().gpga_selftest_bounded_wait(self._h, self._sp(stream)))

    def selftest_run_wait(self, stream=None):
        self._check(lib().gpga_selftest_run_wait(self._h, self._sp(stream)))

    def run_adaptive(self, K, H_init, warmup_iters, stream=None, max_periods=4096):
        periods = (_i64 * max_periods)()
        count = _i64()
        self._check(lib().gpga_run_adaptive(self._h, K, H_init, warmup_iters, self._sp(stream),
                                            periods, max_periods, C.byref(count)))
        return [int(periods[t]) for t in range(min(count.value, max_periods))]

    # -- accessors
    def get_x(self):
        """The torch tensor currently holding X (no copy)."""
        p = _P()
        self._check(lib().gpga_get_x(self._h, C.byref(p)))
        for t in self.x_bufs or ():
            if t.data_ptr() == p.value:
                return t
        return p.value

    def get_k(self) -> int:
        k = _i64()
        self._check(lib().gpga_get_k(self._h, C.byref(k)))
        return k.value

    def set_k(self, k):
        self._check(lib().gpga_set_k(self._h, k))

    def set_gamma(self, gamma):
        self._check(lib().gpga_set_gamma(self._h, gamma))

    def set_period(self, H):
        self._check(lib().gpga_set_period(self._h, H))

    def launch_count(self) -> int:
        return int(lib().gpga_launch_count(self._h))


# -- generator surface (torch CUDA tensors in, out) --------------------------------
def philox_words(ctr, key0, key1, stream=None):
    """ctr: int32/uint32-valued torch CUDA tensor of shape (count, 4) stored as int32."""
    import torch
    out = torch.empty_like(ctr)
    st = lib().gpga_philox_words(ctr.data_ptr(), key0, key1, ctr.shape[0], out.data_ptr(),
                                 _stream_ptr(stream))
    if st != GPGA_OK:
        raise GpgaError(st, lib().gpga_last_error(None).decode())
    return out


def box_muller_words(a, b, stream=None):
    import torch
    z = torch.empty((a.numel(), 2), dtype=torch.float32, device=a.device)
    st = lib().gpga_box_muller_words(a.data_ptr(), b.data_ptr(), a.numel(), z.data_ptr(),
                                     _stream_ptr(stream))
    if st != GPGA_OK:
        raise GpgaError(st, lib().gpga_last_error(None).decode())
    return z


def normal_fill(seed, stream_id, k, i, q0, count, device="cuda", stream=None):
    import torch
    out = torch.empty((count, 4), dtype=torch.float32, device=device)
    st = lib().gpga_normal_fill(seed, stream_id, k, i, q0, count, out.data_ptr(), _stream_ptr(stream))
    if st != GPGA_OK:
        raise GpgaError(st, lib().gpga_last_error(None).decode())
    return out


def logistic_gradient_noalloc(A, y, x, batch, l2, seed, k, out=None, stream=None):
    """Mini-batch logistic gradient matrix without any device allocation by the library.

    For callers that cannot allocate device memory themselves at the point of the call
    (no-sync loops, plug-ins that only receive tensors): the library's built-in scratch
    array holds the intermediate partial sums.  A (n, m, d), y (n, m), x (n, d or a view
    with a row stride) and `out` (n, d) are the caller's CUDA tensors; `out` must be given
    by such callers (it is only created here as a convenience when omitted).  Returns
    (status, needed_scratch_bytes, out); the status is GPGA_ERR_UNSUPPORTED when the
    problem needs more than GPGA_NOALLOC_SCRATCH_BYTES.  Calls sharing a device must not
    overlap on the GPU; make the first call on a device outside stream capture.
    """
    import torch
    n, m, d = A.shape
    if out is None:
        out = torch.empty((n, d), dtype=torch.float32, device=A.device)
    # the library runs on the current device with that device's scratch array: all tensors must
    # live on one device, which is made current for the call
    devices = {t.device for t in (A, y, x, out)}
    if len(devices) != 1 or not A.is_cuda:
        raise ValueError(f"A, y, x and out must be CUDA tensors on one device, got {sorted(map(str, devices))}")
    need = _i64()
    with torch.cuda.device(A.device):
        st = lib().gpga_logistic_gradient_noalloc(A.data_ptr(), y.data_ptr(), x.data_ptr(), x.stride(0), n, d, m,
                                                  batch, l2, seed, k, out.data_ptr(), _stream_ptr(stream),
                                                  C.byref(need))
    return st, int(need.value), out
