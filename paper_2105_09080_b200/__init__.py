"""B200-native Gossip-PGA iteration: a C-ABI CUDA library (libgpga.so) and its ctypes binding.

Importing the package is light; the shared library is loaded on first use and its absence
is an error (no CPU fallback).
"""
from .binding import (  # noqa: F401
    GPGA_ERR_CUDA, GPGA_ERR_INVALID_ARG, GPGA_ERR_NOT_READY, GPGA_ERR_TIMEOUT, GPGA_ERR_UNSUPPORTED, GPGA_OK,
    GPGA_OBJ_LOGISTIC, GPGA_OBJ_QUADRATIC, GPGA_TOPO_EXP, GPGA_TOPO_GRID, GPGA_TOPO_NONE,
    GPGA_TOPO_RING, GPGA_TOPO_SPARSE, GPGA_TOPO_STATIC_EXP, GPGA_X0_PER_NODE_NORMAL, GPGA_X0_SHARED_NORMAL,
    GPGA_X0_ZERO, Gpga, GpgaError, lib)
