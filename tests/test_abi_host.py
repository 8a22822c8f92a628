"""Host-side checks of the C ABI that need no GPU: the library loads, exports every
symbol the header declares, and rejects bad arguments before touching CUDA."""
import ctypes as C
import re
from pathlib import Path

import pytest

import paper_2105_09080_b200 as pkg
from paper_2105_09080_b200 import binding, build

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def L():
    build.build_library()
    return pkg.lib()


def _declared_symbols():
    text = (ROOT / "include" / "gpga.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gpga_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(L):
    names = _declared_symbols()
    assert len(names) >= 20
    for name in names:
        assert hasattr(L, name), name
    # and the binding lists a signature for each of them
    assert sorted(binding.SIGNATURES) == names


def test_missing_library_is_an_error(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", tmp_path / "nope.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.lib()


def _create(L, n=8, d=64, topo=0, H=4, gamma=0.1, seed=1):
    h = C.c_void_p()
    st = L.gpga_create(n, d, topo, H, gamma, seed, C.byref(h))
    return st, h


def test_create_argument_checks(L):
    st, h = _create(L)
    assert st == pkg.GPGA_OK and h.value
    assert L.gpga_destroy(h) == pkg.GPGA_OK
    for kw in (dict(n=0), dict(d=0), dict(H=-1), dict(gamma=-0.1), dict(gamma=float("nan")),
               dict(gamma=float("inf")), dict(topo=9), dict(topo=-1), dict(n=2**31), dict(d=2**34)):
        st, h = _create(L, **kw)
        assert st == pkg.GPGA_ERR_INVALID_ARG, kw
        assert not h.value
        assert L.gpga_last_error(None)
    st, h = _create(L, n=12, topo=pkg.GPGA_TOPO_EXP)
    assert st == pkg.GPGA_ERR_UNSUPPORTED
    st, h = _create(L, n=12, topo=pkg.GPGA_TOPO_STATIC_EXP)
    assert st == pkg.GPGA_ERR_UNSUPPORTED
    assert L.gpga_create(8, 8, 0, 0, 0.1, 1, None) == pkg.GPGA_ERR_INVALID_ARG
    assert L.gpga_destroy(None) == pkg.GPGA_OK


def test_not_ready_and_setter_checks(L):
    st, h = _create(L)
    assert L.gpga_step(h, 0, None) == pkg.GPGA_ERR_NOT_READY
    assert L.gpga_run(h, 3, None) == pkg.GPGA_ERR_NOT_READY
    out = C.c_double()
    assert L.gpga_consensus_distance(h, None, C.byref(out)) == pkg.GPGA_ERR_NOT_READY
    assert b"bind" in L.gpga_last_error(h)
    assert L.gpga_step(None, 0, None) == pkg.GPGA_ERR_NOT_READY
    assert L.gpga_set_k(h, -1) == pkg.GPGA_ERR_INVALID_ARG
    assert L.gpga_set_k(h, 2**32) == pkg.GPGA_ERR_INVALID_ARG
    assert L.gpga_set_k(h, 5) == pkg.GPGA_OK
    k = C.c_int64()
    assert L.gpga_get_k(h, C.byref(k)) == pkg.GPGA_OK and k.value == 5
    assert L.gpga_set_gamma(h, float("nan")) == pkg.GPGA_ERR_INVALID_ARG
    assert L.gpga_set_gamma(h, 0.05) == pkg.GPGA_OK
    assert L.gpga_set_period(h, -2) == pkg.GPGA_ERR_INVALID_ARG
    assert L.gpga_set_period(h, 0) == pkg.GPGA_OK
    assert L.gpga_set_column_offset(h, 6) == pkg.GPGA_ERR_INVALID_ARG
    assert L.gpga_set_column_offset(h, -4) == pkg.GPGA_ERR_INVALID_ARG
    assert L.gpga_set_column_offset(h, 2**34) == pkg.GPGA_ERR_INVALID_ARG
    assert L.gpga_set_column_offset(h, 1024) == pkg.GPGA_OK
    assert L.gpga_set_row_stride(h, 63) == pkg.GPGA_ERR_INVALID_ARG
    assert L.gpga_set_row_stride(h, 96) == pkg.GPGA_OK
    assert L.gpga_set_grid_cols(h, 3) == pkg.GPGA_ERR_INVALID_ARG
    assert L.gpga_set_grid_cols(h, 4) == pkg.GPGA_OK
    assert L.gpga_launch_count(h) == 0
    p = C.c_void_p()
    assert L.gpga_get_x(h, C.byref(p)) == pkg.GPGA_ERR_NOT_READY
    L.gpga_destroy(h)


def test_objective_and_bind_checks(L):
    st, h = _create(L, n=4, d=64)
    assert L.gpga_set_objective(h, 0, -1.0, 0.0, 0, 0) == pkg.GPGA_ERR_INVALID_ARG
    assert L.gpga_set_objective(h, 7, 0.0, 0.0, 0, 0) == pkg.GPGA_ERR_INVALID_ARG
    assert L.gpga_set_objective(h, 1, 0.0, 1e-4, 0, 8) == pkg.GPGA_ERR_INVALID_ARG     # m < 1
    assert L.gpga_set_objective(h, 1, 0.0, 1e-4, 16, 0) == pkg.GPGA_ERR_INVALID_ARG    # batch < 1
    assert L.gpga_set_objective(h, 1, 0.0, -1.0, 16, 8) == pkg.GPGA_ERR_INVALID_ARG
    quad_bytes = L.gpga_scratch_bytes(h)
    assert quad_bytes >= 148 * 8 * 8
    assert L.gpga_set_objective(h, 1, 0.0, 1e-4, 16, 40) == pkg.GPGA_OK
    # logistic scratch adds G (n d floats) and ceil(40/32) = 2 chunk partials
    assert L.gpga_scratch_bytes(h) >= quad_bytes + 3 * 4 * 64 * 4
    assert L.gpga_set_objective(h, 0, 0.1, 0.0, 0, 0) == pkg.GPGA_OK
    nbytes = L.gpga_scratch_bytes(h)
    a, b, c, s = 0x10000, 0x20000, 0x30000, 0x40000       # fake aligned addresses, never dereferenced
    assert L.gpga_bind(h, None, b, c, None, s, nbytes) == pkg.GPGA_ERR_INVALID_ARG
    assert L.gpga_bind(h, a, a + 16, c, None, s, nbytes) == pkg.GPGA_ERR_INVALID_ARG   # partial overlap
    assert L.gpga_bind(h, a, a, c, None, s, nbytes) == pkg.GPGA_OK                     # in-place update
    assert L.gpga_bind(h, a + 4, b, c, None, s, nbytes) == pkg.GPGA_ERR_INVALID_ARG
    assert L.gpga_bind(h, a, b, c, None, s, nbytes - 1) == pkg.GPGA_ERR_INVALID_ARG
    assert L.gpga_bind(h, a, b, c, None, s, nbytes) == pkg.GPGA_OK
    assert L.gpga_set_objective(h, 0, 0.2, 0.0, 0, 0) == pkg.GPGA_ERR_INVALID_ARG      # after bind
    assert L.gpga_set_row_stride(h, 128) == pkg.GPGA_ERR_INVALID_ARG                   # after bind
    assert L.gpga_step(h, -1, None) == pkg.GPGA_ERR_INVALID_ARG
    assert L.gpga_step(h, 2**32, None) == pkg.GPGA_ERR_INVALID_ARG
    assert L.gpga_run(h, -1, None) == pkg.GPGA_ERR_INVALID_ARG
    assert L.gpga_run(h, 0, None) == pkg.GPGA_OK                                      # no launch
    assert L.gpga_run_host(h, None, None, 1, None, None) == pkg.GPGA_ERR_INVALID_ARG
    assert L.gpga_consensus_distance(h, None, None) == pkg.GPGA_ERR_INVALID_ARG
    assert L.gpga_global_loss(h, None, None) == pkg.GPGA_ERR_INVALID_ARG
    assert L.gpga_run_adaptive(h, 4, 0, 0, None, None, 0, None) == pkg.GPGA_ERR_INVALID_ARG
    L.gpga_destroy(h)
    # logistic objective needs labels at bind, and d % 4 == 0
    st, h = _create(L, n=4, d=64)
    assert L.gpga_set_objective(h, 1, 0.0, 1e-4, 16, 8) == pkg.GPGA_OK
    assert L.gpga_bind(h, a, b, c, None, s, L.gpga_scratch_bytes(h)) == pkg.GPGA_ERR_INVALID_ARG
    L.gpga_destroy(h)
    st, h = _create(L, n=4, d=66)
    assert L.gpga_set_objective(h, 1, 0.0, 1e-4, 16, 8) == pkg.GPGA_ERR_UNSUPPORTED
    L.gpga_destroy(h)


def test_generator_surface_argument_checks(L):
    assert L.gpga_philox_words(None, 0, 0, 4, None, None) == pkg.GPGA_ERR_INVALID_ARG
    assert L.gpga_box_muller_words(None, None, -1, None, None) == pkg.GPGA_ERR_INVALID_ARG
    assert L.gpga_normal_fill(1, 0, 0, 0, 0, 8, None, None) == pkg.GPGA_ERR_INVALID_ARG


def test_noalloc_entry_point_checks_arguments_before_any_launch(L):
    """Sizes are judged first (no CUDA call), then the pointers are looked up: addresses that are
    not the current device's memory -- or no device at all, as on a CPU-only box -- end the call
    with a status and nothing is launched."""
    a, y, x, g = 0x10000, 0x20000, 0x30000, 0x40000       # fake aligned addresses, never dereferenced
    need = C.c_int64(-1)
    call = L.gpga_logistic_gradient_noalloc
    assert call(a, y, x, 64, 4, 64, 16, 8, 0.0, 1, 0, g + 4, None, C.byref(need)) == pkg.GPGA_ERR_INVALID_ARG
    assert call(a, y, x, 60, 4, 64, 16, 8, 0.0, 1, 0, g, None, C.byref(need)) == pkg.GPGA_ERR_INVALID_ARG   # ldx < d
    assert call(a, y, x, 64, 4, 66, 16, 8, 0.0, 1, 0, g, None, C.byref(need)) == pkg.GPGA_ERR_INVALID_ARG   # d % 4
    assert call(a, y, x, 64, 4, 64, 16, 8, -1.0, 1, 0, g, None, C.byref(need)) == pkg.GPGA_ERR_INVALID_ARG
    assert call(a, y, x, 64, 4, 64, 16, 8, 0.0, 1, -1, g, None, C.byref(need)) == pkg.GPGA_ERR_INVALID_ARG
    # too large for the built-in scratch: refused with the need reported, before any CUDA call
    assert call(a, y, x, 4096, 64, 4096, 64, 256, 0.0, 1, 0, g, None, C.byref(need)) == pkg.GPGA_ERR_UNSUPPORTED
    assert need.value == 8 * 64 * 4096 * 4 > binding.GPGA_NOALLOC_SCRATCH_BYTES
    # sizes fine, pointers not device memory of a current device
    st = call(a, y, x, 64, 4, 64, 16, 8, 0.0, 1, 0, g, None, C.byref(need))
    assert st in (pkg.GPGA_ERR_INVALID_ARG, pkg.GPGA_ERR_CUDA)
    assert need.value == 1 * 4 * 64 * 4


def test_header_is_plain_c_and_a_c_program_links_against_the_library(tmp_path, L):
    """include/gpga.h compiles as C99 and as C++, and a C program that only includes it can create and
    destroy a handle and read the exchange plan through the shared library (no CUDA device needed)."""
    import shutil
    import subprocess
    header = ROOT / "include" / "gpga.h"
    if not shutil.which("gcc"):
        pytest.skip("no C compiler")
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-fsyntax-only", "-x", "c", str(header)],
                   check=True)
    if shutil.which("g++"):
        subprocess.run(["g++", "-std=c++11", "-fsyntax-only", "-x", "c++", str(header)], check=True)
    src = tmp_path / "use.c"
    src.write_text('#include <stdio.h>\n#include "gpga.h"\n'
                   'int main(void) {\n'
                   '    gpga_t* h = 0;\n'
                   '    if (gpga_create(8, 64, GPGA_TOPO_RING, 4, 0.1f, 1u, &h) != GPGA_OK) return 1;\n'
                   '    if (gpga_step(h, 0, 0) != GPGA_ERR_NOT_READY) return 2;\n'
                   '    gpga_shard_plan_t plan;\n'
                   '    if (gpga_shard_plan(GPGA_TOPO_EXP, 0, 16, 2, 0, 40, 3, &plan) != GPGA_OK) return 3;\n'
                   '    printf("%d %lld %lld\\n", (int)plan.kind, (long long)plan.hop, (long long)plan.bytes[0]);\n'
                   '    return gpga_destroy(h);\n}\n')
    exe = tmp_path / "use"
    lib = binding.LIB_PATH
    subprocess.run(["gcc", "-std=c99", "-I", str(header.parent), str(src), "-o", str(exe), str(lib),
                    f"-Wl,-rpath,{lib.parent}", "-lstdc++", "-lm", "-ldl", "-lpthread", "-lrt"], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()
    assert out == ["1", "8", str(8 * 40 * 4)]
