"""Are the oracle's pins sharp?  Each case plants one plausible mistake in a COPY of the oracle's C
source (a wrong sign, index, constant or predicate), builds it, and requires that at least one pin
of tests/test_oracle_pins.py fails against the broken copy.  CPU only; the real oracle and the
CUDA path are untouched."""
import subprocess
from pathlib import Path

import pytest

from oracle import gpga_oracle as o
import test_oracle_pins as pins

SRC = Path(o.__file__).resolve().parent / "gpga_oracle.c"

# (name, text in the oracle source, replacement)
MUTATIONS = [
    ("local_update_sign", "Y[i * dloc + j] = x - gamma * g;", "Y[i * dloc + j] = x + gamma * g;"),
    ("noise_sign", "double g = (x - B[i * dloc + j]) + sigma * xi;", "double g = (x - B[i * dloc + j]) - sigma * xi;"),
    ("gradient_target_sign", "double g = (x - B[i * dloc + j]) + sigma * xi;", "double g = (x + B[i * dloc + j]) + sigma * xi;"),
    ("gamma_dropped", "Y[i * dloc + j] = x - gamma * g;", "Y[i * dloc + j] = x - g;"),
    ("ring_neighbour_index", "int64_t up = (i + n - 1) % n, dn = (i + 1) % n;", "int64_t up = (i + n - 2) % n, dn = (i + 1) % n;"),
    ("ring_weight", "+ Y[dn * d + j]) / 3.0;", "+ Y[dn * d + j]) / 2.0;"),
    ("ring_self_term_dropped", "(Y[up * d + j] + Y[i * d + j] + Y[dn * d + j]) / 3.0", "(Y[up * d + j] + Y[up * d + j] + Y[dn * d + j]) / 3.0"),
    ("exp_peer_index", "int64_t p = (i + hop) % n;", "int64_t p = (i + hop + 1) % n;"),
    ("exp_hop_schedule", "return (int64_t)1 << (k % tau);", "return (int64_t)1 << ((k + 1) % tau);"),
    ("exp_weight", "Z[i * d + j] = (Y[i * d + j] + Y[p * d + j]) / 2.0;", "Z[i * d + j] = (Y[i * d + j] + 2.0 * Y[p * d + j]) / 3.0;"),
    ("global_predicate_off_by_one", "return (H > 0 && ((k + 1) % H) == 0) ? 1 : 0;", "return (H > 0 && (k % H) == 0) ? 1 : 0;"),
    ("global_mean_divisor", "double m = s / (double)n;", "double m = s / (double)(n + 1);"),
    ("philox_multiplier", "(uint64_t)0xD2511F53u * (uint64_t)c0", "(uint64_t)0xD2511F54u * (uint64_t)c0"),
    ("philox_key_schedule", "k1 += 0xBB67AE85u;", "k1 += 0xBB67AE84u;"),
    ("philox_rounds", "round < 10; ++round", "round < 9; ++round"),
    ("philox_word_order", "c0 = n0; c1 = n1; c2 = n2; c3 = n3;", "c0 = n2; c1 = n1; c2 = n0; c3 = n3;"),
    ("box_muller_radius", "double r = sqrt(-2.0 * log(u1));", "double r = sqrt(-1.0 * log(u1));"),
    ("box_muller_sin_cos_swapped", "z[0] = r * cos(two_pi * u2);\n    z[1] = r * sin(two_pi * u2);", "z[0] = r * sin(two_pi * u2);\n    z[1] = r * cos(two_pi * u2);"),
    ("uniform_offset_dropped", "double u1 = ((double)(a >> 8) + 1.0) / 16777216.0;", "double u1 = ((double)(a >> 8) + 0.5) / 16777216.0;"),
    ("noise_counter_words_swapped", "uint32_t ctr[4] = {q, i, k, stream};", "uint32_t ctr[4] = {i, q, k, stream};"),
    ("consensus_not_squared", "total += dev * dev;", "total += fabs(dev);"),
    ("consensus_mean_divisor", "double mean = s / (double)n;\n        for (int64_t i = 0; i < n; ++i) {\n            double dev", "double mean = s / (double)(n - 1);\n        for (int64_t i = 0; i < n; ++i) {\n            double dev"),
    ("logistic_gradient_sign", "double s = -y[r] / (1.0 + exp(y[r] * z));", "double s = y[r] / (1.0 + exp(y[r] * z));"),
    ("logistic_gradient_sigmoid_argument", "double s = -y[r] / (1.0 + exp(y[r] * z));", "double s = -y[r] / (1.0 + exp(-y[r] * z));"),
    ("logistic_loss_sign", "double t = -y[r] * z;", "double t = y[r] * z;"),
    ("logistic_l2_dropped", "g[j] = g[j] / (double)count + l2 * x[j];", "g[j] = g[j] / (double)count;"),
    ("batch_word_selection", "idx[t] = (int32_t)(w[t & 3] % (uint32_t)m);", "idx[t] = (int32_t)(w[0] % (uint32_t)m);"),
    ("aga_floor_instead_of_ceil", "*H = (int64_t)ceil((*F_init / F) * (double)H_init);", "*H = (int64_t)floor((*F_init / F) * (double)H_init);"),
    ("aga_warmup_average", "*F_init = 0.5 * (*F_init + F);", "*F_init = F;"),
    ("init_shift_sign", "col0 + j) + shift * s;", "col0 + j) - shift * s;"),
    ("init_x0_shared_uses_node_index", "if (kind == 1) v = std * normal_at(seed, ORACLE_STREAM_X0, 0u, 0u, col0 + j);", "if (kind == 1) v = std * normal_at(seed, ORACLE_STREAM_X0, 0u, (uint32_t)i, col0 + j);"),
    ("grid_neighbour", "int64_t lf = a * c + (b + c - 1) % c, rt = a * c + (b + 1) % c;", "int64_t lf = a * c + (b + c - 1) % c, rt = a * c + (b + 2) % c;"),
    ("static_exp_weight", "Z[i * d + j] = s / (double)(tau + 1);", "Z[i * d + j] = s / (double)tau;"),
]


def _pin_calls():
    """Every pin of test_oracle_pins.py as (name, callable), parametrised ones expanded."""
    calls = []
    for name, fn in sorted(vars(pins).items()):
        if not name.startswith("test_") or not callable(fn):
            continue
        marks = [m for m in getattr(fn, "pytestmark", []) if m.name == "parametrize"]
        if not marks:
            calls.append((name, fn, ()))
            continue
        assert len(marks) == 1
        for value in marks[0].args[1]:
            args = value if isinstance(value, (tuple, list)) else (value,)
            calls.append((name, fn, tuple(args)))
    # the slow statistical pin last
    calls.sort(key=lambda c: c[0] == "test_normals_are_standard_normal")
    return calls


def _first_failing_pin():
    for name, fn, args in _pin_calls():
        try:
            fn(*args)
        except Exception:      # an assertion, or numerics gone wrong (inf/nan) inside a pin
            return name
    return None


def test_the_intact_oracle_passes_every_pin():
    assert _first_failing_pin() is None


@pytest.mark.parametrize("name,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_planted_mistake_is_caught_by_a_pin(name, old, new, tmp_path, monkeypatch):
    text = SRC.read_text()
    assert text.count(old) >= 1, f"mutation target for {name} not found in the oracle source"
    broken_c = tmp_path / "broken.c"
    broken_so = tmp_path / "broken.so"
    broken_c.write_text(text.replace(old, new, 1))
    subprocess.run(["gcc", "-O1", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
                    str(broken_c), "-o", str(broken_so), "-lm"], check=True)
    o.lib()                                            # make sure the real one is loaded first
    monkeypatch.setattr(o, "_lib", o.load(broken_so))
    caught_by = _first_failing_pin()
    assert caught_by is not None, f"no pin noticed the planted mistake '{name}'"
