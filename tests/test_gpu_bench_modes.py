"""The benchmark's own modes on small workloads: every mode must print one JSON line that keeps
the record's contract (metric, value, roofline with its achieved / peak / fraction, clocks sampled
during the timed region, launches counted, the end-to-end leg through the host entry)."""
import json
import subprocess
import sys
from pathlib import Path

import pytest

pytestmark = pytest.mark.gpu

ROOT = Path(__file__).resolve().parent.parent


def _bench(*flags):
    proc = subprocess.run([sys.executable, str(ROOT / "bench.py"), *flags], capture_output=True, text=True, timeout=600)
    assert proc.returncode == 0, proc.stderr[-2000:]
    lines = [ln for ln in proc.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, proc.stdout[-2000:]
    return json.loads(lines[0])


def _common(rec, steps):
    assert rec["unit"] == "node-param updates/s" and rec["value"] > 0 and rec["higher_is_better"] is True
    assert rec["n_gpus"] == 1 and rec["steps"] == steps and rec["warmup"] >= 3 and rec["data"] == "synthetic"
    assert rec["dtype"] == "f32" and rec["vs_baseline"] is None and "workload" in rec["config"]
    assert rec["gpu_launches"] >= 1
    assert set(rec["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}


def test_small_quadratic_workload_line():
    rec = _bench("--workload", "c2_exp_h8", "--steps", "16", "--warmup", "3", "--no-cpu-baseline", "--sustained-seconds", "0.2")
    _common(rec, 16)
    roof = rec["roofline"]
    assert roof["bound"] == "hbm" and roof["unit"] == "GB/s" and roof["kernel"].startswith("step_")
    assert abs(roof["frac"] - roof["achieved"] / roof["peak"]) < 1e-9 and 0.3 < roof["frac"] < 1.3
    assert rec["gpu_launches"] == 16                                   # one launch per timed step
    e2e = rec["e2e"]
    assert e2e["value"] > 0 and e2e["h2d_bytes_per_step"] > 0 and e2e["d2h_bytes_per_step"] > 0
    assert rec["gpga_run"]["launches"] == 1 and rec["gpga_run"]["iterations"] == 64   # the configuration's K in one launch


def test_logistic_workload_line():
    rec = _bench("--workload", "c5_exp_hinf", "--steps", "300", "--warmup", "3", "--no-cpu-baseline")
    _common(rec, 300)
    assert rec["roofline"]["kernel"] == "logreg_run_kernel" and rec["gpu_launches"] == 1
    assert 0.0 < rec["roofline"]["frac"] < 1.2 and rec["e2e"]["value"] > 0


@pytest.mark.parametrize("fused", [False, True])
def test_node_shard_mode_line(fused):
    flags = ["--workload", "c2_exp_h8", "--node-shards", "2", "--steps", "12", "--warmup", "3"]
    rec = _bench(*flags, *(["--fused-send"] if fused else []))
    _common(rec, 12)
    kinds = rec["per_kind"]
    assert "global" in kinds and any(k.startswith("exp_hop") for k in kinds)
    assert all(v["export_ms"] > 0 and v["step_ms"] > 0 for v in kinds.values())
    assert ("stores its messages" in rec["config"]["workload"]) == fused
