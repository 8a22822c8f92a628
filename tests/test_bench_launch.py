"""`bench.py --gpus N` starts its own N ranks (one process per GPU) when it is not already under a
launcher.  Checked here without a GPU: the `--dry-run` flag keeps the launch path, the rendezvous
(gloo instead of nccl), the column-shard arithmetic, the barrier and the MAX reduction that the
timing uses, and drops the CUDA work."""
import json
import os
import subprocess
import sys
from pathlib import Path

import pytest

from paper_2105_09080_b200.sharding import weak_shard_offset

ROOT = Path(__file__).resolve().parent.parent


def _run(*flags):
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR",
                                                            "MASTER_PORT")}
    proc = subprocess.run([sys.executable, str(ROOT / "bench.py"), *flags], capture_output=True, text=True,
                          env=env, timeout=300)
    assert proc.returncode == 0, proc.stderr[-2000:]
    lines = [ln for ln in proc.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, proc.stdout          # rank 0 alone prints
    return json.loads(lines[0])


@pytest.mark.parametrize("ranks,workload,d", [(2, None, 335_141_888), (3, "c3_ring_h4", 25_557_032)])
def test_gpus_flag_starts_that_many_ranks_with_disjoint_column_shards(ranks, workload, d):
    flags = ["--gpus", str(ranks), "--dry-run"] + (["--workload", workload] if workload else [])
    line = _run(*flags)
    assert line["dry_run"] is True and line["n_gpus"] == ranks and line["scaling"] == "weak"
    shards = line["shards"]
    assert [s[0] for s in shards] == list(range(ranks))
    for r, col0, width in shards:
        assert col0 == weak_shard_offset(r, d) and width == d and col0 % 4 == 0
    ends = [col0 + width for _, col0, width in shards]
    assert all(e <= nxt[1] for e, nxt in zip(ends, shards[1:]))      # disjoint, in rank order
    assert line["max_over_ranks"] == float(ranks)                   # the slowest rank's number
    assert f"{ranks} shard(s)" in line["config"]["sharding"]


def test_single_rank_needs_no_launcher():
    line = _run("--dry-run", "--workload", "c1_ring_h4")
    assert line["n_gpus"] == 1 and line["shards"] == [[0, 0, 65_536]]
