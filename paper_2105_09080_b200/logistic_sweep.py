"""Convex logistic-regression sweep: global loss and consensus distance versus iteration.

    python -m paper_2105_09080_b200.logistic_sweep [--iters 2000] [--every 100] [--out sweep.jsonl]

Runs Gossip-PGA on the synthetic per-node logistic problem (n = 64 nodes, m = 4096 samples of
d = 1024 features, mini-batch 128, l2 = 1e-4, gamma = 0.1) over the ring and the one-peer
exponential graph with H in {1, 4, 16, 64, inf} and prints one JSON line per run with the
trajectory of f(xbar) (global loss over all samples at the node average), the consensus
distance sum_i ||x_i - xbar||^2 and the iteration throughput.  Every number comes from the
library's kernels; this script only drives the C ABI.
"""
from __future__ import annotations

import argparse
import json
import sys

from . import binding as B
from .inputs import logistic_inputs_device


def run_one(A, y, topo_name, H, iters, every, gamma=0.1, l2=1e-4, batch=128, seed=20210509):
    import torch
    n, m, d = A.shape
    topo = {"ring": B.GPGA_TOPO_RING, "exp": B.GPGA_TOPO_EXP}[topo_name]
    g = B.Gpga(n, d, topo, H, gamma, seed)
    g.set_objective(B.GPGA_OBJ_LOGISTIC, l2=l2, m=m, batch=batch)
    xa = torch.zeros((n, d), device=A.device)
    g.bind(xa, torch.empty_like(xa), A, y)
    traj = [{"k": 0, "loss": g.global_loss(), "consensus": g.consensus_distance()}]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ms = 0.0
    done = 0
    while done < iters:
        step = min(every, iters - done)
        e0.record()
        g.run(step)
        e1.record()
        torch.cuda.synchronize()
        ms += e0.elapsed_time(e1)
        done += step
        traj.append({"k": done, "loss": g.global_loss(), "consensus": g.consensus_distance()})
    out = {"topology": topo_name, "H": H or "inf", "n": n, "m": m, "d": d, "batch": batch, "gamma": gamma, "l2": l2,
           "iterations": iters, "us_per_iteration": ms / iters * 1e3,
           "node_param_updates_per_s": n * d * iters / (ms * 1e-3), "trajectory": traj}
    g.close()
    return out


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--iters", type=int, default=2000)
    ap.add_argument("--every", type=int, default=100)
    ap.add_argument("--n", type=int, default=64)
    ap.add_argument("--m", type=int, default=4096)
    ap.add_argument("--d", type=int, default=1024)
    ap.add_argument("--out", default="")
    args = ap.parse_args(argv)
    import torch
    if not torch.cuda.is_available():
        raise RuntimeError("the sweep needs a CUDA device (there is no CPU fallback)")
    A, y = logistic_inputs_device(args.n, args.m, args.d, 20210509)
    sink = open(args.out, "w") if args.out else sys.stdout
    for topo in ("ring", "exp"):
        for H in (1, 4, 16, 64, 0):
            sink.write(json.dumps(run_one(A, y, topo, H, args.iters, args.every)) + "\n")
            sink.flush()
    if args.out:
        sink.close()


if __name__ == "__main__":
    main()
