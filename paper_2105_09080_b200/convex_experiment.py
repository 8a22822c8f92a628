"""The paper's convex experiment (Section 5.1) on the library: distributed logistic regression
over a ring of n = 20 / 50 / 100 nodes, d = 10, M = 8000 samples per node, non-iid data,
step size 0.2 halved every 1000 iterations, comparing parallel SGD (H = 1), Gossip SGD
(H = infinity) and Gossip-PGA (H = 16).

    python -m paper_2105_09080_b200.convex_experiment [--trials 5] [--iters 6000] [--out runs.jsonl]

Prints one JSON line per (n, method) with the global loss f(xbar) and the consensus distance
every `--every` iterations, averaged over the trials (different seeds for data order and
mini-batches).  The data recipe follows the paper; the mini-batch size, which the paper does
not state, is an option.  Everything numerical runs in the library's kernels.
"""
from __future__ import annotations

import argparse
import json
import sys

import numpy as np

from . import binding as B
from .inputs import convex_experiment_inputs

METHODS = {"parallel_sgd": 1, "gossip_sgd": 0, "gossip_pga": 16}


def run_one(A_dev, y_dev, topology, H, iters, every, batch, seed, gamma0=0.2, halve_every=1000):
    import torch
    n, m, d = A_dev.shape
    g = B.Gpga(n, d, topology, H, gamma0, seed)
    g.set_objective(B.GPGA_OBJ_LOGISTIC, l2=0.0, m=m, batch=batch)
    xa = torch.zeros((n, d), device=A_dev.device)
    g.bind(xa, torch.empty_like(xa), A_dev, y_dev)
    loss, cons = [g.global_loss()], [g.consensus_distance()]
    done = 0
    while done < iters:
        g.set_gamma(gamma0 * 0.5 ** (done // halve_every))
        next_record = min((done // every + 1) * every, iters)
        next_halving = (done // halve_every + 1) * halve_every
        step = min(next_record, next_halving) - done
        g.run(step)
        done += step
        if done == next_record:
            loss.append(g.global_loss())
            cons.append(g.consensus_distance())
    g.close()
    return np.array(loss), np.array(cons)


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--sizes", type=int, nargs="+", default=[20, 50, 100])
    ap.add_argument("--trials", type=int, default=5)
    ap.add_argument("--iters", type=int, default=6000)
    ap.add_argument("--every", type=int, default=200)
    ap.add_argument("--batch", type=int, default=8)
    ap.add_argument("--samples", type=int, default=8000)
    ap.add_argument("--iid", action="store_true")
    ap.add_argument("--topology", default="ring", choices=["ring", "grid", "static_exp"])
    ap.add_argument("--out", default="")
    args = ap.parse_args(argv)
    import torch
    if not torch.cuda.is_available():
        raise RuntimeError("the experiment needs a CUDA device (there is no CPU fallback)")
    topo = {"ring": B.GPGA_TOPO_RING, "grid": B.GPGA_TOPO_GRID, "static_exp": B.GPGA_TOPO_STATIC_EXP}[args.topology]
    sink = open(args.out, "w") if args.out else sys.stdout
    for n in args.sizes:
        A, y = convex_experiment_inputs(n, args.samples, 10, seed=1000 + n, iid=args.iid)
        A_dev, y_dev = torch.from_numpy(A).cuda(), torch.from_numpy(y).cuda()
        for name, H in METHODS.items():
            runs = [run_one(A_dev, y_dev, topo, H, args.iters, args.every, args.batch, seed=trial + 1)
                    for trial in range(args.trials)]
            loss = np.mean([r[0] for r in runs], axis=0)
            cons = np.mean([r[1] for r in runs], axis=0)
            sink.write(json.dumps({"n": n, "method": name, "H": H or "inf", "topology": args.topology,
                                   "iid": args.iid, "trials": args.trials, "batch": args.batch,
                                   "iterations": list(range(0, args.iters + 1, args.every)),
                                   "global_loss": loss.tolist(), "consensus_distance": cons.tolist()}) + "\n")
            sink.flush()
    if args.out:
        sink.close()


if __name__ == "__main__":
    main()
