"""The paper's convex experiment (Section 5.1 and the appendix's additional experiments) on the
library: distributed logistic regression over n = 20 / 50 / 100 nodes, d = 10, M = 8000 samples
per node, step size 0.2 halved every 1000 iterations, repeated over many trials, comparing
parallel SGD (a global average every iteration), Gossip SGD (H = infinity), Gossip-PGA (H = 16)
and Local SGD (W = I between global averages), on the ring, the grid and the static exponential
graph, with non-iid or iid data.

    python -m paper_2105_09080_b200.convex_experiment [--sizes 20 50 100] [--trials 50] [--iters 6000]
           [--topology ring|grid|static_exp] [--period 16] [--iid] [--out runs.jsonl]

All trials of one (n, method) run as ONE problem: T independent copies of the n-node network are
the diagonal blocks of a (T n)-node weight matrix given to the library in CSR form (topology
SPARSE), each node with its own data, so a sweep is one launch sequence instead of T.  The
global-averaging step of Algorithm 1 is then a matrix too (1/n on every node of the same copy):
the driver hands the library the gossip matrix for the gossip iterations and the averaging matrix
for the iterations with mod(k + 1, H) = 0.  Per-trial diagnostics (the loss f(xbar) of problem (1)
at the copy's node average, and its consensus distance) come from small handles bound to each
copy's rows of the same buffers.  Everything numerical runs in the library's kernels.

Prints one JSON line per (n, method): mean and standard deviation over the trials of the loss and of
the consensus distance every `--every` iterations, the loss in excess of parallel SGD's (a paired
difference: all methods of a trial share its data and mini-batch draws) and the transient stage read
off the curves (the last recorded iteration at which that excess is still apart from zero).
The data recipe follows the paper; the mini-batch size, which the paper does not state, is an option.
"""
from __future__ import annotations

import argparse
import json
import sys

import numpy as np

from . import binding as B
from . import topologies
from .inputs import convex_experiment_inputs

# method -> (weight matrix of the gossip iterations, uses the period)
METHODS = {"parallel_sgd": ("average", False), "gossip_sgd": (None, False), "gossip_pga": (None, True),
           "local_sgd": ("none", True)}
MAX_NODES = 4096        # what topology SPARSE takes


def _to_device(arrays, device):
    import torch
    return tuple(torch.from_numpy(a).to(device) for a in arrays)


class BatchedTrials:
    """T copies of an n-node problem as one (T n)-node problem with a block-diagonal W."""

    def __init__(self, A_dev, y_dev, n, topology, batch, seed, gamma0=0.2, halve_every=1000, grid_cols=0):
        import torch
        N, m, d = A_dev.shape
        assert N % n == 0 and N <= MAX_NODES
        self.n, self.trials, self.m, self.d, self.batch = n, N // n, m, d, batch
        self.gamma0, self.halve_every = gamma0, halve_every
        self.A, self.y = A_dev, y_dev
        dev = A_dev.device
        self.W = {name: _to_device(topologies.csr(name, n, self.trials, grid_cols), dev)
                  for name in {topology, "average", "none"}}
        self.topology = topology
        self.g = B.Gpga(N, d, B.GPGA_TOPO_SPARSE, 0, gamma0, seed)
        self.g.set_objective(B.GPGA_OBJ_LOGISTIC, l2=0.0, m=m, batch=batch)
        self.xa = torch.zeros((N, d), device=dev)
        self.xb = torch.empty_like(self.xa)
        self.scratch = torch.empty(self.g.scratch_bytes(), dtype=torch.uint8, device=dev)
        self.g.bind(self.xa, self.xb, A_dev, y_dev, scratch=self.scratch)
        # one small handle per copy, for the copy's own loss and consensus distance
        self.diag = []
        for t in range(self.trials):
            h = B.Gpga(n, d, B.GPGA_TOPO_RING, 0, gamma0, seed)
            h.set_objective(B.GPGA_OBJ_LOGISTIC, l2=0.0, m=m, batch=batch)
            self.diag.append((h, torch.empty(h.scratch_bytes(), dtype=torch.uint8, device=dev)))

    def reset(self):
        self.xa.zero_()
        self.g.bind(self.xa, self.xb, self.A, self.y, scratch=self.scratch)       # x_a current, counter 0

    def diagnostics(self):
        """(loss at the node average, consensus distance) of every copy's current state."""
        cur = self.g.get_x()
        other = self.xb if cur.data_ptr() == self.xa.data_ptr() else self.xa
        n = self.n
        loss, cons = np.empty(self.trials), np.empty(self.trials)
        for t, (h, scratch) in enumerate(self.diag):
            rows = slice(t * n, (t + 1) * n)
            h.bind(cur[rows], other[rows], self.A[rows], self.y[rows], scratch=scratch)
            loss[t] = h.global_loss()
            cons[t] = h.consensus_distance()
        return loss, cons

    def run(self, method, period, iters, every):
        """Iterations 0 .. iters-1 of `method`; returns (iterations, loss[record][trial], cons[record][trial])."""
        gossip_name, periodic = METHODS[method]
        gossip = self.W[gossip_name or self.topology]
        H = period if periodic else 0
        self.reset()
        marks, loss, cons = [0], [], []
        l0, c0 = self.diagnostics()
        loss.append(l0)
        cons.append(c0)
        k = 0
        while k < iters:
            self.g.set_gamma(self.gamma0 * 0.5 ** (k // self.halve_every))
            stop = min(iters, (k // every + 1) * every, (k // self.halve_every + 1) * self.halve_every)
            if H and (k + 1) % H == 0:           # Algorithm 1: global average when mod(k + 1, H) = 0
                self.g.set_weight_matrix(*self.W["average"])
                self.g.run(1)
                k += 1
            else:
                if H:
                    stop = min(stop, (k + 1 + H - 1) // H * H - 1)     # up to the next averaging iteration
                self.g.set_weight_matrix(*gossip)
                self.g.run(stop - k)
                k = stop
            if k % every == 0 or k == iters:
                l, c = self.diagnostics()
                marks.append(k)
                loss.append(l)
                cons.append(c)
        return marks, np.array(loss), np.array(cons)

    def close(self):
        self.g.close()
        for h, _ in self.diag:
            h.close()


def excess_over(loss, reference):
    """Per record: mean and standard error over trials of loss - reference, trial by trial (the
    trials of two methods share data sets and mini-batch draws, so the difference is paired)."""
    diff = loss - reference
    return diff.mean(1), diff.std(1) / np.sqrt(diff.shape[1])


def transient_stage(marks, loss, reference):
    """Last recorded iteration at which the method's loss is still apart from the reference method's:
    the paired difference over trials is more than three standard errors from zero (and more than
    0.1 % of the reference's total decrease, so that significant but negligible gaps do not count).
    0 if never."""
    mean, sem = excess_over(loss, reference)
    ref = reference.mean(1)
    floor = 1e-3 * abs(ref[0] - ref[-1])        # and more than 0.1 % of what the reference gains over the run
    apart = (np.abs(mean) > 3.0 * sem + 1e-12) & (np.abs(mean) > floor)
    idx = np.nonzero(apart)[0]
    return int(marks[idx[-1]]) if idx.size else 0


def run_size(n, trials, iters, every, batch, samples, iid, topology, period, methods, seed=1, device="cuda"):
    """All methods for one network size; trials go in batches of at most MAX_NODES // n copies."""
    import torch
    per_batch = max(1, min(trials, MAX_NODES // n))
    out = {name: ([], [], None) for name in methods}
    done = 0
    while done < trials:
        T = min(per_batch, trials - done)
        parts = [convex_experiment_inputs(n, samples, 10, seed=1000 * n + done + t, iid=iid) for t in range(T)]
        A = torch.from_numpy(np.concatenate([p[0] for p in parts])).to(device)
        y = torch.from_numpy(np.concatenate([p[1] for p in parts])).to(device)
        bt = BatchedTrials(A, y, n, topology, batch, seed + done)
        for name in methods:
            marks, loss, cons = bt.run(name, period, iters, every)
            out[name][0].append(loss)
            out[name][1].append(cons)
            out[name] = (out[name][0], out[name][1], marks)
        bt.close()
        done += T
    return {name: (marks, np.concatenate(l, axis=1), np.concatenate(c, axis=1)) for name, (l, c, marks) in out.items()}


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--sizes", type=int, nargs="+", default=[20, 50, 100])
    ap.add_argument("--trials", type=int, default=50)
    ap.add_argument("--iters", type=int, default=6000)
    ap.add_argument("--every", type=int, default=200)
    ap.add_argument("--batch", type=int, default=8)
    ap.add_argument("--samples", type=int, default=8000)
    ap.add_argument("--period", type=int, default=16)
    ap.add_argument("--iid", action="store_true")
    ap.add_argument("--topology", default="ring", choices=["ring", "grid", "static_exp"])
    ap.add_argument("--methods", nargs="+", default=list(METHODS), choices=list(METHODS))
    ap.add_argument("--out", default="")
    args = ap.parse_args(argv)
    import torch
    if not torch.cuda.is_available():
        raise RuntimeError("the experiment needs a CUDA device (there is no CPU fallback)")
    methods = list(args.methods)
    if "parallel_sgd" not in methods:
        methods.insert(0, "parallel_sgd")        # the reference curve of the transient stage
    sink = open(args.out, "w") if args.out else sys.stdout
    for n in args.sizes:
        res = run_size(n, args.trials, args.iters, args.every, args.batch, args.samples, args.iid, args.topology,
                       args.period, methods)
        ref = res["parallel_sgd"][1]
        for name in methods:
            marks, loss, cons = res[name]
            sink.write(json.dumps({
                "n": n, "method": name, "period": args.period if METHODS[name][1] else None,
                "topology": args.topology, "iid": args.iid, "trials": args.trials, "batch": args.batch,
                "iterations": marks, "loss_mean": loss.mean(1).tolist(), "loss_std": loss.std(1).tolist(),
                "consensus_mean": cons.mean(1).tolist(), "consensus_std": cons.std(1).tolist(),
                "excess_over_parallel_sgd_mean": excess_over(loss, ref)[0].tolist(),
                "excess_over_parallel_sgd_sem": excess_over(loss, ref)[1].tolist(),
                "transient_stage": transient_stage(marks, loss, ref)}) + "\n")
            sink.flush()
    if args.out:
        sink.close()


if __name__ == "__main__":
    main()
