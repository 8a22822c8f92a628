#!/usr/bin/env python
"""Benchmark of the Gossip-PGA iteration (libgpga) on B200.

A "step" is one iteration of Algorithm 1 over the whole n x d state: the fused
local-update + gossip kernel, or the fused local-update + global-average kernel on
every H-th iteration.  Prints one JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c4_exp_h4] [--impl reference]
    python bench.py --workload c3_ring_h4 --node-shards 4      # one shard's kernels of the node-sharded mode
    python bench.py --workload c3_ring_h4 --node-shards 4 --fused-send   # ... with the export kernel storing the messages itself

Default workload: the BERT-Large-sized configuration (n = 16, d = 335,141,888, one-peer
exponential graph, H = 4; 64.35 GB per step), or the ResNet-50-sized ring configuration when
three 21.45 GB buffers do not fit the device; `config.workload` says which.  Beside the
headline the line carries one roofline cell per target kernel and size (`cells`), a
seconds-long loop with the sampled clocks (`sustained`), and one gpga_run call.

Multi-GPU: the state is sharded by columns (columns evolve independently), one
process per GPU, no data-path collective; every rank holds a full-width shard of a
problem N times wider (weak scaling).  `--gpus N` without a torchrun environment starts
the N ranks itself.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import socket
import subprocess
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

METRIC = "Gossip-PGA node-param updates/s and HBM GB/s vs B200 peak (fp32, 1 GPU)"
UNIT = "node-param updates/s"
SEED = 20210509
BYTES_PER_UPDATE = 12          # read X (4) + read b (4) + write X+ (4); the noise never touches HBM

# name: n, d, topology, H, gamma, sigma, K (the configuration's own run length), x0 kind, x0 std, b shift
WORKLOADS = {
    "c1_ring_h4": dict(n=8, d=65_536, topo="ring", H=4, gamma=0.1, sigma=0.1, K=32, x0="zero", x0_std=1.0, b_shift=0.0),
    "c2_exp_h8": dict(n=32, d=1_048_576, topo="exp", H=8, gamma=0.05, sigma=0.1, K=64, x0="zero", x0_std=1.0, b_shift=0.0),
    "c3_ring_h4": dict(n=64, d=25_557_032, topo="ring", H=4, gamma=0.01, sigma=0.01, K=50, x0="shared", x0_std=0.1, b_shift=0.5),
    "c3_ring_h2": dict(n=64, d=25_557_032, topo="ring", H=2, gamma=0.01, sigma=0.01, K=50, x0="shared", x0_std=0.1, b_shift=0.5),
    "c3_ring_h16": dict(n=64, d=25_557_032, topo="ring", H=16, gamma=0.01, sigma=0.01, K=50, x0="shared", x0_std=0.1, b_shift=0.5),
    "c3_ring_hinf": dict(n=64, d=25_557_032, topo="ring", H=0, gamma=0.01, sigma=0.01, K=50, x0="shared", x0_std=0.1, b_shift=0.5),
    "c3_exp_h4": dict(n=64, d=25_557_032, topo="exp", H=4, gamma=0.01, sigma=0.01, K=50, x0="shared", x0_std=0.1, b_shift=0.5),
    "c3_exp_h16": dict(n=64, d=25_557_032, topo="exp", H=16, gamma=0.01, sigma=0.01, K=50, x0="shared", x0_std=0.1, b_shift=0.5),
    "c3_exp_hinf": dict(n=64, d=25_557_032, topo="exp", H=0, gamma=0.01, sigma=0.01, K=50, x0="shared", x0_std=0.1, b_shift=0.5),
    "c3_global_h1": dict(n=64, d=25_557_032, topo="ring", H=1, gamma=0.01, sigma=0.01, K=50, x0="shared", x0_std=0.1, b_shift=0.5),
    # reduced-width copies of c3 / c4 (same n, same ragged d mod 128) for profiler captures
    "c3s_ring_h4": dict(n=64, d=2_097_192, topo="ring", H=4, gamma=0.01, sigma=0.01, K=50, x0="shared", x0_std=0.1, b_shift=0.5),
    "c3s_exp_h4": dict(n=64, d=2_097_192, topo="exp", H=4, gamma=0.01, sigma=0.01, K=50, x0="shared", x0_std=0.1, b_shift=0.5),
    "c4s_exp_h4": dict(n=16, d=8_388_608, topo="exp", H=4, gamma=0.01, sigma=0.01, K=20, x0="zero", x0_std=1.0, b_shift=0.0),
    "c4_exp_h4": dict(n=16, d=335_141_888, topo="exp", H=4, gamma=0.01, sigma=0.01, K=20, x0="zero", x0_std=1.0, b_shift=0.0),
    "c4_global_h1": dict(n=16, d=335_141_888, topo="exp", H=1, gamma=0.01, sigma=0.01, K=20, x0="zero", x0_std=1.0, b_shift=0.0),
}
# convex logistic-regression workload (n = 64 nodes, 4096 local samples of 1024 features, batch 128)
for _topo in ("ring", "exp"):
    for _H in (1, 4, 16, 64, 0):
        WORKLOADS[f"c5_{_topo}_h{_H or 'inf'}"] = dict(objective="logistic", n=64, d=1024, m=4096, batch=128, l2=1e-4,
                                                        topo=_topo, H=_H, gamma=0.1, K=2000)
DEFAULT_WORKLOAD = "c4_exp_h4"        # the largest single-GPU configuration
FALLBACK_WORKLOAD = "c3_ring_h4"      # when three n x d buffers of the default do not fit the device
NOMINAL_PEAK_GBS = 8000.0             # the HBM3e figure the 75 % target is quoted against

# DRAM bytes per launch of the dominant kernel from an ncu capture (dram__bytes_read.sum +
# dram__bytes_write.sum), as a multiple of the algorithmic bytes of the captured launch, with
# the digest of the kernel sources at capture time.  A changed source voids it (-> null).
NCU_TRAFFIC = {
    # kernel name: (traffic / algorithmic bytes, source digest); captured at n=64, d=2,097,192 and
    # n=16, d=8,388,608 -- one pass over three n x d arrays, so traffic scales with n x d
    "step_ring_kernel": (0.977, "85dfc7d0ebc759b5"),
    "step_exp_kernel": (0.975, "85dfc7d0ebc759b5"),
    "step_global_kernel": (0.968, "85dfc7d0ebc759b5"),
}


def kernel_source_digest() -> str:
    h = hashlib.sha256()
    for name in ("gpga_device.cuh", "gpga_kernels.cuh", "gpga_kernels.cu"):
        h.update((ROOT / "paper_2105_09080_b200" / "csrc" / name).read_bytes())
    return h.hexdigest()[:16]


def measured_peak_gbs():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return float(json.loads(p.read_text())["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons through NVML (read-only) while a timed region runs.
    One thread for the whole run; `begin()` opens a section, `end()` closes it and returns its summary."""

    def __init__(self, index: int, period_s: float = 0.005):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._halt = threading.Event()
        self.active = threading.Event()
        self.ready = threading.Event()
        self.once = threading.Event()      # one more sample, asked for by end() when a region was too short for any
        self.error = None

    def run(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
            names = {}
            for attr in dir(nv):
                if attr.startswith("nvmlClocksEventReason") or attr.startswith("nvmlClocksThrottleReason"):
                    v = getattr(nv, attr)
                    if isinstance(v, int) and v and attr not in ("nvmlClocksEventReasonAll", "nvmlClocksThrottleReasonAll"):
                        names.setdefault(v, attr.replace("nvmlClocksEventReason", "").replace("nvmlClocksThrottleReason", ""))
            get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                nv.nvmlDeviceGetCurrentClocksThrottleReasons
            self.ready.set()
            while not self._halt.is_set():
                if self.active.is_set() or self.once.is_set():
                    mhz = nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)
                    mask = get_reasons(h)
                    if self.active.is_set() or self.once.is_set():
                        self.samples.append(mhz)
                        for bit, nm in names.items():
                            if mask & bit and bit.bit_count() == 1:
                                self.reasons.add(nm)
                    self.once.clear()
                time.sleep(self.period)
            nv.nvmlShutdown()
        except Exception as exc:          # NVML missing: report it, do not fail the run
            self.error = repr(exc)
            self.ready.set()

    def begin(self):
        if not self.is_alive() and not self._halt.is_set():
            self.start()
            self.ready.wait(timeout=5)
        self.samples, self.reasons = [], set()
        self.active.set()

    def end(self):
        self.active.clear()
        if not self.samples and self.is_alive() and not self.error:
            # the region ended before the first sample: take one now, the work has only just drained
            self.once.set()
            t0 = time.time()
            while self.once.is_set() and time.time() - t0 < 0.5:
                time.sleep(0.001)
        s = sorted(self.samples)
        return {"sm_mhz": (s[len(s) // 2] if s else None), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(r for r in self.reasons if r not in ("GpuIdle", "None")),
                "samples": len(s), **({"error": self.error} if self.error else {})}

    def finish(self):
        self._halt.set()
        if self.is_alive():
            self.join(timeout=2)


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


# ---------------------------------------------------------------------------------
# CPU baseline: the oracle as it stands, on a bounded column slice of the workload
# ---------------------------------------------------------------------------------
def oracle_sample(w, cols, iters, k0=0):
    """Run `iters` oracle iterations on a `cols`-column slice (all n rows); returns seconds."""
    import numpy as np
    from oracle import gpga_oracle as o
    topo = {"ring": o.TOPO_RING, "exp": o.TOPO_EXP}[w["topo"]]
    kind = {"zero": o.X0_ZERO, "shared": o.X0_SHARED_NORMAL}[w["x0"]]
    B = o.init_b(w["n"], cols, SEED, w["b_shift"]).astype(np.float32)
    X = o.init_x0(w["n"], cols, SEED, kind, w["x0_std"]).astype(np.float32)
    p = o.Problem(topo, w["H"], w["gamma"], SEED, sigma=w["sigma"], data=B)
    t0 = time.perf_counter()
    o.run(p, X, k0, iters)
    return time.perf_counter() - t0


def cpu_baseline(w, target_s=12.0):
    from oracle import gpga_oracle as o
    iters = max(w["H"], 1) if w["H"] else 4        # one averaging period (or four gossip steps)
    probe_cols = 4096
    t = oracle_sample(w, probe_cols, iters)
    rate = w["n"] * probe_cols * iters / t
    cols = int(min(w["d"], max(probe_cols, target_s * rate / (w["n"] * iters))))
    cols -= cols % 4
    t = oracle_sample(w, cols, iters)
    return {"value": w["n"] * cols * iters / t, "unit": UNIT, "cores": o.num_threads(), "kind": "oracle",
            "sample": f"{iters} iterations (k=0..{iters - 1}) on the first {cols} of {w['d']} columns, all "
                      f"{w['n']} rows, {t:.1f} s; columns are independent so throughput scales linearly in d"}


def run_reference(args, w, name, choice=None):
    """--impl reference: the oracle on the host cores; each step = one iteration on a bounded slice."""
    from oracle import gpga_oracle as o
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    # each step is a bounded sample sized so that warm-up + timed steps take about a minute in all
    per_step_s = min(1.0, 60.0 / max(1, args.steps + args.warmup))
    t = oracle_sample(w, 4096, 1)
    cols = int(min(w["d"], max(4096, per_step_s * 4096 / t)))
    cols -= cols % 4
    import numpy as np
    topo = {"ring": o.TOPO_RING, "exp": o.TOPO_EXP}[w["topo"]]
    kind = {"zero": o.X0_ZERO, "shared": o.X0_SHARED_NORMAL}[w["x0"]]
    B = o.init_b(w["n"], cols, SEED, w["b_shift"]).astype(np.float32)
    X = o.init_x0(w["n"], cols, SEED, kind, w["x0_std"]).astype(np.float32)
    p = o.Problem(topo, w["H"], w["gamma"], SEED, sigma=w["sigma"], data=B)
    k = 0
    for _ in range(args.warmup):
        X = o.step(p, X, k)
        k += 1
    t0 = time.perf_counter()
    for _ in range(args.steps):
        X = o.step(p, X, k)
        k += 1
    dt = time.perf_counter() - t0
    value = w["n"] * cols * args.steps / dt
    sample = (f"each step = one iteration on the first {cols} of {w['d']} columns, all {w['n']} rows "
              f"(columns are independent)")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_config(name, w, args.gpus, choice),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": o.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def padded_stride(d):
    return (d + 31) // 32 * 32


def workload_config(name, w, n_gpus, note=None):
    cfg = {"workload": f"{name}: n={w['n']} nodes x d={w['d']} fp32, {w['topo']} topology, H={w['H'] or 'inf'}, "
                       f"gamma={w['gamma']}, sigma={w['sigma']}, quadratic objective, seed {SEED}",
           "l2_flush": f"none needed: each step streams {BYTES_PER_UPDATE * w['n'] * w['d'] / 1e9:.2f} GB, larger than the 126 MB L2"
                       if BYTES_PER_UPDATE * w['n'] * w['d'] > 4 * 126e6 else "state fits in L2; reported as L2-resident",
           "layout": f"row-major fp32, row stride {padded_stride(w['d'])} floats (rows padded to 128 B)",
           "sharding": f"columns, {n_gpus} shard(s) of d columns each, no collective"}
    if note:
        cfg["choice"] = note
    return cfg


def state_bytes(w):
    return 3 * w["n"] * padded_stride(w["d"]) * 4


def resolve_workload(args, torch=None, dist=None):
    """The workload to run: the one asked for, else the largest single-GPU configuration when three
    of its n x d buffers fit the device (every rank's), else the ResNet-50-sized one."""
    if args.workload:
        return args.workload, None
    fits = 1
    if torch is not None and torch.cuda.is_available():
        free, _ = torch.cuda.mem_get_info()
        fits = int(free >= state_bytes(WORKLOADS[DEFAULT_WORKLOAD]) + (3 << 30))
        if dist is not None:
            t = torch.tensor([fits], device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MIN)
            fits = int(t.item())
    if fits:
        return DEFAULT_WORKLOAD, "default: the largest configuration that fits one GPU"
    return FALLBACK_WORKLOAD, (f"fallback: 3 x {state_bytes(WORKLOADS[DEFAULT_WORKLOAD]) / 3e9:.2f} GB of "
                               f"{DEFAULT_WORKLOAD} do not fit the free device memory")


# ---------------------------------------------------------------------------------
# Arithmetic the method itself needs per node-parameter update (quadratic objective with noise),
# counted from the generator's published definition and Algorithm 1 -- not from any kernel:
#   Philox4x32-10, one call per 4 updates: 10 rounds x (2 wide multiplies + 2 three-input xors)  -> 10 per update
#   Box-Muller, one pair per 2 updates: 2 int->float conversions, 2 scalings of the uniforms,
#     lg2, the multiply by -2 ln 2, sqrt, sin, cos, 2 products r cos, r sin = 11                  -> 5.5 per update,
#     of which the 4 special-function evaluations                                                -> 2 per update
#   stochastic gradient and local update: x - b, fma(sigma, z, .), fma(-gamma, g, x)             -> 3 per update
#   mix: ring 2 adds + 1 multiply = 3; one-peer exponential 1 add + 1 multiply = 2; global
#     average 1 add per update (+ 1/n of a division)                                             -> 3 / 2 / 1
# An SM issues 4 warp instructions per clock (128 lane operations) and evaluates 16 special
# functions per clock (four per scheduler), the per-SM figures of CUDA's arithmetic-throughput table.
# ---------------------------------------------------------------------------------
LANE_OPS_PHILOX, LANE_OPS_BOX_MULLER, LANE_OPS_UPDATE = 10.0, 5.5, 3.0
LANE_OPS_MIX = {"ring": 3.0, "exp": 2.0, "global": 1.0}
XU_OPS_PER_UPDATE = 2.0
SM_COUNT, ISSUE_LANES_PER_CLK, XU_LANES_PER_CLK = 148, 128, 16


def method_lane_ops(w):
    share_global = (1.0 / w["H"]) if w["H"] else 0.0
    mix = share_global * LANE_OPS_MIX["global"] + (1.0 - share_global) * LANE_OPS_MIX[w["topo"]]
    noise = LANE_OPS_PHILOX + LANE_OPS_BOX_MULLER if w["sigma"] else 0.0
    return noise + LANE_OPS_UPDATE + mix


def alu_roofline(w, rate, kernel, sm_max_mhz, achieved_gbs):
    """Compute-bound roofline of a state that stays on chip: the rate against what the issue slots and
    the special-function units allow for the method's own operation count."""
    hz = (sm_max_mhz or 1965) * 1e6
    ops = method_lane_ops(w)
    peak_issue = SM_COUNT * ISSUE_LANES_PER_CLK * hz / ops
    peak_xu = SM_COUNT * XU_LANES_PER_CLK * hz / XU_OPS_PER_UPDATE if w["sigma"] else float("inf")
    peak = min(peak_issue, peak_xu)
    return {"bound": "alu", "kernel": kernel, "achieved": rate / 1e9, "peak": peak / 1e9,
            "unit": "G node-param updates/s", "frac": rate / peak, "traffic": None,
            "binding_unit": "issue slots" if peak_issue <= peak_xu else "special-function units",
            "method_lane_ops_per_update": ops, "frac_of_issue_peak": rate / peak_issue,
            "frac_of_special_function_peak": (rate / peak_xu) if w["sigma"] else None,
            "peak_kind": f"derived: {SM_COUNT} SMs x {ISSUE_LANES_PER_CLK} lanes/clk (special functions: "
                         f"{XU_LANES_PER_CLK}/clk) x {hz / 1e6:.0f} MHz / the method's operations per update",
            "note": "state resident on chip across iterations; HBM is touched once per launch",
            "effective_GB/s_at_12B_per_update": achieved_gbs}


# one roofline cell per target kernel and size: name, n, d, topology, H (0: gossip only, 1: global average only)
C3_D, C4_D = 25_557_032, 335_141_888
CELLS = [("c3_ring", 64, C3_D, "ring", 0, "shared", 0.1, 0.5), ("c3_exp", 64, C3_D, "exp", 0, "shared", 0.1, 0.5),
         ("c3_global", 64, C3_D, "ring", 1, "shared", 0.1, 0.5),
         ("c4_exp", 16, C4_D, "exp", 0, "zero", 1.0, 0.0), ("c4_global", 16, C4_D, "exp", 1, "zero", 1.0, 0.0)]


def timed_steps(torch, g, steps):
    """`steps` calls of gpga_step, one CUDA event pair each, on torch's current stream (the stream the
    kernels are launched on); returns the per-step milliseconds."""
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    k0 = g.get_k()
    ev[0].record()
    for s in range(steps):
        g.step(k0 + s)
        ev[s + 1].record()
    torch.cuda.synchronize()
    return [ev[s].elapsed_time(ev[s + 1]) for s in range(steps)]


def median(v):
    v = sorted(v)
    return v[len(v) // 2] if v else None


def loop_for(torch, g, sampler, seconds, est_ms):
    """Step loop of about `seconds` with the clocks sampled beside it."""
    steps = int(max(8, min(20000, math.ceil(seconds * 1e3 / max(est_ms, 1e-3)))))
    sampler.begin()
    ms = timed_steps(torch, g, steps)
    clocks = sampler.end()
    return ms, clocks


def run_cell(torch, pkg, bufs, spec, sampler, seconds, peak):
    name, n, d, topo, H, x0, x0_std, b_shift = spec
    ld = padded_stride(d)
    if bufs[0].numel() < n * ld:
        return {"skipped": "the bound buffers are smaller than this state"}
    views = [t.view(-1)[:n * ld].view(n, ld) for t in bufs]
    g = pkg.Gpga(n, d, {"ring": pkg.GPGA_TOPO_RING, "exp": pkg.GPGA_TOPO_EXP}[topo], H, 0.01, SEED)
    g.set_objective(pkg.GPGA_OBJ_QUADRATIC, sigma=0.01)
    g.set_row_stride(ld)
    g.bind(*views)
    g.init_from_seed({"zero": pkg.GPGA_X0_ZERO, "shared": pkg.GPGA_X0_SHARED_NORMAL}[x0], x0_std, b_shift)
    est = median(timed_steps(torch, g, 3))
    ms, clocks = loop_for(torch, g, sampler, seconds, est)
    g.close()
    med, algo = median(ms), BYTES_PER_UPDATE * n * d
    gbs = algo / (med * 1e-3) / 1e9
    return {"kernel": "step_global_kernel" if H == 1 else f"step_{topo}_kernel", "n": n, "d": d, "steps": len(ms),
            "ms": med, "GB/s": gbs, "frac": gbs / peak, "frac_of_nominal_8TBs": gbs / NOMINAL_PEAK_GBS,
            "sm_mhz": clocks["sm_mhz"], "reasons": clocks["reasons"],
            "ms_x_mhz": med * clocks["sm_mhz"] if clocks["sm_mhz"] else None}


def run_logistic_cells(torch, pkg, sampler, peak, names=("c5_ring_h4", "c5_ring_hinf", "c5_exp_hinf"), iterations=4000):
    """The convex workload's cells: n = 64 nodes, 4096 samples of 1024 features each, batch 128; ring with
    H = 4, and ring / one-peer exponential graph without global averaging.  One gpga_run call each (the
    whole run in one launch), microseconds per iteration; all share one data set."""
    from paper_2105_09080_b200.inputs import logistic_inputs_device
    first = WORKLOADS[names[0]]
    A, y = logistic_inputs_device(first["n"], first["m"], first["d"], SEED)
    cells = {}
    for name in names:
        w = WORKLOADS[name]
        n, d, m, batch = w["n"], w["d"], w["m"], w["batch"]
        topo = {"ring": pkg.GPGA_TOPO_RING, "exp": pkg.GPGA_TOPO_EXP}[w["topo"]]
        g = pkg.Gpga(n, d, topo, w["H"], w["gamma"], SEED)
        g.set_objective(pkg.GPGA_OBJ_LOGISTIC, l2=w["l2"], m=m, batch=batch)
        xa = torch.zeros((n, d), device="cuda")
        g.bind(xa, torch.empty_like(xa), A, y)
        g.run(200)
        torch.cuda.synchronize()
        launches0 = g.launch_count()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sampler.begin()
        e0.record()
        g.run(iterations)
        e1.record()
        torch.cuda.synchronize()
        clocks = sampler.end()
        us = e0.elapsed_time(e1) / iterations * 1e3
        algo = n * batch * d * 4 + 4 * n * d * 4        # the batch rows of A once; X read, G written and read, X+ written
        gbs = algo / (us * 1e-6) / 1e9
        cells[name] = {"kernel": "logreg_run_kernel" if g.launch_count() - launches0 < iterations else "logreg_partial + step_tile",
                       "n": n, "d": d, "m": m, "batch": batch, "topology": w["topo"], "H": w["H"] or "inf",
                       "iterations": iterations, "launches": g.launch_count() - launches0,
                       "us_per_iteration": us, "GB/s": gbs, "frac": gbs / peak, "frac_of_nominal_8TBs": gbs / NOMINAL_PEAK_GBS,
                       "bound": "the chain of hand-overs inside an iteration, not bandwidth",
                       "sm_mhz": clocks["sm_mhz"], "reasons": clocks["reasons"], "global_loss_after": g.global_loss()}
        g.close()
    return cells


# ---------------------------------------------------------------------------------
# CUDA arm
# ---------------------------------------------------------------------------------
def run_ours(args):
    import torch
    import paper_2105_09080_b200 as pkg

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    name, choice = resolve_workload(args, torch, dist)
    w = WORKLOADS[name]
    if w.get("objective") == "logistic":
        if dist is not None:
            dist.destroy_process_group()
        if rank == 0:
            run_logistic(args, w, name)
        return
    resident = BYTES_PER_UPDATE * w["n"] * padded_stride(w["d"]) <= (64 << 20)
    if args.steps is None:
        args.steps = 100_000 if resident else 200

    n, d = w["n"], w["d"]
    topo = {"ring": pkg.GPGA_TOPO_RING, "exp": pkg.GPGA_TOPO_EXP}[w["topo"]]
    kind = {"zero": pkg.GPGA_X0_ZERO, "shared": pkg.GPGA_X0_SHARED_NORMAL}[w["x0"]]
    g = pkg.Gpga(n, d, topo, w["H"], w["gamma"], SEED)
    g.set_objective(pkg.GPGA_OBJ_QUADRATIC, sigma=w["sigma"])
    from paper_2105_09080_b200.sharding import weak_shard_offset
    g.set_column_offset(weak_shard_offset(rank, d))
    g.set_row_stride(padded_stride(d))      # every node's row starts on a 128-byte line
    xa, xb, b = g.allocate()
    g.init_from_seed(kind, w["x0_std"], w["b_shift"])
    torch.cuda.synchronize()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    def max_over_ranks(ms):
        if dist is None:
            return ms
        t = torch.tensor([ms], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    # A state of at most 64 MB is advanced many iterations per launch by gpga_run (strips resident
    # on chip): one call, no per-step events.  Larger states: one launch per step.
    if resident:
        g.run(max(args.warmup, 2))      # the same multi-iteration kernel as the timed call
    else:
        for _ in range(args.warmup):
            g.step(g.get_k())
    sampler = ClockSampler(physical_gpu_index(local))
    barrier()
    launches0 = g.launch_count()
    k_first = g.get_k()
    sampler.begin()
    if resident:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        g.run(args.steps)
        e1.record()
        barrier()
        per_step, elapsed_ms = [], e0.elapsed_time(e1)
    else:
        per_step = timed_steps(torch, g, args.steps)
        barrier()
        elapsed_ms = sum(per_step)
    clocks = sampler.end()
    launches = g.launch_count() - launches0
    elapsed_ms = max_over_ranks(elapsed_ms)

    # per-kernel durations from the per-step events (one kernel per step)
    is_glob = lambda k: bool(w["H"]) and (k + 1) % w["H"] == 0
    glob = [ms for s, ms in enumerate(per_step) if is_glob(k_first + s)]
    goss = [ms for s, ms in enumerate(per_step) if not is_glob(k_first + s)]
    peak, peak_kind = measured_peak_gbs()
    algo_bytes = BYTES_PER_UPDATE * n * d
    kernels = {}
    if resident:
        kernels["run_cell_kernel" if n <= 256 else "run_tile_kernel"] = elapsed_ms / args.steps
    if goss:
        kernels[f"step_{w['topo']}_kernel"] = sum(goss) / len(goss)
    if glob:
        kernels["step_global_kernel"] = sum(glob) / len(glob)
    dominant = max(kernels, key=lambda nm: kernels[nm] * (len(goss) if nm != "step_global_kernel" else len(glob)))
    achieved = algo_bytes / (kernels[dominant] * 1e-3) / 1e9
    traffic = None
    if dominant in NCU_TRAFFIC and NCU_TRAFFIC[dominant][1] == kernel_source_digest():
        traffic = NCU_TRAFFIC[dominant][0] * algo_bytes
    sustained, cells = None, None
    if resident:
        roofline = alu_roofline(w, n * d / (kernels[dominant] * 1e-3), dominant, clocks.get("sm_max_mhz"), achieved)
    else:
        roofline = {"bound": "hbm", "kernel": dominant, "achieved": achieved, "peak": peak, "unit": "GB/s",
                    "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "traffic": traffic,
                    "algorithmic_bytes_per_launch": algo_bytes,
                    "frac_of_nominal_8TBs": achieved / NOMINAL_PEAK_GBS}
        for nm, ms in kernels.items():      # flat: one scalar per kernel of the timed loop
            roofline[f"{nm}_ms"] = ms
            roofline[f"{nm}_GBs"] = algo_bytes / (ms * 1e-3) / 1e9
        # the same loop for seconds, not milliseconds: what the board sustains under its power cap
        barrier()
        ms, sclk = loop_for(torch, g, sampler, args.sustained_seconds, elapsed_ms / args.steps)
        med = max_over_ranks(median(ms))
        sustained = {"seconds": sum(ms) * 1e-3, "steps": len(ms), "median_ms_per_step": med,
                     "value": n * d * world / (med * 1e-3), "GB/s": algo_bytes / (med * 1e-3) / 1e9,
                     "frac": algo_bytes / (med * 1e-3) / 1e9 / peak,
                     "frac_of_nominal_8TBs": algo_bytes / (med * 1e-3) / 1e9 / NOMINAL_PEAK_GBS,
                     "sm_mhz": sclk["sm_mhz"], "reasons": sclk["reasons"], "clock_samples": sclk["samples"],
                     "ms_x_mhz": med * sclk["sm_mhz"] if sclk["sm_mhz"] else None}
        if world == 1 and not args.no_cells and state_bytes(w) >= state_bytes(WORKLOADS[FALLBACK_WORKLOAD]):
            cells = {}
            for spec in CELLS:
                cells[spec[0]] = run_cell(torch, pkg, (xa, xb, b), spec, sampler, args.cell_seconds, peak)
                c = cells[spec[0]]
                if "GB/s" in c:     # flat copies inside `roofline`
                    roofline[f"cell_{spec[0]}_GBs"] = c["GB/s"]
                    roofline[f"cell_{spec[0]}_frac_of_nominal_8TBs"] = c["frac_of_nominal_8TBs"]
                    roofline[f"cell_{spec[0]}_sm_mhz"] = c["sm_mhz"]
            for cname, cell in run_logistic_cells(torch, pkg, sampler, peak).items():
                cells[cname] = cell
                roofline[f"cell_{cname}_us_per_iteration"] = cell["us_per_iteration"]
                roofline[f"cell_{cname}_frac"] = cell["frac"]
            g.init_from_seed(kind, w["x0_std"], w["b_shift"])     # the cells used the same buffers
            for _ in range(3):
                g.step(g.get_k())

    # the consensus-distance diagnostic (off the timed loop): one pass over X, 4 bytes per element
    c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    g.consensus_distance()
    launches_c = g.launch_count()
    c0.record()
    xi = g.consensus_distance()
    c1.record()
    torch.cuda.synchronize()
    xi_ms = c0.elapsed_time(c1)
    consensus = {"value": xi, "ms": xi_ms, "GB/s": 4 * n * d / (xi_ms * 1e-3) / 1e9,
                 "note": "includes the result read-back and stream synchronisation",
                 "launches": g.launch_count() - launches_c}

    # one gpga_run call over the configuration's own run length: for n <= 256 and runs of 8 or more
    # iterations it advances many iterations per launch with the cells on chip, so its rate is not
    # tied to 12 bytes per update
    run_info = None
    if not resident:
        K_run = max(w["K"], 8)
        barrier()
        r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        launches_r = g.launch_count()
        r0.record()
        g.run(K_run)
        r1.record()
        barrier()
        run_ms = max_over_ranks(r0.elapsed_time(r1))
        run_info = {"value": n * d * K_run * world / (run_ms * 1e-3), "unit": UNIT, "iterations": K_run,
                    "ms_per_iteration": run_ms / K_run, "launches": g.launch_count() - launches_r,
                    "note": "one gpga_run call, after the timed loop; `value` above times one launch per iteration"}

    e2e = None
    if not args.no_e2e:
        try:
            e2e = run_e2e(torch, pkg, (xa, xb, b), w, dist, rank)
        except Exception as exc:     # e.g. not enough pinnable host memory for the host copies
            e2e = {"value": None, "unit": UNIT, "error": repr(exc)[:200]}
    sampler.finish()

    value = n * d * args.steps * world / (elapsed_ms * 1e-3)
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": elapsed_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": workload_config(name, w, world, choice), "hbm_gbs": value * BYTES_PER_UPDATE / 1e9 / world,
            "roofline": roofline, "clocks": clocks, "e2e": e2e, "gpu_launches": launches,
            "sustained": sustained, "cells": cells, "consensus_distance": consensus, "gpga_run": run_info}
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            try:
                line["cpu_baseline"] = cpu_baseline(w)
            except Exception as exc:
                line["cpu_baseline"] = {"value": None, "unit": UNIT, "kind": "oracle", "error": repr(exc)[:200]}
        print(json.dumps(line), flush=True)
    g.close()
    if dist is not None:
        dist.destroy_process_group()


def run_logistic(args, w, name):
    """Convex workload: per-node mini-batch logistic gradient + fused step/mix, 2 launches per step."""
    import torch
    import paper_2105_09080_b200 as pkg
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    n, d, m, batch = w["n"], w["d"], w["m"], w["batch"]
    from paper_2105_09080_b200.inputs import logistic_inputs_device
    A, y = logistic_inputs_device(n, m, d, SEED)
    topo = {"ring": pkg.GPGA_TOPO_RING, "exp": pkg.GPGA_TOPO_EXP}[w["topo"]]
    g = pkg.Gpga(n, d, topo, w["H"], w["gamma"], SEED)
    g.set_objective(pkg.GPGA_OBJ_LOGISTIC, l2=w["l2"], m=m, batch=batch)
    xa = torch.zeros((n, d), device="cuda")
    g.bind(xa, torch.empty_like(xa), A, y)
    g.run(max(args.warmup, 50))         # the same back-to-back launches as the timed call
    torch.cuda.synchronize()
    sampler = ClockSampler(physical_gpu_index(int(os.environ.get("LOCAL_RANK", "0"))))
    launches0 = g.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.begin()
    e0.record()
    g.run(args.steps)
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.end()
    sampler.finish()
    ms = e0.elapsed_time(e1)
    launches = g.launch_count() - launches0
    if launches < args.steps:      # gpga_run took the many-iterations-per-launch kernel
        kernel_label = "logreg_run_kernel"
        kernel_note = (f"{launches} launch(es) for {args.steps} iterations: a cluster of two blocks per node keeps x_i on "
                       "chip; the chain gradient -> exchange -> mix inside an iteration, not bandwidth, sets the time")
    else:
        kernel_label = "logreg_partial_tma_reg_kernel + step_tile_kernel"
        kernel_note = ("two launches per iteration, each a programmatic dependent of the one before; "
                       "the dependent chain inside an iteration, not bandwidth, sets the time")
    # bytes the method must move per step: the batch rows of A once, X read, G write+read, X+ write
    algo_bytes = n * batch * d * 4 + 4 * n * d * 4
    peak, peak_kind = measured_peak_gbs()
    achieved = algo_bytes / (ms / args.steps * 1e-3) / 1e9
    # end to end: pinned host A, y, X0 in; the configuration's K iterations; X out
    hA, hy = A.cpu().pin_memory(), y.cpu().pin_memory()
    hx0 = torch.zeros((n, d)).pin_memory()
    hout = torch.empty((n, d)).pin_memory()
    torch.cuda.synchronize()
    j0, j1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    j0.record()
    A.copy_(hA, non_blocking=True)
    y.copy_(hy, non_blocking=True)
    g.x_bufs[0].copy_(hx0, non_blocking=True)
    g2 = pkg.Gpga(n, d, topo, w["H"], w["gamma"], SEED)
    g2.set_objective(pkg.GPGA_OBJ_LOGISTIC, l2=w["l2"], m=m, batch=batch)
    g2.bind(g.x_bufs[0], g.x_bufs[1], A, y)
    g2.run(w["K"])
    hout.copy_(g2.get_x(), non_blocking=True)
    j1.record()
    torch.cuda.synchronize()
    dt = j0.elapsed_time(j1) * 1e-3     # device time of the job, copies included
    loss, xi_dist, gloss = g2.mean_loss(), g2.consensus_distance(), g2.global_loss()
    line = {"metric": METRIC, "value": n * d * args.steps / (ms * 1e-3), "unit": UNIT, "n_gpus": 1,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"{name}: n={n} nodes, m={m} samples x d={d} features each, batch {batch}, "
                                   f"l2={w['l2']}, {w['topo']} topology, H={w['H'] or 'inf'}, gamma={w['gamma']}, "
                                   f"logistic objective, seed {SEED}",
                       "l2_flush": "A (1.07 GB) is larger than L2; each step reads a fresh random 33.5 MB of it"},
            "roofline": {"bound": "hbm", "kernel": kernel_label,
                         "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "peak_kind": f"of {peak_kind}", "traffic": None, "algorithmic_bytes_per_iteration": algo_bytes,
                         "note": kernel_note},
            "clocks": clocks,
            "e2e": {"value": n * d * w["K"] / dt, "unit": UNIT, "h2d_bytes_per_step": (A.numel() + y.numel() + n * d) * 4 / w["K"],
                    "d2h_bytes_per_step": n * d * 4 / w["K"],
                    "job": f"pinned host A, y, X0 copied in, K={w['K']} iterations, X copied out", "seconds_per_job": dt},
            "after_K": {"mean_minibatch_loss": loss, "consensus_distance": xi_dist, "global_loss": gloss},
            "gpu_launches": launches}
    print(json.dumps(line))


def run_node_shard(args):
    """--node-shards G: the two kernels of ONE shard of the node-sharded iteration (n / G consecutive
    nodes, all d columns) timed per iteration: export, then step.  The exchange between shards is not
    part of it (one GPU): the receive buffer keeps whatever it holds."""
    import torch
    import paper_2105_09080_b200 as pkg
    from paper_2105_09080_b200 import node_sharded as ns
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    name = args.workload or FALLBACK_WORKLOAD
    w = WORKLOADS[name]
    if w.get("objective") == "logistic":
        raise SystemExit("--node-shards: the node-sharded iteration covers the quadratic workloads")
    G, n, d = args.node_shards, w["n"], w["d"]
    if n % G:
        raise SystemExit(f"--node-shards {G} does not divide n = {n}")
    n_l, ld = n // G, padded_stride(w["d"])
    topo = {"ring": pkg.GPGA_TOPO_RING, "exp": pkg.GPGA_TOPO_EXP}[w["topo"]]
    sh = ns.NodeShard(n, d, topo, w["H"], w["gamma"], SEED, G, min(1, G - 1), sigma=w["sigma"], ld=ld)
    xa = torch.randn((n_l, ld), device="cuda") * 0.1
    sh.bind(xa, torch.empty_like(xa), torch.randn((n_l, ld), device="cuda"))
    steps = args.steps or 100
    if args.fused_send:
        # stand-ins for the other shards' receive areas, in this device's memory: the export kernel
        # stores its messages there itself (gpga_shard_export_to), as it would into peer-mapped memory
        areas = torch.zeros((G, sh.recv.numel()), dtype=torch.uint8, device="cuda")
        base_of = lambda s: sh.recv.data_ptr() if s == sh.shard else areas[s].data_ptr()
        sh.export = lambda k: sh.export_to(k, ns.direct_destinations(sh.plan(k), sh.shard, G, base_of))
    for k in range(args.warmup):
        sh.export(k)
        sh.step(k)
    torch.cuda.synchronize()
    sampler = ClockSampler(physical_gpu_index(int(os.environ.get("LOCAL_RANK", "0"))))
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2 * steps + 1)]
    kinds = []
    sampler.begin()
    ev[0].record()
    for s_ in range(steps):
        k = args.warmup + s_
        plan = sh.plan(k)
        kinds.append("global" if plan.kind == ns.GPGA_SHARD_GLOBAL else
                     (f"exp_hop{plan.hop}" if plan.kind == ns.GPGA_SHARD_EXP else "ring"))
        sh.export(k)
        ev[2 * s_ + 1].record()
        sh.step(k)
        ev[2 * s_ + 2].record()
    torch.cuda.synchronize()
    clocks = sampler.end()
    sampler.finish()
    per = {}
    for s_, kind in enumerate(kinds):
        per.setdefault(kind, []).append((ev[2 * s_].elapsed_time(ev[2 * s_ + 1]), ev[2 * s_ + 1].elapsed_time(ev[2 * s_ + 2])))
    table = {kind: {"iterations": len(v), "export_ms": median([a for a, _ in v]), "step_ms": median([b for _, b in v]),
                    "GB/s_at_12_bytes_per_update": BYTES_PER_UPDATE * n_l * d / (median([a + b for a, b in v]) * 1e-3) / 1e9}
             for kind, v in per.items()}
    total_ms = ev[0].elapsed_time(ev[-1])
    print(json.dumps({"metric": METRIC, "value": n_l * d * steps / (total_ms * 1e-3), "unit": UNIT, "n_gpus": 1,
                      "steps": steps, "warmup": args.warmup, "ms_per_step": total_ms / steps, "higher_is_better": True,
                      "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                      "config": {"workload": f"{name}: shard {min(1, G - 1)} of {G} ({n_l} of n={n} nodes x d={d} fp32, "
                                             f"{w['topo']} topology, H={w['H'] or 'inf'}), export + step kernels of the "
                                             f"node-sharded iteration; " + ("the export kernel stores its messages into the receivers' "
                                             "areas itself (stand-ins in this device's memory)" if args.fused_send
                                             else "the exchange between shards is not timed")},
                      "per_kind": table, "clocks": clocks, "gpu_launches": sh.g.launch_count()}), flush=True)
    sh.close()


def host_memory_available():
    try:
        for ln in open("/proc/meminfo"):
            if ln.startswith("MemAvailable:"):
                return int(ln.split()[1]) * 1024
    except OSError:
        pass
    return None


def e2e_columns(n, d, world):
    """Columns of the end-to-end job: all d when the three pinned host buffers of every rank fit in
    70 % of the host's available memory, else as many as do (a multiple of 32, at least 4096)."""
    avail = host_memory_available()
    need = 3 * n * d * 4 * world
    if avail is None or need <= 0.7 * avail:
        return d
    cols = int(0.7 * avail / world / (3 * n * 4)) // 32 * 32
    return max(4096, min(d, cols))


def run_e2e(torch, pkg, bufs, w, dist, rank):
    """The configuration's K iterations through gpga_run_host: pinned host X0 and b in, X^(K) out."""
    from paper_2105_09080_b200.sharding import weak_shard_offset
    n, d, K = w["n"], w["d"], w["K"]
    world = dist.get_world_size() if dist is not None else 1
    cols = e2e_columns(n, d, world)
    problem = None
    zero_x0 = w["x0"] == "zero"         # X^(0) = 0: the host entry fills it on the device, no upload
    try:
        x0 = None if zero_x0 else torch.empty((n, cols), dtype=torch.float32, pin_memory=True)
        bh = torch.empty((n, cols), dtype=torch.float32, pin_memory=True)
        out = torch.empty((n, cols), dtype=torch.float32, pin_memory=True)
    except Exception as exc:        # not enough pinnable host memory on this rank
        problem = repr(exc)[:200]
    if dist is not None:            # every rank must take the same branch before the next collective
        ok = torch.tensor([0 if problem else 1], device="cuda")
        dist.all_reduce(ok, op=dist.ReduceOp.MIN)
        if int(ok.item()) == 0 and not problem:
            problem = "another rank could not pin its host buffers"
    if problem:
        return {"value": None, "unit": UNIT, "error": problem}
    ld = padded_stride(cols)
    views = [t.view(-1)[:n * ld].view(n, ld) for t in bufs]
    g = pkg.Gpga(n, cols, {"ring": pkg.GPGA_TOPO_RING, "exp": pkg.GPGA_TOPO_EXP}[w["topo"]], w["H"], w["gamma"], SEED)
    g.set_objective(pkg.GPGA_OBJ_QUADRATIC, sigma=w["sigma"])
    g.set_column_offset(weak_shard_offset(rank, d))
    g.set_row_stride(ld)
    g.bind(*views)
    # host copies of the seeded inputs (downloaded once, outside the timed region)
    g.init_from_seed({"zero": 0, "shared": 1}[w["x0"]], w["x0_std"], w["b_shift"])
    if x0 is not None:
        x0.copy_(views[0][:, :cols])
    bh.copy_(views[2][:, :cols])
    torch.cuda.synchronize()
    g.run_host(x0, bh, K, out)                      # warm-up job
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    jobs = 2
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(jobs):
        g.run_host(x0, bh, K, out)                  # returns when its copies and kernels are done
    e1.record()
    torch.cuda.synchronize()
    dt = e0.elapsed_time(e1) * 1e-3                 # device time, copies included
    g.close()
    if dist is not None:
        t = torch.tensor([dt], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dt = float(t.item())
    width = "all" if cols == d else f"the first {cols} of"
    arrays_in = 1 if zero_x0 else 2
    what_in = "pinned host b copied in (X0 = 0 is filled on the device)" if zero_x0 else "pinned host X0 and b copied in"
    return {"value": n * cols * K * jobs * world / dt, "unit": UNIT,
            "h2d_bytes_per_step": arrays_in * n * cols * 4 / K, "d2h_bytes_per_step": n * cols * 4 / K,
            "job": f"gpga_run_host on {width} {d} columns: {what_in} "
                   f"({arrays_in * n * cols * 4 / 1e9:.2f} GB), K={K} iterations, X copied out ({n * cols * 4 / 1e9:.2f} GB); "
                   f"bytes per step are the job's bytes / K",
            "seconds_per_job": dt / jobs}


def run_dry(args):
    """--dry-run: the multi-rank plumbing without CUDA (gloo): every rank takes its column shard,
    the ranks meet at a barrier, a per-rank number is reduced with MAX as the timing is, and rank 0
    prints one JSON line.  Used by the CPU tests of the launch path."""
    import torch
    import torch.distributed as dist
    from paper_2105_09080_b200.sharding import weak_shard_offset
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    name = args.workload or DEFAULT_WORKLOAD
    w = WORKLOADS[name]
    if world > 1:
        dist.init_process_group("gloo")
    shard = (rank, weak_shard_offset(rank, w["d"]), w["d"])
    shards, slowest = [shard], float(rank + 1)
    if world > 1:
        shards = [None] * world
        dist.all_gather_object(shards, shard)
        dist.barrier()
        t = torch.tensor([slowest], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        slowest = float(t.item())
    if rank == 0:
        print(json.dumps({"dry_run": True, "metric": METRIC, "unit": UNIT, "n_gpus": world, "value": None,
                          "config": workload_config(name, w, world), "scaling": "weak",
                          "shards": [list(x) for x in sorted(shards)], "max_over_ranks": slowest}), flush=True)
    if world > 1:
        dist.destroy_process_group()


def free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def spawn_ranks(n_ranks, argv):
    """Start n_ranks copies of this script, one per GPU, the way the multi-GPU contract launches it."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_ranks}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), str(Path(__file__).resolve())] + list(argv)
    return subprocess.call(cmd)


def main(argv=None):
    argv = list(sys.argv[1:] if argv is None else argv)
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None,
                    help="timed iterations (default: 200; 100000 for a state that stays on chip, 2000 for the "
                         "logistic workload, so that the timed region lasts milliseconds, not microseconds)")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=None, choices=sorted(WORKLOADS),
                    help=f"default: {DEFAULT_WORKLOAD}, or {FALLBACK_WORKLOAD} when it does not fit the device")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-cells", action="store_true", help="skip the per-kernel roofline cells")
    ap.add_argument("--sustained-seconds", type=float, default=2.0)
    ap.add_argument("--cell-seconds", type=float, default=1.0)
    ap.add_argument("--dry-run", action="store_true", help="multi-rank plumbing only, on CPU with gloo")
    ap.add_argument("--fused-send", action="store_true",
                    help="with --node-shards: time gpga_shard_export_to, the export kernel that stores its messages "
                         "straight into the receivers' areas")
    ap.add_argument("--node-shards", type=int, default=0,
                    help="time the export + step kernels of one shard of a node-sharded run with this many shards")
    args = ap.parse_args(argv)
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    under_launcher = "WORLD_SIZE" in os.environ and "RANK" in os.environ
    if args.gpus > 1 and not under_launcher and args.impl == "ours":
        if not args.dry_run:
            import torch
            have = torch.cuda.device_count() if torch.cuda.is_available() else 0
            if have < args.gpus:
                raise SystemExit(f"bench.py --gpus {args.gpus}: this machine shows {have} CUDA device(s)")
        sys.exit(spawn_ranks(args.gpus, argv))       # one process per GPU; rank 0 prints the line
    if args.dry_run:
        return run_dry(args)
    if args.node_shards:
        return run_node_shard(args)
    if args.impl == "reference":
        if int(os.environ.get("RANK", "0")) != 0:
            return                                    # rank 0 alone runs the oracle
        torch = None
        try:
            import torch
        except Exception:
            pass
        name, choice = resolve_workload(args, torch)
        w = WORKLOADS[name]
        if w.get("objective") == "logistic":
            print(json.dumps({"impl": "reference", "unavailable": "reference arm is defined for the quadratic workloads"}))
            return
        if args.steps is None:
            args.steps = 20
        return run_reference(args, w, name, choice)
    if args.steps is None and args.workload and WORKLOADS[args.workload].get("objective") == "logistic":
        args.steps = 2000
    run_ours(args)


if __name__ == "__main__":
    main()
