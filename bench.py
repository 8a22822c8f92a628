#!/usr/bin/env python
"""Benchmark of the Gossip-PGA iteration (libgpga) on B200.

A "step" is one iteration of Algorithm 1 over the whole n x d state: the fused
local-update + gossip kernel, or the fused local-update + global-average kernel on
every H-th iteration.  Prints one JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3_ring_h4] [--impl reference]

Multi-GPU: the state is sharded by columns (columns evolve independently), one
process per GPU, no data-path collective; every rank holds a full-width shard of a
problem N times wider (weak scaling).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
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
DEFAULT_WORKLOAD = "c3_ring_h4"

# DRAM bytes per launch of the dominant kernel from an ncu capture (dram__bytes_read.sum +
# dram__bytes_write.sum), as a multiple of the algorithmic bytes of the captured launch, with
# the digest of the kernel sources at capture time.  A changed source voids it (-> null).
NCU_TRAFFIC = {
    # kernel name: (traffic / algorithmic bytes, source digest); captured at n=64, d=2,097,192 and
    # n=16, d=8,388,608 -- one pass over three n x d arrays, so traffic scales with n x d
    "step_ring_kernel": (0.977, "3199e78917cf862e"),
    "step_exp_kernel": (0.977, "3199e78917cf862e"),
    "step_global_kernel": (0.968, "3199e78917cf862e"),
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
    """Samples SM clock and clock-event reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.02):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._halt = threading.Event()
        self.active = threading.Event()
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
            while not self._halt.is_set():
                if self.active.is_set():
                    self.samples.append(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                    mask = get_reasons(h)
                    for bit, nm in names.items():
                        if mask & bit and bit.bit_count() == 1:
                            self.reasons.add(nm)
                time.sleep(self.period)
            nv.nvmlShutdown()
        except Exception as exc:          # NVML missing: report it, do not fail the run
            self.error = repr(exc)

    def finish(self):
        self._halt.set()
        self.join(timeout=2)
        s = sorted(self.samples)
        return {"sm_mhz": (s[len(s) // 2] if s else None), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(r for r in self.reasons if r not in ("GpuIdle", "None")),
                "samples": len(s), **({"error": self.error} if self.error else {})}


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


def run_reference(args, w, name):
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
        "data": "synthetic", "config": workload_config(name, w, args.gpus),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": o.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def padded_stride(d):
    return (d + 31) // 32 * 32


def workload_config(name, w, n_gpus):
    return {"workload": f"{name}: n={w['n']} nodes x d={w['d']} fp32, {w['topo']} topology, H={w['H'] or 'inf'}, "
                        f"gamma={w['gamma']}, sigma={w['sigma']}, quadratic objective, seed {SEED}",
            "l2_flush": f"none needed: each step streams {BYTES_PER_UPDATE * w['n'] * w['d'] / 1e9:.2f} GB, larger than the 126 MB L2"
                        if BYTES_PER_UPDATE * w['n'] * w['d'] > 4 * 126e6 else "state fits in L2; reported as L2-resident",
            "layout": f"row-major fp32, row stride {padded_stride(w['d'])} floats (rows padded to 128 B)",
            "sharding": f"columns, {n_gpus} shard(s) of d columns each, no collective"}


# ---------------------------------------------------------------------------------
# CUDA arm
# ---------------------------------------------------------------------------------
def run_ours(args, w, name):
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

    # A state of at most 64 MB is advanced many iterations per launch by gpga_run (strips resident
    # in shared memory): one call, no per-step events.  Larger states: one launch per step.
    resident = BYTES_PER_UPDATE * n * padded_stride(d) <= (64 << 20)
    events = [torch.cuda.Event(enable_timing=True) for _ in range(2 if resident else args.steps + 1)]
    if resident:
        g.run(max(args.warmup, 2))      # the same multi-iteration kernel as the timed call
    else:
        for _ in range(args.warmup):
            g.step(g.get_k())
    barrier()
    sampler = ClockSampler(physical_gpu_index(local))
    sampler.start()
    launches0 = g.launch_count()
    k_first = g.get_k()
    sampler.active.set()
    events[0].record()
    if resident:
        g.run(args.steps)
        events[-1].record()
    else:
        for s in range(args.steps):
            g.step(k_first + s)
            events[s + 1].record()
    barrier()
    sampler.active.clear()
    clocks = sampler.finish()
    launches = g.launch_count() - launches0
    elapsed_ms = events[0].elapsed_time(events[-1])
    per_step = [] if resident else [events[s].elapsed_time(events[s + 1]) for s in range(args.steps)]
    if dist is not None:
        t = torch.tensor([elapsed_ms], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        elapsed_ms = float(t.item())

    # per-kernel durations from the per-step events (one kernel per step)
    glob = [ms for s, ms in enumerate(per_step) if w["H"] and (k_first + s + 1) % w["H"] == 0]
    goss = [ms for s, ms in enumerate(per_step) if not (w["H"] and (k_first + s + 1) % w["H"] == 0)]
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
    if resident:
        # Compute-bound: X and b stay on chip.  Peak = SMs x 128 lanes/clk x max SM clock / lane
        # operations per update (42 = the 169 warp instructions that run_cell_kernel executes per warp
        # and iteration, ncu smsp__inst_executed, over the 4 updates of a thread).
        alu_peak = 148 * 128 * (clocks.get("sm_max_mhz") or 1965) * 1e6 / 42.0
        rate = n * d / (kernels[dominant] * 1e-3)
        roofline = {"bound": "alu", "kernel": dominant, "achieved": rate / 1e9, "peak": alu_peak / 1e9,
                    "unit": "G node-param updates/s", "frac": rate / alu_peak, "traffic": None,
                    "note": "state resident in shared memory across iterations; HBM is touched once per launch",
                    "effective_GB/s_at_12B_per_update": achieved}
    else:
      roofline = {"bound": "hbm", "kernel": dominant, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "traffic": traffic,
                "algorithmic_bytes_per_launch": algo_bytes,
                "per_kernel": {nm: {"ms": ms, "GB/s": algo_bytes / (ms * 1e-3) / 1e9,
                                    "frac": algo_bytes / (ms * 1e-3) / 1e9 / peak} for nm, ms in kernels.items()},
                "frac_of_nominal_8TBs": achieved / 8000.0}

    # end to end through the host entry point: pinned host buffers in, K iterations, result out
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

    # the same iterations through gpga_run: for n <= 128 and long runs it advances many iterations
    # per launch with the cells on chip, so its rate is not tied to 12 bytes per update
    run_info = None
    if not resident:
        barrier()
        r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        launches_r = g.launch_count()
        r0.record()
        g.run(args.steps)
        r1.record()
        barrier()
        run_ms = r0.elapsed_time(r1)
        if dist is not None:
            t = torch.tensor([run_ms], device="cuda", dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            run_ms = float(t.item())
        run_info = {"value": n * d * args.steps * world / (run_ms * 1e-3), "unit": UNIT, "iterations": args.steps,
                    "ms_per_iteration": run_ms / args.steps, "launches": g.launch_count() - launches_r,
                    "note": "one gpga_run call over the same number of iterations, after the timed loop; "
                            "reported beside `value`, which times one launch per iteration"}

    e2e = None
    if not args.no_e2e:
        try:
            e2e = run_e2e(torch, g, w, dist)
        except Exception as exc:     # e.g. not enough pinnable host memory for the host copies
            e2e = {"value": None, "unit": UNIT, "error": repr(exc)[:200]}

    value = n * d * args.steps * world / (elapsed_ms * 1e-3)
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": elapsed_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": workload_config(name, w, world), "hbm_gbs": value * BYTES_PER_UPDATE / 1e9 / world,
            "roofline": roofline, "clocks": clocks, "e2e": e2e, "gpu_launches": launches,
            "consensus_distance": consensus, "gpga_run": run_info}
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            try:
                line["cpu_baseline"] = cpu_baseline(w)
            except Exception as exc:
                line["cpu_baseline"] = {"value": None, "unit": UNIT, "kind": "oracle", "error": repr(exc)[:200]}
        print(json.dumps(line))
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
    sampler.start()
    launches0 = g.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.active.set()
    e0.record()
    g.run(args.steps)
    e1.record()
    torch.cuda.synchronize()
    sampler.active.clear()
    clocks = sampler.finish()
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


def run_e2e(torch, g, w, dist):
    n, d, K = w["n"], w["d"], w["K"]
    problem = None
    try:
        x0 = torch.empty((n, d), dtype=torch.float32, pin_memory=True)
        bh = torch.empty((n, d), dtype=torch.float32, pin_memory=True)
        out = torch.empty((n, d), dtype=torch.float32, pin_memory=True)
    except Exception as exc:        # not enough pinnable host memory on this rank
        problem = repr(exc)[:200]
    if dist is not None:            # every rank must take the same branch before the next collective
        ok = torch.tensor([0 if problem else 1], device="cuda")
        dist.all_reduce(ok, op=dist.ReduceOp.MIN)
        if int(ok.item()) == 0 and not problem:
            problem = "another rank could not pin its host buffers"
    if problem:
        return {"value": None, "unit": UNIT, "error": problem}
    # host copies of the seeded inputs (downloaded once, outside the timed region)
    g.init_from_seed({"zero": 0, "shared": 1}[w["x0"]], w["x0_std"], w["b_shift"])
    x0.copy_(g.x_bufs[0][:, :d])
    bh.copy_(g._keep[2][:, :d])
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
    world = 1
    if dist is not None:
        t = torch.tensor([dt], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dt = float(t.item())
        world = dist.get_world_size()
    return {"value": n * d * K * jobs * world / dt, "unit": UNIT,
            "h2d_bytes_per_step": 2 * n * d * 4 / K, "d2h_bytes_per_step": n * d * 4 / K,
            "job": f"gpga_run_host: pinned host X0 and b copied in ({2 * n * d * 4 / 1e9:.2f} GB), K={K} iterations, "
                   f"X copied out ({n * d * 4 / 1e9:.2f} GB); bytes per step are the job's bytes / K",
            "seconds_per_job": dt / jobs}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None,
                    help="timed iterations (default: 200; 100000 for a state that stays on chip, 2000 for the "
                         "logistic workload, so that the timed region lasts milliseconds, not microseconds)")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    w = WORKLOADS[args.workload]
    if args.steps is None:
        if w.get("objective") == "logistic":
            args.steps = 2000
        elif BYTES_PER_UPDATE * w["n"] * padded_stride(w["d"]) <= (64 << 20):
            args.steps = 100_000
        else:
            args.steps = 200
    if w.get("objective") == "logistic":
        if args.impl == "reference":
            print(json.dumps({"impl": "reference", "unavailable": "reference arm is defined for the quadratic workloads"}))
        else:
            run_logistic(args, w, args.workload)
    elif args.impl == "reference":
        run_reference(args, w, args.workload)
    else:
        run_ours(args, w, args.workload)


if __name__ == "__main__":
    main()
