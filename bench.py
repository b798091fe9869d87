#!/usr/bin/env python
"""Benchmark of the PowerSGD+ compression hot path on B200.

One "step" is one iteration of Algorithm 2 (without the optimizer) over ALL
matrices of the workload: error-feedback add, SSP-Comp or (every tau steps)
SVD-Comp, residual update.  Default workload: the 130M-parameter LLaMA-shaped
stack (84 matrices, r = 8, N = 8 simulated nodes, refresh every 50 steps) with
synthetic gradients.  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                  [--workload 2|3|4|5] [--rank r] [--no-sweep] [--no-e2e] [--no-cpu]

Metric: gradient GB/s = bytes of G consumed per second, whole job.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "powersgd_plus_step_gradient_throughput"
UNIT = "GB/s"
FALLBACK_HBM = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum per element of one launch, from the ncu captures summarised under
# profiles/ (taken on the 16384x4096, N=4 workload, where traffic grows in proportion to the elements)
TRAFFIC_BYTES_PER_ELEMENT = {"k_fused_step": 11.87}

# default (rank, nodes, refresh period) per workload id
DEFAULTS = {2: (8, 8, 50), 3: (16, 16, 20), 4: (32, 8, 100), 5: (16, 4, 0), 1: (4, 4, 5)}


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=2)
    ap.add_argument("--rank", type=int, default=None)
    ap.add_argument("--mode", default="deferred", choices=["eager", "deferred"])
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-refresh", action="store_true", help="tau = 0 (plain PowerSGD steps only)")
    ap.add_argument("--refresh-period", type=int, default=None, help="override the workload's refresh period tau")
    ap.add_argument("--grad-dtype", default="float32", choices=["float32", "bfloat16"],
                    help="storage type of the gradients G (bfloat16: 2 bytes per element read instead of 4)")
    return ap.parse_args()


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM, "fallback"


class ClockSampler:
    """nvidia-smi clock/throttle samples taken DURING a timed region."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.idx = gpu_index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(self.idx), "--query-gpu=" + self.Q,
                                       "--format=csv,noheader,nounits", "-lms", "100"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        for line in self.f.read().splitlines():
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1])); mx.append(float(c[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), c[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.unlink(self.f.name)
        except OSError:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def stack_for(workload):
    from paper_2509_11254_b200 import synth

    return synth.STACKS[workload]


def algorithmic_bytes(shapes, r, N, g_bytes_per_element=4):
    """Minimum traffic of a step: read G, read E, write E per element (12 B with float32 G) plus the P/Q traffic."""
    el = sum(m * n * c for m, n, c in shapes) * N
    pq = sum(4 * (2 * N * m * r + 2 * m * r + 2 * N * n * r + 2 * n * r) * c for m, n, c in shapes)
    return (8 + g_bytes_per_element) * el + pq, g_bytes_per_element * el


# ----------------------------------------------------------------------------
# CPU baseline: the oracle as it stands, on a bounded sample
# ----------------------------------------------------------------------------
def cpu_baseline(workload, r, N, budget_s=12.0):
    import numpy as np

    from oracle import psgd_oracle as orc
    from paper_2509_11254_b200 import synth

    shapes = stack_for(workload)
    t_used, g_bytes, nsteps = 0.0, 0, 0
    desc = []
    for (m, n, _c) in shapes:
        G = synth.make_gradients(workload, m, n, N, step=1, matrix_id=0)
        o = orc.PowerSGDPlusOracle(m, n, r, N, 0, synth.init_Q(n, r))
        reps = 0
        t0 = time.perf_counter()
        while True:
            o.step(G)
            reps += 1
            if time.perf_counter() - t0 > budget_s / len(shapes) or reps >= 20:
                break
        dt = time.perf_counter() - t0
        t_used += dt
        g_bytes += reps * G.nbytes
        nsteps += reps
        desc.append(f"{reps} SSP steps of one {m}x{n} matrix (N={N})")
    try:
        cores = len(os.sched_getaffinity(0))
    except Exception:
        cores = os.cpu_count()
    return {"value": g_bytes / t_used / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "; ".join(desc) + f"; r={r}; numpy float64 (OpenBLAS threads = cores)"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    r, N, tau = DEFAULTS[args.workload]
    r = args.rank or r
    import numpy as np

    from oracle import psgd_oracle as orc
    from paper_2509_11254_b200 import synth

    shapes = stack_for(args.workload)
    m, n, _ = shapes[0]
    o = orc.PowerSGDPlusOracle(m, n, r, N, 0, synth.init_Q(n, r))
    Gs = [synth.make_gradients(args.workload, m, n, N, step=s) for s in range(2)]
    steps = max(1, min(args.steps, 50))
    for w in range(max(1, min(args.warmup, 3))):
        o.step(Gs[w % 2])
    t0 = time.perf_counter()
    for s in range(steps):
        o.step(Gs[s % 2])
    dt = time.perf_counter() - t0
    val = steps * Gs[0].nbytes / dt / 1e9
    try:
        cores = len(os.sched_getaffinity(0))
    except Exception:
        cores = os.cpu_count()
    sample = f"each step = one SSP step of one {m}x{n} matrix (N={N}, r={r}) of workload {args.workload}"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": args.warmup, "ms_per_step": dt / steps * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": synth.WORKLOADS[args.workload]["name"], "r": r, "N": N, "sample": sample},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ----------------------------------------------------------------------------
# GPU arm
# ----------------------------------------------------------------------------
def build_handles(workload, r, N, tau, device, mode, seed=1, grad_dtype="float32"):
    from paper_2509_11254_b200 import PowerSGDPlus

    return [PowerSGDPlus(m, n, r, N, refresh_period=tau, seed=seed + i, count=c, device=device, mode=mode, grad_dtype=grad_dtype)
            for i, (m, n, c) in enumerate(stack_for(workload))]


def make_inputs(workload, N, device, nbuf, grad_dtype="float32"):
    import torch
    from paper_2509_11254_b200 import synth

    bufs = []
    for b in range(nbuf):
        row = []
        for (m, n, c) in stack_for(workload):
            g = synth.make_gradients_torch(workload, m, n, N, c, step=b, device=device)
            row.append(g.to(torch.bfloat16) if grad_dtype == "bfloat16" else g)
        bufs.append(row)
    return bufs


def timed_steps(torch, stack, bufs, steps, dist_barrier):
    """K steps of the whole stack; every step forks from and joins the current stream, where the two events are."""
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    dist_barrier()
    torch.cuda.synchronize()
    ev0.record()
    for s in range(steps):
        stack.step(bufs[s % len(bufs)])
    ev1.record()
    torch.cuda.synchronize()
    dist_barrier()
    return ev0.elapsed_time(ev1)


def sweep_config5(torch, device, peak, mode):
    """Workload 5: m=16384, n=4096, N=4, per-rank step and refresh latency."""
    from paper_2509_11254_b200 import PowerSGDPlus, synth

    m, n, N = 16384, 4096, 4
    bufs = [synth.make_gradients_torch(5, m, n, N, 1, step=b, device=device) for b in range(2)]
    out = []
    for r in (1, 4, 16, 64, 128):
        h = PowerSGDPlus(m, n, r, N, refresh_period=0, seed=5, device=device, mode=mode)
        for s in range(3):
            h.step(bufs[s % 2])
        steps = 10
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        ev0.record()
        for s in range(steps):
            h.step(bufs[s % 2])
        ev1.record()
        torch.cuda.synchronize()
        ms = ev0.elapsed_time(ev1) / steps
        h.refresh(bufs[0])
        torch.cuda.synchronize()
        ev0.record()
        for s in range(2):
            h.refresh(bufs[s % 2])
        ev1.record()
        torch.cuda.synchronize()
        rms = ev0.elapsed_time(ev1) / 2
        flags = h.last_status()
        alg, gb = algorithmic_bytes([(m, n, 1)], r, N)
        plan = h.plan_info()
        path = "three-pass"
        if mode == "deferred":
            path = "single-pass" if plan["single_pass"] else ("two-pass" if r <= 16 else "three-pass")
        out.append({"r": r, "kernel": path, "step_ms": round(ms, 4), "grad_GBps": round(gb / ms / 1e6, 1),
                    "min_bytes_frac": round(alg / ms / 1e6 / peak, 4), "refresh_ms": round(rms, 3),
                    "flags": flags})
        h.close()
        del h
        torch.cuda.empty_cache()
    return out


def run_ours(args):
    import torch

    from paper_2509_11254_b200.replicas import Replicas, env_rank

    rank, local, world = env_rank()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local)
    device = f"cuda:{local}"
    reps = Replicas("nccl", device)
    barrier = reps.barrier

    from paper_2509_11254_b200 import synth

    r, N, tau = DEFAULTS[args.workload]
    r = args.rank or r
    if args.refresh_period is not None:
        tau = args.refresh_period
    if args.no_refresh:
        tau = 0
    shapes = stack_for(args.workload)
    peak, peak_kind = peaks()
    gbpe = 2 if args.grad_dtype == "bfloat16" else 4
    alg_bytes, g_bytes = algorithmic_bytes(shapes, r, N, gbpe)

    nbuf = 1 if args.workload == 4 else 2
    bufs = make_inputs(args.workload, N, device, nbuf, args.grad_dtype)
    handles = build_handles(args.workload, r, N, tau, device, args.mode, grad_dtype=args.grad_dtype)
    torch.cuda.synchronize()

    from paper_2509_11254_b200 import StreamedStack

    stack = StreamedStack(handles, device)       # one stream per shape class
    # warm-up (includes the t = 0 refresh when tau > 0)
    for s in range(max(args.warmup, 3)):
        stack.step(bufs[s % nbuf])
    torch.cuda.synchronize()

    sampler = ClockSampler(local)
    sampler.start()
    l0 = sum(h.launch_count() for h in handles)
    ms_total = timed_steps(torch, stack, bufs, args.steps, barrier)
    l1 = sum(h.launch_count() for h in handles)
    clocks = sampler.stop()
    ms_total = reps.max_over_ranks(ms_total)
    ms_step = ms_total / args.steps
    value = reps.job_throughput(g_bytes, ms_step) / 1e9  # GB/s of gradient, all replicas

    # second pass over the same number of steps with per-launch CUDA events (roofline of the dominant kernel)
    for h in handles:
        h.profile_begin()
    prof_steps = min(args.steps, 20)
    t_now = [h.t for h in handles]
    ssp_only = [s for s in range(prof_steps)]
    for s in ssp_only:
        for h, g in zip(handles, bufs[s % nbuf]):
            h.step(g)
    fam = {}
    for h in handles:
        for k, (ms, ln) in h.profile_read().items():
            a = fam.setdefault(k, [0.0, 0])
            a[0] += ms
            a[1] += ln
    n_refresh = sum(1 for h, t0 in zip(handles, t_now) for s in range(prof_steps) if tau > 0 and (t0 + s) % tau == 0)
    n_ssp = prof_steps * len(handles) - n_refresh
    el = sum(m * n * c for m, n, c in shapes) * N
    per_family_bytes = {"project": (8 + gbpe) * el, "backproject": 4 * el, "residual": 8 * el}
    dom = max(("project", "backproject", "residual"), key=lambda k: fam.get(k, [0, 0])[0])
    # a family's kernels run once per handle per step; average duration of one launch set over all handles
    dom_ms_per_step = fam[dom][0] / prof_steps if prof_steps else float("nan")
    ssp_frac = n_ssp / max(1, prof_steps * len(handles))
    if dom != "project":
        ssp_frac = 1.0  # the tail kernels run on refresh steps too
    achieved = per_family_bytes[dom] * ssp_frac / dom_ms_per_step / 1e6 if dom_ms_per_step else None
    plans = [h.plan_info() for h in handles]
    single_pass = args.mode == "deferred" and all(p["single_pass"] for p in plans)
    kernel_name = "k_fused_step" if (dom == "project" and single_pass) else "k_" + dom
    # DRAM bytes per element of the dominant kernel from the committed ncu capture (profiles/), scaled to this
    # workload's elements; None for kernels without a current capture
    traffic = TRAFFIC_BYTES_PER_ELEMENT.get(kernel_name) if args.grad_dtype == "float32" else None   # captured with float32 G
    traffic = traffic * el * ssp_frac if traffic is not None else None
    roofline = {"bound": "hbm", "kernel": kernel_name, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak if achieved else None, "traffic": traffic, "peak_source": f"of {peak_kind}",
                "algorithmic_bytes_per_launch_set": per_family_bytes[dom],
                "per_family_ms_per_step": {k: round(v[0] / prof_steps, 4) for k, v in fam.items()},
                "note": "second pass of the same steps with per-launch CUDA events on the launching stream"}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": synth.WORKLOADS[args.workload]["name"], "matrices": [list(s) for s in shapes],
                       "r": r, "N": N, "refresh_period": tau, "mode": args.mode,
                       "launch_plan": [{k: p[k] for k in ("single_pass", "WC", "CS", "KC", "active_clusters")} for p in plans],
                       "l2": "inputs (%.2f GB of G per step, 2 alternating sets) exceed L2" % (g_bytes / 1e9),
                       "streams": len(handles), "grad_dtype": args.grad_dtype,
                       "parallelism": "replicas" if world > 1 else "single"},
            "min_bytes_frac": alg_bytes / ms_step / 1e6 / peak,
            "min_bytes_per_step": alg_bytes,
            "gpu_launches": l1 - l0, "clocks": clocks, "roofline": roofline}

    if rank == 0 and not args.no_e2e:
        # end to end through the host-buffer entry point: H2D of G and D2H of (P~, Q) inside the timed region
        e2e_steps = max(1, min(args.steps, 5))
        Gh = [torch.empty(g.shape, dtype=g.dtype).pin_memory() for g in bufs[0]]
        for gh, g in zip(Gh, bufs[0]):
            gh.copy_(g)
        Ph = [torch.empty(h.P_hat.shape, dtype=torch.float32).pin_memory() for h in handles]
        Qh = [torch.empty(h.Q.shape, dtype=torch.float32).pin_memory() for h in handles]
        stage = bufs[0]
        stack.step_host(Gh, stage, Ph, Qh)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for s in range(e2e_steps):
            stack.step_host(Gh, stage, Ph, Qh)
        torch.cuda.synchronize()
        dt = (time.perf_counter() - t0) / e2e_steps
        line["e2e"] = {"value": g_bytes / dt / 1e9, "unit": UNIT, "h2d_bytes_per_step": g_bytes,
                       "d2h_bytes_per_step": sum(p.numel() * 4 for p in Ph) + sum(q.numel() * 4 for q in Qh),
                       "steps": e2e_steps, "ms_per_step": dt * 1e3}
        del Gh

    for h in handles:
        h.close()
    del handles, bufs
    torch.cuda.empty_cache()

    if rank == 0 and world == 1 and not args.no_sweep:
        line["sweep_config5"] = sweep_config5(torch, device, peak, args.mode)
    if rank == 0 and world == 1 and not args.no_cpu:
        line["cpu_baseline"] = cpu_baseline(args.workload if args.workload != 4 else 4, r, N)
    if rank == 0:
        print(json.dumps(line))
    reps.close()


def main():
    args = parse()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
