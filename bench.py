#!/usr/bin/env python
"""Benchmark of the PowerSGD+ compression hot path on B200.

One "step" is one iteration of Algorithm 2 (without the optimizer) over ALL matrices of a
workload: error-feedback add, SSP-Comp or (every tau steps) SVD-Comp, residual update.

The metric is quoted per rank r on the single large matrix (m = 16384, n = 4096, N = 4 simulated
nodes, low-rank-plus-noise gradients), so that sweep is the body of the line: for every
r in {1, 4, 8, 16, 64, 128} the step latency (median and minimum over blocks of steps), the
gradient GB/s, the fraction of the 12-bytes-per-element HBM roofline, the dominant kernel with
its own achieved bandwidth, and the latency of one SVD refresh.  The headline `value` is the one
at r = 16, where the target binds.  The three model-shaped stacks follow as `stacks` (refreshes
amortised at their period).  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                  [--rank r] [--stacks 2,3,4|none] [--no-sweep] [--no-e2e] [--no-cpu]
                  [--single-pass auto|cluster|none|l2] [--mode deferred|eager]

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
SWEEP_SHAPE = (16384, 4096, 4)          # m, n, N of the sweep workload
SWEEP_RANKS = (1, 4, 8, 16, 64, 128)
HEADLINE_RANK = 16
# dram__bytes_read.sum + dram__bytes_write.sum per element of one launch, from the ncu captures summarised under
# profiles/ (small case of the same kernel; traffic grows in proportion to the elements).  None: no current capture.
TRAFFIC_BYTES_PER_ELEMENT = {"k_fused_step": 11.87, "k_project": 11.4, "k_project_tc<pend>": 11.49, "k_backproject": 4.1, "k_stream_step": 13.6}

# (rank, nodes, refresh period) of the stacks
STACK_DEFAULTS = {2: [(8, 8, 50)], 3: [(4, 16, 20), (16, 16, 20)], 4: [(32, 8, 100)]}


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300, help="timed steps of the headline (r = 16) measurement")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--rank", type=int, default=HEADLINE_RANK, help="rank of the headline measurement")
    ap.add_argument("--mode", default="deferred", choices=["eager", "deferred"])
    ap.add_argument("--single-pass", default="auto", choices=["auto", "cluster", "none", "l2"])
    ap.add_argument("--pending-tc", default=None, choices=["auto", "always", "never"],
                    help="two-pass steps: fold the pending residual in on the tensor cores (default: the library's choice per rank)")
    ap.add_argument("--stacks", default="2,3,4", help="model-shaped stacks to add (workload ids), or 'none'")
    ap.add_argument("--no-sweep", action="store_true", help="only the headline rank")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--grad-dtype", default="float32", choices=["float32", "bfloat16"],
                    help="storage type of the gradients G of the headline measurement (bfloat16: 2 bytes per element read instead of 4)")
    ap.add_argument("--refresh-period", type=int, default=0, help="refresh period tau of the headline handle (0: SSP steps only, as the metric asks)")
    ap.add_argument("--small", action="store_true", help="a quarter of the sweep matrix (m = 4096): for profiler captures")
    return ap.parse_args()


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM, "fallback"


def host_cores():
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count()


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


def algorithmic_bytes(shapes, r, N, g_bytes_per_element=4):
    """Minimum traffic of a step: read G, read E, write E per element (12 B with float32 G) plus the P/Q traffic."""
    el = sum(m * n * c for m, n, c in shapes) * N
    pq = sum(4 * (2 * N * m * r + 2 * m * r + 2 * N * n * r + 2 * n * r) * c for m, n, c in shapes)
    return (8 + g_bytes_per_element) * el + pq, g_bytes_per_element * el


FAMILY_BYTES = {"project": 12, "backproject": 4, "residual": 8}   # algorithmic bytes per element of one launch set


def kernel_name(family, r, step_kernel):
    if family == "project":
        if step_kernel == 1:
            return "k_fused_step"
        if step_kernel == 2:
            return "k_stream_step"
        if step_kernel == 3:
            return "k_project_tc<pend>"
        return "k_project_tc" if r > 16 else "k_project"
    return ("k_%s_tc" if r > 16 else "k_%s") % family


# ----------------------------------------------------------------------------
# timing helpers
# ----------------------------------------------------------------------------
def time_blocks(torch, step_fn, total_steps, block=50, min_seconds=0.0, max_blocks=40):
    """Blocks of `block` steps timed with CUDA events on the current stream until `total_steps` steps and
    `min_seconds` of device time have passed.  Returns (ms per step of every block, steps done)."""
    per_block, done, spent = [], 0, 0.0
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    while (done < total_steps or spent < min_seconds * 1e3) and len(per_block) < max_blocks:
        k = min(block, max(1, total_steps - done)) if done < total_steps else block
        torch.cuda.synchronize()
        ev0.record()
        for s in range(k):
            step_fn(done + s)
        ev1.record()
        torch.cuda.synchronize()
        ms = ev0.elapsed_time(ev1)
        per_block.append(ms / k)
        done += k
        spent += ms
    return per_block, done


def family_profile(handles, step_fn, steps):
    """Second pass with per-launch CUDA events on the launching stream: milliseconds per step of every kernel family."""
    for h in handles:
        h.profile_begin()
    for s in range(steps):
        step_fn(s)
    fam = {}
    for h in handles:
        for k, (ms, ln) in h.profile_read().items():
            a = fam.setdefault(k, [0.0, 0])
            a[0] += ms
            a[1] += ln
    return {k: (v[0] / steps, v[1] / steps) for k, v in fam.items() if v[1]}


def roofline_entry(fam, r, step_kernel, elements, peak, peak_kind):
    dom = max(("project", "backproject", "residual"), key=lambda k: fam.get(k, (0.0, 0))[0])
    ms = fam[dom][0]
    name = kernel_name(dom, r, step_kernel)
    achieved = FAMILY_BYTES[dom] * elements / ms / 1e6
    tb = TRAFFIC_BYTES_PER_ELEMENT.get(name)
    return {"bound": "hbm", "kernel": name, "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
            "frac": round(achieved / peak, 4), "traffic": tb * elements if tb is not None else None,
            "peak_source": f"of {peak_kind}", "ms_per_launch_set": round(ms, 4),
            "algorithmic_bytes_per_launch_set": FAMILY_BYTES[dom] * elements,
            "per_family_ms_per_step": {k: round(v[0], 4) for k, v in fam.items()}}


# ----------------------------------------------------------------------------
# the sweep (workload 5)
# ----------------------------------------------------------------------------
PENDING_TC = None      # --pending-tc: which projection folds the pending residual in (None: the library's choice)


def sweep_point(torch, device, r, bufs, mode, single_pass, steps, min_seconds, peak, peak_kind, refresh=True):
    from paper_2509_11254_b200 import PowerSGDPlus

    N, m, n = bufs[0].shape[1], bufs[0].shape[2], bufs[0].shape[3]
    h = PowerSGDPlus(m, n, r, N, refresh_period=0, seed=5, device=device, mode=mode, single_pass=single_pass, pending_tc=PENDING_TC)
    for s in range(5):
        h.step(bufs[s % 2])
    l0 = h.launch_count()
    blocks, done = time_blocks(torch, lambda s: h.step(bufs[s % 2]), steps, min_seconds=min_seconds)
    launches = h.launch_count() - l0
    fam = family_profile([h], lambda s: h.step(bufs[s % 2]), 20)
    plan = h.plan_info()
    out = {"r": r, "step_ms": round(statistics.median(blocks), 4), "step_ms_min": round(min(blocks), 4), "steps_timed": done,
           "blocks": len(blocks)}
    alg, gb = algorithmic_bytes([(m, n, 1)], r, N)
    ms = out["step_ms"]
    out.update(grad_GBps=round(gb / ms / 1e6, 1), min_bytes_frac=round(alg / ms / 1e6 / peak, 4),
               path={0: ("two-pass" if (mode == "deferred" and r <= 16) else "three-pass"), 1: "single-pass (cluster kernel)",
                     2: "single-pass (L2-pipelined kernel)", 3: "two-pass (pending residual folded in on the tensor cores)"}[plan["step_kernel"]],
               roofline=roofline_entry(fam, r, plan["step_kernel"], m * n * N, peak, peak_kind),
               launches_per_step=round(launches / done, 2))
    if refresh:
        h.refresh(bufs[0])
        rb, _ = time_blocks(torch, lambda s: h.refresh(bufs[s % 2]), 3, block=1)
        out["refresh_ms"] = round(statistics.median(rb), 3)
        out["refresh_ms_min"] = round(min(rb), 3)
    out["flags"] = h.last_status()
    return out, h, launches, done


# ----------------------------------------------------------------------------
# the model-shaped stacks (workloads 2, 3, 4)
# ----------------------------------------------------------------------------
def stack_bench(torch, device, workload, r, N, tau, mode, single_pass, peak, peak_kind):
    from paper_2509_11254_b200 import PowerSGDPlus, StreamedStack, synth

    shapes = synth.STACKS[workload]
    nbuf = 1 if workload == 4 else 2
    bufs = [[synth.make_gradients_torch(workload, m, n, N, c, step=b, device=device) for (m, n, c) in shapes] for b in range(nbuf)]
    handles = [PowerSGDPlus(m, n, r, N, refresh_period=tau, seed=1 + i, count=c, device=device, mode=mode, single_pass=single_pass, pending_tc=PENDING_TC)
               for i, (m, n, c) in enumerate(shapes)]
    stack = StreamedStack(handles, device)
    for s in range(3):            # t = 0 is a refresh
        stack.step(bufs[s % nbuf])
    # SSP steps only (t = 3 .. < tau), then one refresh step on its own; the amortised figure follows from the two
    n_ssp = max(4, min(40 if workload != 4 else 10, tau - 8))
    blocks, done = time_blocks(torch, lambda s: stack.step(bufs[s % nbuf]), n_ssp, block=max(1, n_ssp // 2), max_blocks=2)
    ssp_ms = statistics.median(blocks)
    fam = family_profile(handles, lambda s: [h.step(g) for h, g in zip(handles, bufs[s % nbuf])], 3)
    plans = [h.plan_info() for h in handles]
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    ev0.record()
    for h, g in zip(handles, bufs[0]):
        h.refresh(g)
    ev1.record()
    torch.cuda.synchronize()
    refresh_ms = ev0.elapsed_time(ev1)
    flags = [h.last_status() for h in handles]
    alg, gb = algorithmic_bytes(shapes, r, N)
    ms = ((tau - 1) * ssp_ms + refresh_ms) / tau if tau > 0 else ssp_ms
    el = sum(m * n * c for m, n, c in shapes) * N
    out = {"workload": synth.WORKLOADS[workload]["name"], "r": r, "N": N, "refresh_period": tau,
           "ms_per_step": round(ms, 4), "ssp_step_ms": round(ssp_ms, 4), "refresh_step_ms": round(refresh_ms, 3),
           "grad_GBps": round(gb / ms / 1e6, 1), "min_bytes_frac": round(alg / ms / 1e6 / peak, 4),
           "min_bytes_frac_ssp_only": round(alg / ssp_ms / 1e6 / peak, 4),
           "roofline": roofline_entry(fam, r, plans[0]["step_kernel"], el, peak, peak_kind),
           "gradient_sets": nbuf, "g_bytes_per_step": gb, "flags": flags}
    for h in handles:
        h.close()
    del handles, bufs, stack
    torch.cuda.empty_cache()
    return out


# ----------------------------------------------------------------------------
# CPU baseline: the oracle as it stands, on a bounded sample
# ----------------------------------------------------------------------------
def cpu_baseline(r, budget_s=10.0, small=False):
    """SSP steps of the oracle on the sweep matrix at rank r, and its dense-SVD refresh on a row sample of it."""
    import numpy as np

    from oracle import psgd_oracle as orc
    from paper_2509_11254_b200 import synth

    m, n, N = SWEEP_SHAPE
    ms_rows = n                    # the SSP sample: a square (n x n) row sample of the sweep matrix, all nodes (the method needs m >= n)
    G = synth.make_gradients(5, ms_rows, n, N, step=1)
    o = orc.PowerSGDPlusOracle(ms_rows, n, r, N, 0, synth.init_Q(n, r))
    o.step(G)
    reps, t0 = 0, time.perf_counter()
    while True:
        o.step(G)
        reps += 1
        if time.perf_counter() - t0 > budget_s or reps >= 20:
            break
    dt = (time.perf_counter() - t0) / reps
    val = G.nbytes / dt / 1e9
    # refresh: svd_comp on a square row sample (n x n): the dense SVD is what the oracle's refresh costs
    sv_rows = n if not small else n // 4
    Gs = synth.make_gradients(5, sv_rows, n, N, step=2)
    t1 = time.perf_counter()
    orc.svd_comp(Gs.astype(np.float64), r)
    svd_s = time.perf_counter() - t1
    return {"value": val, "unit": UNIT, "cores": host_cores(), "kind": "oracle",
            "sample": f"{reps} SSP steps (r={r}) of a {ms_rows}x{n} row sample of the {m}x{n} sweep matrix, N={N}; "
                      f"refresh: one svd_comp (dense SVD) of a {sv_rows}x{n} row sample; numpy float64, OpenBLAS threads = cores",
            "ssp_step_ms_sample": round(dt * 1e3, 2), "ssp_step_ms_scaled_to_full_matrix": round(dt * 1e3 * m / ms_rows, 1),
            "refresh_ms_sample": round(svd_s * 1e3, 1)}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np  # noqa: F401

    from oracle import psgd_oracle as orc
    from paper_2509_11254_b200 import synth

    m, n, N = SWEEP_SHAPE
    r = args.rank
    rows = n                       # a square row sample: the method needs m >= n
    o = orc.PowerSGDPlusOracle(rows, n, r, N, 0, synth.init_Q(n, r))
    Gs = [synth.make_gradients(5, rows, n, N, step=s) for s in range(2)]
    steps = max(1, min(args.steps, 20))
    for w in range(max(1, min(args.warmup, 3))):
        o.step(Gs[w % 2])
    t0 = time.perf_counter()
    for s in range(steps):
        o.step(Gs[s % 2])
    dt = time.perf_counter() - t0
    val = steps * Gs[0].nbytes / dt / 1e9
    sample = f"each step = one SSP step (r={r}) of a {rows}x{n} row sample of the {m}x{n} sweep matrix, N={N}"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": args.warmup, "ms_per_step": dt / steps * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "sweep", "m": m, "n": n, "N": N, "r": r, "sample": sample},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": host_cores(), "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ----------------------------------------------------------------------------
# GPU arm
# ----------------------------------------------------------------------------
def run_ours(args):
    import torch

    from paper_2509_11254_b200.replicas import Replicas, env_rank

    rank, local, world = env_rank()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local)
    device = f"cuda:{local}"
    reps = Replicas("nccl", device)

    from paper_2509_11254_b200 import synth

    m, n, N = SWEEP_SHAPE
    if args.small:
        m //= 4
    peak, peak_kind = peaks()
    bufs = [synth.make_gradients_torch(5, m, n, N, 1, step=b, device=device) for b in range(2)]
    r = args.rank
    gbpe = 2 if args.grad_dtype == "bfloat16" else 4
    alg_bytes, g_bytes = algorithmic_bytes([(m, n, 1)], r, N, gbpe)
    hbufs = [b.to(torch.bfloat16) for b in bufs] if gbpe == 2 else bufs

    # ---- headline: the step at the headline rank, on every replica, max over ranks ----
    from paper_2509_11254_b200 import PowerSGDPlus

    h = PowerSGDPlus(m, n, r, N, refresh_period=args.refresh_period, seed=5, device=device, mode=args.mode, single_pass=args.single_pass, pending_tc=PENDING_TC,
                     grad_dtype=args.grad_dtype)
    for s in range(max(args.warmup, 3)):
        h.step(hbufs[s % 2])
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    sampler.start()
    l0 = h.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps.barrier()
    torch.cuda.synchronize()
    ev0.record()
    for s in range(args.steps):
        h.step(hbufs[s % 2])
    ev1.record()
    torch.cuda.synchronize()
    reps.barrier()
    ms_total = reps.max_over_ranks(ev0.elapsed_time(ev1))
    launches = h.launch_count() - l0
    ms_step = ms_total / args.steps
    value = reps.job_throughput(g_bytes, ms_step) / 1e9          # GB/s of gradient, all replicas
    # a longer look at the same step: blocks of 50 steps for at least half a second of device time
    # (--small is the profiler's case: no more launches than needed)
    blocks, done = time_blocks(torch, lambda s: h.step(hbufs[s % 2]), 100, min_seconds=0.5) if not args.small else ([ms_step], args.steps)
    clocks = sampler.stop()
    fam = family_profile([h], lambda s: h.step(hbufs[s % 2]), 20 if not args.small else 2)
    plan = h.plan_info()
    roofline = roofline_entry(fam, r, plan["step_kernel"], m * n * N, peak, peak_kind)
    roofline["note"] = "dominant kernel family of the headline step; a second pass of 20 steps with per-launch CUDA events on the launching stream"

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": "sweep", "m": m, "n": n, "N": N, "ranks": list(SWEEP_RANKS), "headline_rank": r,
                       "refresh_period": args.refresh_period, "mode": args.mode, "single_pass": args.single_pass, "pending_tc": args.pending_tc or "auto", "grad_dtype": args.grad_dtype,
                       "gradients": "low rank (s_k = 0.9^k, 256 terms) plus 5 % Gaussian noise, 2 alternating sets generated on the device",
                       "l2": "inputs (%.2f GB of G and as much of E per step) exceed L2" % (g_bytes / 1e9),
                       "parallelism": "replicas" if world > 1 else "single"},
            "min_bytes_frac": alg_bytes / ms_step / 1e6 / peak,
            "min_bytes_per_step": alg_bytes,
            "step_ms_blocks": {"median": round(statistics.median(blocks), 4), "min": round(min(blocks), 4), "blocks": len(blocks), "steps": done},
            "gpu_launches": launches, "clocks": clocks, "roofline": roofline}

    if rank == 0 and not args.no_e2e:
        # end to end through the host-buffer entry point: H2D of G and D2H of (P~, Q) inside the timed region
        e2e_steps = 5
        Gh = torch.empty(hbufs[0].shape, dtype=hbufs[0].dtype).pin_memory()
        Gh.copy_(hbufs[0])
        Ph = torch.empty(h.P_hat.shape, dtype=torch.float32).pin_memory()
        Qh = torch.empty(h.Q.shape, dtype=torch.float32).pin_memory()
        stage = torch.empty_like(hbufs[0])
        h.step_host(Gh, stage, Ph, Qh)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for s in range(e2e_steps):
            h.step_host(Gh, stage, Ph, Qh)
        torch.cuda.synchronize()
        dt = (time.perf_counter() - t0) / e2e_steps
        line["e2e"] = {"value": g_bytes / dt / 1e9, "unit": UNIT, "h2d_bytes_per_step": g_bytes,
                       "d2h_bytes_per_step": Ph.numel() * 4 + Qh.numel() * 4, "steps": e2e_steps, "ms_per_step": dt * 1e3}
        del Gh, stage
    h.close()
    del h
    torch.cuda.empty_cache()

    if rank == 0 and world == 1 and not args.no_sweep:
        sweep = []
        for rr in SWEEP_RANKS:
            pt, hh, _, _ = sweep_point(torch, device, rr, bufs, args.mode, args.single_pass, 100, 0.5, peak, peak_kind)
            hh.close()
            del hh
            torch.cuda.empty_cache()
            sweep.append(pt)
        line["sweep"] = sweep
    del bufs
    torch.cuda.empty_cache()
    if rank == 0 and world == 1 and args.stacks != "none":
        stacks = []
        for w in [int(x) for x in args.stacks.split(",") if x]:
            for (sr, sN, stau) in STACK_DEFAULTS[w]:
                stacks.append(stack_bench(torch, device, w, sr, sN, stau, args.mode, args.single_pass, peak, peak_kind))
        line["stacks"] = stacks
    if rank == 0 and world == 1 and not args.no_cpu:
        line["cpu_baseline"] = cpu_baseline(r, small=args.small)
    if rank == 0:
        print(json.dumps(line))
    reps.close()


def main():
    global PENDING_TC
    args = parse()
    PENDING_TC = args.pending_tc
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
