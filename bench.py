#!/usr/bin/env python
"""Benchmark of the CORE round on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A step is one pass of the whole path over the projection-dimension sweep workload:
d = 1e9 fp32 coordinates, n = 2 machines, and for every m in {8, 64, 512, 4096} one round
(project -> aggregate -> reconstruct).  The metric counts coordinate x vector pairs: a step
processes d * sum(m) of them per kernel.  The path does not shard (all machines are simulated
on one GPU, no collectives), so N > 1 runs N independent replicas, one per GPU.

Prints one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "CORE round throughput (coords x m projected+reconstructed/s)"
UNIT = "coord*vector pairs/s"
SEED_DATA, SEED_XI = 0, 1
SM_COUNT = 148
# Philox4x32-10 multiplies two counter words by constants in each of ten rounds.  The first two rounds
# split into a part that depends on the vector alone and one that depends on the coordinate block alone,
# which the kernels evaluate once per thread; what every counter must still execute is the 16 32x32->64-bit
# multiplies of rounds 2..9, and a counter yields four Gaussians: 4 wide multiplies per pair.
WIDE_MULS_PER_GAUSSIAN = 4
# Measured on B200 (tests/test_gpu_pipe_rates.py, profiles/pipe_rates.md): the multiplier behind mul.wide.u32
# retires 32 lanes per clock per SM (a warp instruction holds its pipe for four clocks), against 128 for fp32
# multiply-adds and 64 for logic ops; Philox's rounds 2..9 alone take 75.2 scheduler cycles per warp and counter.
WIDE_MUL_LANES_PER_CLK_SM = 32
PHILOX_ONLY_CYCLES_PER_COUNTER = 75.2
# Planning count of the plain issue bound: 16 lane-instructions per Gaussian for the generator plus the
# consumer's multiply-adds (n per pair in the projection, 1 in the reconstruction), 128 lanes per clock per SM.
PLANNING_INSTR_PER_GAUSSIAN = 16
ISSUE_LANES_PER_CLK_SM = 128


def alu_bounds(sm_max_mhz: float):
    """(multiplier peak, Philox-only floor) in pairs per second at the given SM clock."""
    f = sm_max_mhz * 1e6
    peak = SM_COUNT * WIDE_MUL_LANES_PER_CLK_SM * f / WIDE_MULS_PER_GAUSSIAN
    floor = SM_COUNT * 4 * f / PHILOX_ONLY_CYCLES_PER_COUNTER * 32 * 4
    return peak, floor


def planning_bound(sm_max_mhz: float, fmas_per_pair: int) -> float:
    """The plain issue bound R / (c_g + c_f) in pairs per second."""
    return SM_COUNT * ISSUE_LANES_PER_CLK_SM * sm_max_mhz * 1e6 / (PLANNING_INSTR_PER_GAUSSIAN + fmas_per_pair)


ROUND_KERNEL_SOURCES = ("core_internal.h", "core_project.cu", "core_reconstruct.cu", "core_rng.cuh")


def csrc_digest() -> str:
    """sha256 over the sources of the two kernels the stored DRAM counters cover (the digest the counters
    were stamped with when they were taken): ties the counters to the code they describe."""
    import hashlib
    h = hashlib.sha256()
    for name in ROUND_KERNEL_SOURCES:
        h.update(name.encode())
        h.update(open(os.path.join(ROOT, "paper_2309_13307_b200", "csrc", name), "rb").read())
    return h.hexdigest()


def stored_traffic(kernel: str, d: int, m: int):
    """DRAM bytes per launch from the committed ncu capture (profiles/round_kernels_dram.json), scaled by the
    number of coordinates (traffic of both kernels is proportional to d); None if the kernels have changed
    since the capture or no capture exists for this kernel."""
    try:
        rec = json.load(open(os.path.join(ROOT, "profiles", "round_kernels_dram.json")))
    except (OSError, ValueError):
        return None
    if rec.get("csrc_sha256") != csrc_digest():
        return None
    best = None
    for cap in rec.get("captures", []):
        if cap["kernel"] == kernel and (best is None or abs(cap["m"] - m) < abs(best["m"] - m)):
            best = cap
    if best is None:
        return None
    return int(best["dram_bytes"] * (d / best["d"]))


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--d", type=int, default=None, help="override the coordinate count (development)")
    ap.add_argument("--m", type=int, nargs="*", default=None, help="override the m sweep (development)")
    ap.add_argument("--workload", default="sweep", choices=["sweep", "leastsq", "resnet50", "gpt2small", "tiny"],
                    help="sweep: the headline CORE round; resnet50 / gpt2small / tiny: the round at the other evaluation "
                         "shapes; leastsq: the CORE-GD step (secondary lines)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="skip the short passes over the other evaluation shapes")
    return ap.parse_args()


# ---- clocks ---------------------------------------------------------------------------

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "200"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ---- CPU oracle leg -----------------------------------------------------------------------

def oracle_mini_round(d_s: int, m_s: int, n_s: int, threads: int):
    """One whole oracle round on a bounded sample; returns (seconds, units)."""
    import math
    from concurrent.futures import ThreadPoolExecutor

    import numpy as np

    import core_inputs
    import oracle

    G = core_inputs.gradients(n_s, d_s, seed=SEED_DATA).numpy()
    oracle.lib()
    piece = max(4, (d_s // threads + 3) // 4 * 4)
    cuts = list(range(0, d_s, piece)) + [d_s]
    spans = list(zip(cuts[:-1], cuts[1:]))
    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=threads) as ex:
        def proj(span):
            return [[oracle.project_slice(SEED_XI, 0, j, G[i], span[0], span[1]) for j in range(m_s)]
                    for i in range(n_s)]
        parts = list(ex.map(proj, spans))
        P = np.array([[math.fsum(p[i][j] for p in parts) for j in range(m_s)] for i in range(n_s)])
        pbar = oracle.aggregate(P)
        list(ex.map(lambda span: oracle.reconstruct_slice(SEED_XI, 0, pbar, span[0], span[1]), spans))
    dt = time.perf_counter() - t0
    return dt, d_s * m_s


def cpu_baseline_sample(budget_s: float = 15.0):
    threads = max(1, min(os.cpu_count() or 1, 64))
    n_s, m_s = 2, 8
    d_s = 1 << 18
    dt, units = oracle_mini_round(d_s, m_s, n_s, threads)          # calibration
    scale = max(1, min(1024, int(budget_s / max(dt, 1e-3))))
    if scale > 1:
        d_s *= scale
        dt, units = oracle_mini_round(d_s, m_s, n_s, threads)
    # the same oracle on one core, on a sample sized for about the same wall time
    d_1 = max(1 << 16, d_s // threads // 4 * 4)
    dt_1, units_1 = oracle_mini_round(d_1, m_s, n_s, 1)
    return {"value": units / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"one whole oracle round (project+aggregate+reconstruct, fp64) at d={d_s}, m={m_s}, "
                      f"n={n_s}, N(0,1) gradients, coordinate range split over {threads} host threads; "
                      f"{dt:.1f} s",
            "one_core": {"value": units_1 / dt_1, "unit": UNIT, "cores": 1,
                         "sample": f"the same round at d={d_1} on one host thread; {dt_1:.1f} s"}}


def run_reference(args):
    """The reference arm of this build is the CPU oracle, as it stands, on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    threads = max(1, min(os.cpu_count() or 1, 64))
    n_s, m_s, d_s = 2, 8, 1 << 24
    for _ in range(args.warmup):
        oracle_mini_round(1 << 16, m_s, n_s, threads)
    total_t, total_u = 0.0, 0
    for _ in range(args.steps):
        dt, units = oracle_mini_round(d_s, m_s, n_s, threads)
        total_t += dt
        total_u += units
    value = total_u / total_t
    sample = (f"each step: one whole oracle round at d={d_s}, m={m_s}, n={n_s} (a bounded sample of the "
              f"d=1e9 sweep workload), split over {threads} host threads")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total_t / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "sweep: d=1e9 fp32, n=2, m in {8,64,512,4096} (bounded sample per step)"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


# ---- GPU leg ---------------------------------------------------------------------------------

def slowest_rank(seconds_or_ms: float, world: int, device) -> float:
    """Maximum of a per-rank duration over all ranks (identity for one rank).  The replicas are
    independent, so the job is as slow as its slowest rank."""
    if world <= 1:
        return seconds_or_ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([seconds_or_ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(units_per_step: int, steps: int, world: int, elapsed_ms: float) -> float:
    """Pairs per second over all replicas: every rank processes units_per_step per step (weak scaling)."""
    return world * units_per_step * steps / (elapsed_ms * 1e-3)


def run_ours(args):
    import torch
    import torch.distributed as dist

    import core_inputs
    import paper_2309_13307_b200 as core_mod

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    core_mod.lib()                                   # fails loudly if the CUDA library is missing
    w = core_inputs.WORKLOADS[args.workload]
    d = args.d or w.d
    ms = tuple(args.m) if args.m else w.m
    n = w.n
    G = core_inputs.gradients(n, d, seed=SEED_DATA + rank, dist=w.dist, dtype=w.dtype, device="cuda")
    ctxs = {m: core_mod.Core(SEED_XI, d, m) for m in ms}
    P = {m: torch.empty((n, m), dtype=torch.float32, device="cuda") for m in ms}
    pbar = {m: torch.empty(m, dtype=torch.float32, device="cuda") for m in ms}
    gt = torch.empty(d, dtype=torch.float32, device="cuda")
    units_per_step = d * sum(ms)

    def ev():
        e = torch.cuda.Event(enable_timing=True)
        e.record()
        return e

    marks = []                                        # (m, e0, e_proj, e_agg, e_rec) per timed round

    def step(timed: bool):
        for m in ms:
            c = ctxs[m]
            e0 = ev() if timed else None
            c.core_project(G, P[m])
            e1 = ev() if timed else None
            c.core_aggregate(P[m], pbar[m])
            e2 = ev() if timed else None
            c.core_reconstruct(pbar[m], gt)
            e3 = ev() if timed else None
            c.core_set_round(c.core_get_round() + 1)
            if timed:
                marks.append((m, e0, e1, e2, e3))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step(False)
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(args.steps):
        step(True)
    stop.record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    elapsed_ms = slowest_rank(start.elapsed_time(stop), world, "cuda")
    value = whole_job_throughput(units_per_step, args.steps, world, elapsed_ms)

    # per-kernel times (averages over the timed launches)
    per_m = {}
    for m in ms:
        rows = [r for r in marks if r[0] == m]
        tp = statistics.mean(r[1].elapsed_time(r[2]) for r in rows)
        tr = statistics.mean(r[3].elapsed_time(r[4]) for r in rows)
        ta = statistics.mean(r[2].elapsed_time(r[3]) for r in rows)
        per_m[m] = (tp, ta, tr)

    # end to end through the host-buffer entry point
    e2e = None
    if not args.no_e2e:
        Gh = torch.empty((n, d), dtype=G.dtype).pin_memory()
        Gh.copy_(G)
        gt_h = torch.empty(d, dtype=torch.float32).pin_memory()
        pbar_h = {m: torch.empty(m, dtype=torch.float32).pin_memory() for m in ms}
        for m in ms:                                   # warm-up of every context: slabs, streams, workspace
            ctxs[m].core_round_host(Gh, pbar_h[m], gt_h)
        barrier()
        e2e_steps = 2
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            for m in ms:
                ctxs[m].core_round_host(Gh, pbar_h[m], gt_h)
        torch.cuda.synchronize()
        dt = slowest_rank(time.perf_counter() - t0, world, "cuda")
        e2e = {"value": whole_job_throughput(units_per_step, e2e_steps, world, dt * 1e3), "unit": UNIT,
               "h2d_bytes_per_step": len(ms) * n * d * G.element_size(),
               "d2h_bytes_per_step": len(ms) * (d * 4) + sum(ms) * 4,
               "steps": e2e_steps, "how": "core_round_host from pinned host buffers, host clock around the "
                                          "blocking calls (each returns after its last copy)"}
        del Gh, gt_h

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # roofline of the dominant kernel (largest share of the step)
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except OSError:
        pass
    sm_max = (clocks or {}).get("sm_max_mhz") or peaks.get("sm_max_mhz") or 1965.0
    hbm_peak = peaks.get("hbm_gbs", 6650.0) * 1e9
    hbm_src = "of measured" if "hbm_gbs" in peaks else "of fallback"
    # The binding unit of both round kernels is the pipe that executes the 32x32->64-bit multiplies of
    # Philox: 16 per counter = 4 per pair after hoisting, 32 lanes per clock per SM (profiles/pipe_rates.md).
    peak_pairs, floor_pairs = alu_bounds(sm_max)
    wide_peak = peak_pairs * WIDE_MULS_PER_GAUSSIAN                        # wide multiplies per second
    kernels = []
    for m in ms:
        tp, ta, tr = per_m[m]
        kernels.append(("project", m, tp, n * d * G.element_size(), n))
        kernels.append(("reconstruct", m, tr, 4 * d + 4 * m, 1))
    name, m_dom, t_dom, hbm_bytes, fmas_dom = max(kernels, key=lambda k: k[2])
    pairs_dom = d * m_dom / (t_dom * 1e-3)
    roofline = {"bound": "alu", "kernel": f"{name} m={m_dom}", "achieved": pairs_dom * WIDE_MULS_PER_GAUSSIAN / 1e12,
                "peak": wide_peak / 1e12, "unit": "T wide-multiply/s", "frac": pairs_dom / peak_pairs,
                "traffic": stored_traffic(name, d, m_dom),
                "algorithmic_bytes": hbm_bytes, "ms_per_launch": t_dom,
                "peak_source": f"148 SM x {WIDE_MUL_LANES_PER_CLK_SM} wide multiplies/clk/SM (measured, profiles/pipe_rates.md) x "
                               f"{sm_max:.0f} MHz (max SM clock); {WIDE_MULS_PER_GAUSSIAN} wide multiplies per pair "
                               f"(16 per counter: rounds 2..9; rounds 0 and 1 are hoisted)",
                "pairs_per_s": pairs_dom, "peak_pairs_per_s": peak_pairs,
                "model_floor_pairs_per_s": floor_pairs,
                "model_floor_source": f"Philox rounds 2..9 alone: {PHILOX_ONLY_CYCLES_PER_COUNTER} scheduler cycles per warp and "
                                      f"counter (measured); frac_of_floor = {pairs_dom / floor_pairs:.3f}",
                "frac_of_floor": pairs_dom / floor_pairs,
                "frac_planning": pairs_dom / planning_bound(sm_max, fmas_dom),
                "planning_source": f"issue bound R/(c_g+c_f): 148 SM x 128 lanes x clock / ({PLANNING_INSTR_PER_GAUSSIAN} + "
                                   f"{fmas_dom}) lane-instructions per pair",
                "hbm_frac": (hbm_bytes / (t_dom * 1e-3)) / hbm_peak, "hbm_peak": hbm_src}
    sweep = []
    for kname, m, t_ms, hb, fmas in kernels:
        pps = d * m / (t_ms * 1e-3)
        sweep.append({"kernel": kname, "m": m, "ms": round(t_ms, 4), "pairs_per_s": pps,
                      "alu_frac": pps / peak_pairs, "floor_frac": pps / floor_pairs,
                      "planning_frac": pps / planning_bound(sm_max, fmas), "hbm_frac": hb / (t_ms * 1e-3) / hbm_peak})

    in_gb = n * d * G.element_size() / 1e9
    # the other evaluation shapes, after the headline's timed region (each with its own clock record)
    configs = None
    if args.workload == "sweep" and not args.no_configs and args.d is None and args.m is None:
        del G, gt, P, pbar, ctxs
        torch.cuda.empty_cache()
        configs = [measure_round_config(core_mod, "tiny", local), measure_leastsq(core_mod, local)]
        for name in ("resnet50", "gpt2small"):
            configs.append(measure_round_config(core_mod, name, local))
            torch.cuda.empty_cache()

    cpu = None if args.no_cpu else cpu_baseline_sample()
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": elapsed_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{w.name}: d={d} {w.dtype}, n={n}, {w.dist} gradients, m in {list(ms)}; one round per m",
                   "l2": f"inputs ({in_gb:.2f} GB of gradients per replica) against a 126 MB L2; no flush",
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": 4 * len(ms) * args.steps,
        "roofline": roofline, "sweep": sweep, "configs": configs, "cpu_baseline": cpu,
    }
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def measure_round_config(core_mod, name: str, local: int, min_seconds: float = 1.5) -> dict:
    """Timed passes of one round (project, aggregate, reconstruct) at one of the other evaluation shapes,
    with its own clock record.  The number of passes is chosen so that the timed region lasts about
    min_seconds (the clock sampler needs a few samples under load)."""
    import torch

    import core_inputs

    w = core_inputs.WORKLOADS[name]
    m = w.m[0]
    G = core_inputs.workload_gradients(name, seed=SEED_DATA, device="cuda")
    ctx = core_mod.Core(SEED_XI, w.d, m)
    P = torch.empty((w.n, m), dtype=torch.float32, device="cuda")
    pbar = torch.empty(m, dtype=torch.float32, device="cuda")
    gt = torch.empty(w.d, dtype=torch.float32, device="cuda")

    def one(marks=None):
        e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        e[0].record()
        ctx.core_project(G, P)
        e[1].record()
        ctx.core_aggregate(P, pbar)
        e[2].record()
        ctx.core_reconstruct(pbar, gt)
        e[3].record()
        ctx.core_set_round(ctx.core_get_round() + 1)
        if marks is not None:
            marks.append(e)

    for _ in range(3):
        one()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(3):
        one()
    torch.cuda.synchronize()
    per = max((time.perf_counter() - t0) / 3, 1e-6)
    steps = max(5, min(20000, int(min_seconds / per)))
    sampler = ClockSampler(local)
    sampler.start()
    marks = []
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(steps):
        one(marks)
    stop.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = start.elapsed_time(stop) / steps
    keep = marks[:: max(1, len(marks) // 200)]            # per-kernel averages from a sample of the passes
    tp = statistics.mean(e[0].elapsed_time(e[1]) for e in keep)
    tr = statistics.mean(e[2].elapsed_time(e[3]) for e in keep)
    sm_max = clocks.get("sm_max_mhz") or 1965.0
    peak_pairs, _ = alu_bounds(sm_max)
    units = w.d * m
    in_bytes = w.n * w.d * G.element_size()
    return {"workload": f"{name}: d={w.d} {w.dtype}, n={w.n}, {w.dist} gradients, m={m}", "steps": steps, "ms": ms,
            "pairs_per_s": units / (ms * 1e-3), "project_ms": tp, "reconstruct_ms": tr,
            "project_pairs_per_s": units / (tp * 1e-3), "reconstruct_pairs_per_s": units / (tr * 1e-3),
            "frac": units / (tp * 1e-3) / peak_pairs, "reconstruct_frac": units / (tr * 1e-3) / peak_pairs,
            "bound": "alu", "gpu_launches": 4 * steps,
            "l2": ("inputs larger than the 126 MB L2" if in_bytes > 126e6 else
                   "inputs fit in L2 (launch-bound case; no flush)"),
            "clocks": clocks}


def measure_leastsq(core_mod, local: int, min_steps: int = 50, min_seconds: float = 1.5) -> dict:
    """The least-squares CORE-GD step (n=8 machines, A_i 2048 x 8192, m=64), bound by the streaming pass
    over A, with its own clock record."""
    import torch

    import core_inputs

    ls_in = core_inputs.least_squares(n=8, rows=2048, d=8192, seed=SEED_DATA, device="cuda")
    n, rows, d = ls_in.A.shape
    m = 64
    h = float(1.0 / core_inputs.lipschitz_constant(ls_in.A, iters=30))
    ctx = core_mod.Core(SEED_XI, d, m)
    ls = core_mod.LeastSquares(ls_in.A, ls_in.b)
    x = torch.zeros(d, dtype=torch.float32, device="cuda")
    for _ in range(10):
        ctx.core_gd_step(ls, h, x)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(20):
        ctx.core_gd_step(ls, h, x)
    torch.cuda.synchronize()
    per = max((time.perf_counter() - t0) / 20, 1e-6)
    steps = max(min_steps, min(20000, int(min_seconds / per)))
    sampler = ClockSampler(local)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        ctx.core_gd_step(ls, h, x)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    # the machine gradients alone (the HBM-bound part: one pass over A plus the small reduce)
    Gbuf = torch.empty((n, d), dtype=torch.float32, device="cuda")
    e0.record()
    for _ in range(steps):
        ctx.core_ls_gradients(ls, x, Gbuf)
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    grad_ms = e0.elapsed_time(e1) / steps
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except OSError:
        pass
    a_bytes = ls_in.A.numel() * 4
    hbm_peak = peaks.get("hbm_gbs", 6650.0)
    achieved = a_bytes / (grad_ms * 1e-3) / 1e9
    return {
        "workload": f"leastsq: n={n}, A_i {rows}x{d} fp32 (|A| = {a_bytes} bytes, larger than L2), m={m}, step 1/L",
        "steps": steps, "ms": ms, "loss": float(ctx.core_ls_loss(ls, x).item()),
        "gpu_launches": 4 * steps,   # gradient partials, project (sums them while staging), finish+aggregate, reconstruct+update
        "gradients_ms": grad_ms, "round_and_update_ms": ms - grad_ms, "bound": "hbm", "frac": achieved / hbm_peak,
        "roofline": {"bound": "hbm", "kernel": "ls_fused_kernel + ls_reduce_kernel", "achieved": achieved,
                     "peak": hbm_peak, "unit": "GB/s", "frac": achieved / hbm_peak, "traffic": None,
                     "algorithmic_bytes": a_bytes, "ms_per_launch": grad_ms,
                     "peak_source": "of measured" if "hbm_gbs" in peaks else "of fallback",
                     "note": "A is read once: residual and A^T r of a row come from the same registers"},
        "clocks": clocks}


def run_leastsq(args):
    """Secondary line: the least-squares CORE-GD step alone.  Not the headline metric."""
    import torch

    import paper_2309_13307_b200 as core_mod

    torch.cuda.set_device(0)
    core_mod.lib()
    r = measure_leastsq(core_mod, 0, min_steps=max(args.steps, 50))
    print(json.dumps({"metric": "least-squares CORE-GD step", "value": r["ms"], "unit": "ms/step",
                      "higher_is_better": False, "n_gpus": 1, "dtype": "f32", "data": "synthetic",
                      "config": {"workload": r["workload"]}, **{k: v for k, v in r.items() if k not in ("workload", "ms")}}))


def rank_environment(rank: int, world: int, port: int) -> dict:
    """Environment of one replica's process when this script starts the ranks itself."""
    return dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), NCCL_DEBUG=os.environ.get("NCCL_DEBUG", "WARN"))


def spawn_replicas(argv, world: int, entry=None) -> int:
    """`--gpus N` without a launcher: start N ranks of this script (one per device) and wait for them.
    Rank 0's standard output (the JSON line) passes through; the others' is dropped.  Returns the worst
    exit code."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    entry = entry or [sys.executable, os.path.abspath(__file__)]
    procs = []
    for rank in range(world):
        procs.append(subprocess.Popen(entry + list(argv), env=rank_environment(rank, world, port),
                                      stdout=None if rank == 0 else subprocess.DEVNULL))
    worst = 0
    for proc in procs:
        worst = max(worst, abs(proc.wait()))
    return worst


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.workload == "leastsq":
        run_leastsq(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_replicas(sys.argv[1:], args.gpus))
    else:
        world = int(os.environ.get("WORLD_SIZE", "1"))
        if world != args.gpus:
            sys.exit(f"bench.py: --gpus {args.gpus} but the launcher started {world} rank(s); refusing to report "
                     f"a line whose n_gpus would differ from --gpus")
        run_ours(args)


if __name__ == "__main__":
    main()
