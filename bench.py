#!/usr/bin/env python
"""Benchmark of the RoutePack planner hot path on B200.

A "step" is one complete plan of one synthetic optimizer-step window: input checks and
aggregate demand, LPT placement, demand projection, row count + seed, population annealing
over all temperature levels, validation and return of the best layout.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload heavy] [--impl reference]

Prints ONE JSON line.  `value` = replica-moves evaluated per second over the whole timed
region (all stages, inputs resident in HBM); `e2e` = the same with host buffers in and out
through the C ABI; `roofline` = the per-level chain kernel against the measured HBM peak;
`cpu_baseline` = the C oracle on this machine's host cores.  The headline workload is the largest
window (heavy); `other_workloads` carries the same record for the other four windows.  With
N > 1 every rank plans its own copy of the window (replicas only, no collective on the data path).
"""
from __future__ import annotations

import argparse
import glob
import json
import math
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

from paper_2608_12146_b200.windows import SPECS, make_window

METRIC = "annealing replica-moves evaluated/sec"
UNIT = "moves/s"
FALLBACK_HBM_GBS = 6650.0
# Bounded oracle samples (population, levels): the oracle scores every member of the initial
# population from scratch and holds two rank-load tensors per member, so a sample keeps the window
# and the steps per level and bounds the members and the levels.
CPU_SAMPLE = {"tiny": (8, 20), "medium": (256, 20), "large": (1024, 4), "wide": (512, 2), "heavy": (2048, 2)}
REF_SAMPLE = {"tiny": (8, 20), "medium": (256, 20), "large": (1024, 1), "wide": (128, 1), "heavy": (256, 1)}


def hbm_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def profiled_traffic(kernel, workload):
    """DRAM / L2 bytes per launch from the ncu summaries under profiles/: a summary that wants to be
    used here carries one line `bench_traffic: {json}` naming its kernel, workload and population."""
    for path in sorted(glob.glob(os.path.join(ROOT, "profiles", "*.txt"))):
        try:
            for line in open(path):
                if not line.startswith("bench_traffic:"):
                    continue
                rec = json.loads(line[len("bench_traffic:"):])
                if rec.get("kernel") == kernel and rec.get("workload") == workload:
                    rec["file"] = os.path.relpath(path, ROOT)
                    return rec
        except Exception:
            continue
    return None


def workload_config(spec, extra=None):
    cfg = {"workload": spec.name, "n_samples": spec.n_samples, "n_layers": spec.n_layers,
           "n_experts": spec.n_experts, "top_k": spec.top_k, "token_cap": spec.token_cap,
           "dp_shards": spec.dp_width, "ep_ranks": spec.ep_width, "population": spec.pop_size,
           "sweeps": spec.sweeps, "n_levels": spec.n_levels, "steps_per_level": spec.steps_per_level,
           "l2": "flushed between steps (256 MiB written, then read back so that no dirty lines are left to evict)"}
    if extra:
        cfg.update(extra)
    return cfg


# ---------------------------------------------------------------------------------------------
# the oracle on the host cores (reference arm and cpu_baseline)
# ---------------------------------------------------------------------------------------------
def oracle_sample(w, threads, pop, levels):
    """The oracle on a bounded sample of the workload: the whole front end once, then annealing
    of `pop` members for `levels` whole temperature levels of the window's own step count."""
    import oracle
    s = w.spec
    pop, levels = min(pop, s.pop_size), min(levels, s.n_levels)
    t0 = time.perf_counter()
    res = oracle.plan(w, pop_size=pop, n_levels=levels, n_threads=threads, trace=False)
    dt = time.perf_counter() - t0
    moves = int(res["counters"][0])
    sample = (f"whole front end + {levels} of {s.n_levels} temperature levels x {s.steps_per_level} steps for "
              f"{pop} of {s.pop_size} members ({moves} replica-moves)")
    return moves, dt, sample


def cpu_baseline(w, seconds):
    import oracle
    oracle.build()
    threads = os.cpu_count() or 1
    pop, levels = CPU_SAMPLE[w.spec.name]
    m, d, reps = 0, 0.0, 0
    while reps == 0 or (d < seconds and reps < 4096):
        mi, di, sample = oracle_sample(w, threads, pop, levels)
        m, d, reps = m + mi, d + di, reps + 1
    return {"value": m / d, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"{reps} x ({sample})", "seconds": d}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import oracle
    oracle.build()
    spec = SPECS[args.workload]
    w = make_window(spec)
    threads = os.cpu_count() or 1
    pop, levels = REF_SAMPLE[spec.name]
    for _ in range(min(args.warmup, 2)):
        oracle_sample(w, threads, pop, levels)
    moves, dt, sample = 0, 0.0, ""
    for _ in range(args.steps):
        m, d, sample = oracle_sample(w, threads, pop, levels)
        moves += m
        dt += d
    value = moves / dt
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64",
            "data": "synthetic", "config": workload_config(spec, {"parallelism": "1 gpu" if args.gpus == 1 else "replicas only"}),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                             "sample": f"each step: {sample}"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


# ---------------------------------------------------------------------------------------------
# CUDA arm
# ---------------------------------------------------------------------------------------------
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index):
        self.idx = device_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "20", "-i", str(self.idx)],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, power, reasons = [], [], [], set()
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
                power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm), "power_w_max": max(power) if power else None}


def reduce_job(ms_local, moves_local, dist=None, device="cpu"):
    """Whole-job figures from one rank's: the slowest rank's time and the moves of all ranks.

    With a process group (N > 1, replicas only) the time is the MAX over ranks and the moves
    the SUM; without one the local values stand."""
    if dist is None:
        return float(ms_local), int(moves_local)
    import torch
    tmax = torch.tensor([float(ms_local)], dtype=torch.float64, device=device)
    tsum = torch.tensor([float(moves_local)], dtype=torch.float64, device=device)
    dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
    dist.all_reduce(tsum, op=dist.ReduceOp.SUM)
    return float(tmax.item()), int(round(tsum.item()))


def plan_once(rp, w, t_in, a_in, outs, stream, stages=None, knobs=None):
    """One pass of the whole hot path through the C ABI; returns the annealing stats."""
    s = w.spec
    ctx = rp.rp_window_load(t_in, a_in, top_k=s.top_k, token_cap=s.token_cap, dp_width=s.dp_width,
                            ep_width=s.ep_width, pop_size=s.pop_size, alpha=s.alpha, beta=s.beta,
                            seed=s.anneal_seed, stream=stream)
    for k, v in (knobs or {}).items():
        rp.rp_debug_set_knob(ctx, k, v)
    rp.rp_place_experts(ctx, outs["pi"], outs["rank_load"])
    rp.rp_pack_rows(ctx)
    if stages is not None:
        stages["chain_kernel"] = rp.rp_debug_chain_kernel(ctx)
    stats = rp.rp_anneal(ctx, n_levels=s.n_levels, steps_per_level=s.steps_per_level, t0=s.t0,
                         t_ratio=s.t_ratio, p_reloc=s.p_reloc, p_guide=s.p_guide, want_stats=True)
    rp.rp_best(ctx, outs["layout"], outs["score_fx"], outs["score_f64"])
    if stages is not None:
        for k, v in rp.rp_debug_stage_times(ctx).items():
            if v is not None:
                stages[k] = stages.get(k, 0.0) + v
    rp.rp_destroy(ctx)
    return stats


def measure(rp, torch, args, name, steps, min_seconds, dist, dev, local, cpu_seconds):
    """Time plans of the named workload on this rank (exactly `steps` of them, or as many more as
    `min_seconds` of timed region needs); returns the pieces of the JSON line."""
    spec = SPECS[name]
    overrides = {}
    if args.pop:
        overrides["pop_size"] = args.pop          # profiling aid: a smaller population of the same window
    if args.levels:
        overrides["n_levels"] = args.levels
        overrides["sweeps"] = spec.steps_per_level * args.levels
    w = make_window(spec, **overrides)
    s = spec = w.spec
    moves_per_step = s.pop_size * s.n_levels * s.steps_per_level
    stream = torch.cuda.current_stream()
    t_dev = torch.from_numpy(w.lengths).to(dev)
    a_dev = torch.from_numpy(w.demand).to(dev)
    t_pin = torch.from_numpy(w.lengths).pin_memory()
    a_pin = torch.from_numpy(w.demand).pin_memory()

    def outputs(**kw):
        return dict(pi=torch.empty((s.n_layers, s.n_experts), dtype=torch.int32, **kw),
                    rank_load=torch.empty((s.n_layers, s.ep_width), dtype=torch.int64, **kw),
                    layout=torch.empty(s.n_samples, dtype=torch.int32, **kw),
                    score_fx=torch.empty(3, dtype=torch.int64, **kw),
                    score_f64=torch.empty(3, dtype=torch.float64, **kw))

    outs_dev = outputs(device=dev)
    outs_host = {k: v.pin_memory() for k, v in outputs().items()}
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    flush_sink = torch.empty(1, dtype=torch.uint8, device=dev)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed_loop(t_in, a_in, outs, n, stages=None):
        """n plans, each timed with CUDA events on the launching stream; L2 flushed in between."""
        acc = dict(ms=0.0, chain_ms=0.0, move_bytes=0, gather_bytes=0, staging_bytes=0, feasible=0, accepted=0,
                   chain_launches=0)
        barrier()
        wall0 = time.perf_counter()
        for _ in range(n):
            flush.fill_(1)
            flush_sink.copy_(flush[:1] + flush.max())       # read pass: the cache is left with clean lines only
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            st = plan_once(rp, w, t_in, a_in, outs, stream, stages)
            e1.record(stream)
            e1.synchronize()
            acc["ms"] += e0.elapsed_time(e1)
            acc["chain_ms"] += st.ms_chains
            acc["move_bytes"] += st.move_bytes
            acc["gather_bytes"] += st.gather_bytes
            acc["staging_bytes"] += st.staging_bytes
            acc["feasible"] += st.feasible
            acc["accepted"] += st.accepted
            acc["chain_launches"] += 1 if st.kernel_launches == 1 else s.n_levels
        barrier()
        acc["wall"] = time.perf_counter() - wall0
        return acc

    warm_ms = []
    for _ in range(args.warmup):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        plan_once(rp, w, t_dev, a_dev, outs_dev, stream)
        e1.record(stream)
        e1.synchronize()
        warm_ms.append(e0.elapsed_time(e1))
        plan_once(rp, w, t_pin, a_pin, outs_host, stream)
    if min_seconds:
        steps = max(steps, int(math.ceil(min_seconds * 1e3 / max(min(warm_ms), 1e-3))))
    vis = [x for x in os.environ.get("CUDA_VISIBLE_DEVICES", "").split(",") if x]
    sampler = ClockSampler(vis[local] if local < len(vis) else local)
    sampler.start()
    launches0 = rp.rp_debug_launch_count()
    res = timed_loop(t_dev, a_dev, outs_dev, steps)
    launches = rp.rp_debug_launch_count() - launches0
    clocks = sampler.stop()
    e2e = timed_loop(t_pin, a_pin, outs_host, steps)
    # stage times of the front end: a few more plans with events around its kernels (outside the timed regions)
    stages = {}
    n_st = max(1, min(steps, 5))
    rp.rp_debug_set_stage_timing(True)
    timed_loop(t_dev, a_dev, outs_dev, n_st, stages)
    rp.rp_debug_set_stage_timing(False)
    chain_kernel = stages.pop("chain_kernel")
    stages = {k: v / n_st for k, v in stages.items()}

    ms, total_moves = reduce_job(res["ms"], moves_per_step * steps, dist, dev)
    ms_e2e, _ = reduce_job(e2e["ms"], moves_per_step * steps, dist, dev)
    world = 1 if dist is None else dist.get_world_size()
    peak, peak_kind = hbm_peak()
    nl = res["chain_launches"]
    per_launch_s = res["chain_ms"] * 1e-3 / nl
    alg = (res["move_bytes"] + res["gather_bytes"]) / nl
    achieved = alg / per_launch_s / 1e9
    roofline = {"bound": "hbm", "kernel": chain_kernel, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_source": peak_kind, "served_by": "L2+HBM (algorithmic bytes; see dram)",
                "traffic": None, "algorithmic_bytes_per_launch": alg,
                "move_bytes_per_launch": res["move_bytes"] / nl, "gather_bytes_per_launch": res["gather_bytes"] / nl,
                "staging_bytes_per_launch": res["staging_bytes"] / nl,
                "launch_ms": per_launch_s * 1e3, "launches_per_step": nl / steps,
                "levels_per_launch": s.n_levels * steps / nl, "share_of_step": res["chain_ms"] / res["ms"]}
    prof = profiled_traffic(chain_kernel, s.name)
    if prof:
        scale = s.pop_size / float(prof["population"])
        dram = prof["dram_bytes_per_launch"] * scale
        roofline["traffic"] = dram
        roofline["dram"] = {"source": prof["file"], "captured_population": prof["population"],
                            "scaled_by_population": scale, "bytes_per_launch": dram,
                            "hbm_frac": dram / per_launch_s / 1e9 / peak,
                            "l2_bytes_per_launch": prof.get("lts_bytes_per_launch", 0) * scale or None,
                            "captured_dram_gbs": prof.get("dram_gbs"), "captured_l2_gbs": prof.get("lts_gbs")}
    n_le = s.n_samples * s.n_layers * s.n_experts * 4
    n_lp = s.n_samples * s.n_layers * s.ep_width * 4
    front = {}
    for key, byts in (("check_reduce", n_le), ("projection", n_le + n_lp)):
        if stages.get(key):
            gbs = byts / stages[key] / 1e6
            front[key] = {"ms": stages[key], "algorithmic_bytes": byts, "gbs": gbs, "frac_of_hbm_peak": gbs / peak}
    cpu = None
    if cpu_seconds:
        cpu = cpu_baseline(w, cpu_seconds)
    h2d = int(w.lengths.nbytes + w.demand.nbytes)
    d2h = int(sum(v.numel() * v.element_size() for v in outs_host.values()))
    n_all = moves_per_step * steps
    stage_ms = {"anneal_levels": res["chain_ms"] / steps, "other": (res["ms"] - res["chain_ms"]) / steps}
    stage_ms.update(stages)
    return {"value": total_moves / (ms * 1e-3), "ms_per_step": ms / steps, "steps": steps,
            "config": workload_config(spec, {"parallelism": "replicas only" if world > 1 else "1 gpu"}),
            "plans_per_s": steps * world / (ms * 1e-3),
            "anneal_only_moves_per_s": n_all / (res["chain_ms"] * 1e-3),
            "feasible_fraction": res["feasible"] / n_all, "accepted_fraction": res["accepted"] / n_all,
            "stage_ms_per_step": stage_ms, "front_end": front,
            "roofline": roofline, "cpu_baseline": cpu,
            "e2e": {"value": total_moves / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / steps},
            "gpu_launches": int(launches), "clocks": clocks, "timed_region_s": res["wall"]}


def concurrent_plans(rp, torch, name, dev, n_ctx, reps, per_level=1):
    """Context figure: plans per second with `n_ctx` windows planned at once on separate streams and
    contexts (the ABI allows it), with one launch per level (which lets the windows share the SMs) or
    the default single launch; reported beside the single-plan latency, never instead of it."""
    import threading
    w = make_window(SPECS[name])
    s = w.spec
    t_dev = torch.from_numpy(w.lengths).to(dev)
    a_dev = torch.from_numpy(w.demand).to(dev)
    streams = [torch.cuda.Stream(device=dev) for _ in range(n_ctx)]

    def worker(k, n):
        torch.cuda.set_device(dev)
        outs = dict(pi=torch.empty((s.n_layers, s.n_experts), dtype=torch.int32, device=dev),
                    rank_load=torch.empty((s.n_layers, s.ep_width), dtype=torch.int64, device=dev),
                    layout=torch.empty(s.n_samples, dtype=torch.int32, device=dev),
                    score_fx=torch.empty(3, dtype=torch.int64, device=dev),
                    score_f64=torch.empty(3, dtype=torch.float64, device=dev))
        for _ in range(n):
            plan_once(rp, w, t_dev, a_dev, outs, streams[k], knobs={"LAUNCH_PER_LEVEL": per_level})

    for n in (2, reps):                      # warm up, then time
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        th = [threading.Thread(target=worker, args=(k, n)) for k in range(n_ctx)]
        for x in th:
            x.start()
        for x in th:
            x.join()
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
    return {"workload": name, "concurrent_contexts": n_ctx, "launch_per_level": per_level, "plans": n_ctx * reps,
            "plans_per_s": n_ctx * reps / dt,
            "timing": "wall clock around host threads, one stream and context each"}


def one_launch_latency(rp, torch, name, dev, reps=200):
    """Context figure: latency of a single plan when rp_anneal runs all levels in one launch (the
    library does so by itself only up to 148 members, see RP_KNOB_LAUNCH_PER_LEVEL)."""
    w = make_window(SPECS[name])
    s = w.spec
    stream = torch.cuda.current_stream()
    t_dev = torch.from_numpy(w.lengths).to(dev)
    a_dev = torch.from_numpy(w.demand).to(dev)
    outs = dict(pi=torch.empty((s.n_layers, s.n_experts), dtype=torch.int32, device=dev),
                rank_load=torch.empty((s.n_layers, s.ep_width), dtype=torch.int64, device=dev),
                layout=torch.empty(s.n_samples, dtype=torch.int32, device=dev),
                score_fx=torch.empty(3, dtype=torch.int64, device=dev),
                score_f64=torch.empty(3, dtype=torch.float64, device=dev))
    out = {"workload": name, "plans": reps}
    for label, knob in (("launch_per_level", 1), ("one_launch", 2)):
        for _ in range(5):
            plan_once(rp, w, t_dev, a_dev, outs, stream, knobs={"LAUNCH_PER_LEVEL": knob})
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        chain = 0.0
        for _ in range(reps):
            chain += plan_once(rp, w, t_dev, a_dev, outs, stream, knobs={"LAUNCH_PER_LEVEL": knob}).ms_chains
        e1.record(stream)
        e1.synchronize()
        out[label] = {"ms_per_plan": e0.elapsed_time(e1) / reps, "anneal_ms_per_plan": chain / reps}
    return out


def seeding_stages(rp, torch, name, dev, reps=3, per_stage=True):
    """Context figure: device time of the optional seeding stages (trial loop, pairing, canonical
    map + quality-diversity selection) on the named window, mean over `reps` fresh contexts."""
    w = make_window(SPECS[name])
    s = w.spec
    t_dev = torch.from_numpy(w.lengths).to(dev)
    a_dev = torch.from_numpy(w.demand).to(dev)
    ms = {"seed_population": 0.0, "pair_population": 0.0, "select_population": 0.0}
    n_distinct = 0
    for _ in range(reps if per_stage else 0):      # (the selection grows with the square of the population: not on the big windows)
        ctx = rp.rp_window_load(t_dev, a_dev, top_k=s.top_k, token_cap=s.token_cap, dp_width=s.dp_width,
                                ep_width=s.ep_width, pop_size=s.pop_size, alpha=s.alpha, beta=s.beta, seed=s.anneal_seed)
        rp.rp_place_experts(ctx)
        rp.rp_pack_rows(ctx)
        for key, call in (("seed_population", lambda: rp.rp_seed_population(ctx, 4)),
                          ("pair_population", lambda: rp.rp_pair_population(ctx, 4)),
                          ("select_population", lambda: rp.rp_select_population(ctx, 8, 1 << 16))):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            out = call()
            e1.record()
            e1.synchronize()
            ms[key] += e0.elapsed_time(e1) / reps
            if key == "select_population":
                n_distinct = int(out[0])
        rp.rp_destroy(ctx)
    # Algorithm 2 as one call: M candidates (here as many as members), selected down to the population
    ctx = rp.rp_window_load(t_dev, a_dev, top_k=s.top_k, token_cap=s.token_cap, dp_width=s.dp_width,
                            ep_width=s.ep_width, pop_size=s.pop_size, alpha=s.alpha, beta=s.beta, seed=s.anneal_seed)
    rp.rp_place_experts(ctx)
    rp.rp_pack_rows(ctx)
    m_cand = min(s.pop_size, 256)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    nd_all, _ = rp.rp_init_population(ctx, m_cand, 4, 8, 1 << 16)
    e1.record()
    e1.synchronize()
    rp.rp_destroy(ctx)
    return {"workload": name, "ms": ms if per_stage else None, "n_distinct": n_distinct, "population": s.pop_size,
            "choice_width": 4, "n_proj": 8, "eta_q16": 1 << 16,
            "init_population": {"candidates": m_cand, "n_distinct": nd_all, "ms": e0.elapsed_time(e1)}}


def l2_read_rate(rp, mib=32, reps=50):
    """Read bandwidth of a buffer that stays in L2 (every thread of a full grid sums it with 16-byte
    loads): the denominator for kernels whose operands L2 serves."""
    return rp.rp_debug_l2_read_rate(mib << 20, reps)


def eval_stage(rp, torch, name, dev, l2_gbs, reps=10):
    """Context figure: full scoring of one population-sized batch of distinct layouts
    (rp_eval_population, device inputs and outputs).  The demand rows every layout gathers
    (N*L*P*4 bytes per layout) are shared by all layouts and served by L2, so they are set against a
    measured L2 read rate; what must cross HBM is the assignment (N*2 bytes per layout) plus the
    demand rows once, set against the measured HBM peak."""
    w = make_window(SPECS[name])
    s = w.spec
    t_dev = torch.from_numpy(w.lengths).to(dev)
    a_dev = torch.from_numpy(w.demand).to(dev)
    ctx = rp.rp_window_load(t_dev, a_dev, top_k=s.top_k, token_cap=s.token_cap, dp_width=s.dp_width,
                            ep_width=s.ep_width, pop_size=s.pop_size, alpha=s.alpha, beta=s.beta, seed=s.anneal_seed)
    rp.rp_place_experts(ctx)
    rp.rp_pack_rows(ctx)
    rp.rp_seed_population(ctx, 4)                  # distinct layouts, one per member
    lays = torch.from_numpy(rp.rp_debug_dump(ctx, "POPULATION", (s.pop_size, s.n_samples), np.int32)).to(dev)
    fx = torch.empty((s.pop_size, 3), dtype=torch.int64, device=dev)
    f64 = torch.empty((s.pop_size, 3), dtype=torch.float64, device=dev)
    for _ in range(3):
        rp.rp_eval_population(ctx, lays, fx, f64)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        rp.rp_eval_population(ctx, lays, fx, f64)
    e1.record()
    e1.synchronize()
    ms = e0.elapsed_time(e1) / reps
    rp.rp_destroy(ctx)
    peak, _ = hbm_peak()
    q_bytes = s.n_samples * s.n_layers * s.ep_width * 4
    gathered = s.pop_size * q_bytes
    hbm_min = s.pop_size * s.n_samples * 4 + q_bytes          # int32 layouts in, demand rows once
    return {"workload": name, "layouts": s.pop_size, "ms": ms, "layouts_per_s": s.pop_size / ms * 1e3,
            "roofline": {"bound": "l2", "kernel": "k_eval", "achieved": gathered / ms / 1e6, "peak": l2_gbs, "unit": "GB/s",
                         "frac": gathered / ms / 1e6 / l2_gbs, "peak_source": "read rate of a 32 MiB L2-resident buffer measured in this run (rp_debug_l2_read_rate)",
                         "gathered_bytes_per_launch": gathered, "hbm_bytes_per_launch_min": hbm_min,
                         "hbm_min_gbs": hbm_min / ms / 1e6, "hbm_min_frac": hbm_min / ms / 1e6 / peak}}


def mechanism_diagnostics(rp, torch, name, dev):
    """Context figure: the paper's mechanism diagnostics (global EP-rank CV before / after placement;
    EP peak sum, tail peak, EP balance efficiency, attention proxy and joint cost of the length-only
    seed against the annealed plan) on the named synthetic window."""
    w = make_window(SPECS[name])
    s = w.spec
    t_dev = torch.from_numpy(w.lengths).to(dev)
    a_dev = torch.from_numpy(w.demand).to(dev)
    ctx = rp.rp_window_load(t_dev, a_dev, top_k=s.top_k, token_cap=s.token_cap, dp_width=s.dp_width,
                            ep_width=s.ep_width, pop_size=s.pop_size, alpha=s.alpha, beta=s.beta, seed=s.anneal_seed)
    rp.rp_place_experts(ctx)
    rp.rp_pack_rows(ctx)
    seed = rp.rp_diagnostics(ctx)
    rp.rp_anneal(ctx, n_levels=s.n_levels, steps_per_level=s.steps_per_level, t0=s.t0, t_ratio=s.t_ratio,
                 p_reloc=s.p_reloc, p_guide=s.p_guide, want_stats=False)
    rp.rp_best(ctx)
    best = rp.rp_diagnostics(ctx)
    rp.rp_destroy(ctx)
    rel = lambda k: (best[k] - seed[k]) / seed[k] if seed[k] else 0.0
    return {"workload": name, "cv_identity": seed["cv_identity"], "cv_placed": seed["cv_placed"],
            "seed": {k: seed[k] for k in ("s_ep", "t_ep", "eta_ep", "attention", "joint")},
            "annealed": {k: best[k] for k in ("s_ep", "t_ep", "eta_ep", "attention", "joint")},
            "change": {"s_ep": rel("s_ep"), "t_ep": rel("t_ep"), "attention": rel("attention"), "joint": rel("joint")}}


def run_cuda(args):
    import torch
    import paper_2608_12146_b200.binding as rp

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path); use --impl reference for the oracle")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    rp.lib()
    dev = torch.device("cuda", local)

    if args.eval_only:          # profiling aid: only the population-sized scoring batch of the named window
        l2 = l2_read_rate(rp)
        print(json.dumps(eval_stage(rp, torch, args.workload, dev, l2, reps=max(1, args.steps))))
        return 0
    main_cpu = 0 if (world > 1 or rank != 0 or args.no_cpu_baseline) else 12.0
    main_res = measure(rp, torch, args, args.workload, args.steps, 0.0, dist, dev, local, main_cpu)
    rp.rp_release_cached_memory()
    sweep = {}
    extras = args.sweep and world == 1 and not args.pop and not args.levels
    if args.sweep and world == 1:
        for name in SPECS:            # the other windows: the same record, at least 1 s of timed region each
            if name == args.workload:
                continue
            sweep[name] = measure(rp, torch, args, name, 3, 1.0, None, dev, local, 0 if args.no_cpu_baseline else 4.0)
            rp.rp_release_cached_memory()
    if rank == 0:
        steps = main_res.pop("steps")
        line = {"metric": METRIC, "value": main_res.pop("value"), "unit": UNIT, "n_gpus": world, "steps": steps,
                "warmup": args.warmup, "ms_per_step": main_res.pop("ms_per_step"), "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "int64", "data": "synthetic"}
        line.update(main_res)
        if sweep:
            line["other_workloads"] = sweep
        if extras:
            l2 = l2_read_rate(rp)
            line["l2_read_gbs"] = l2
            # the chain kernels' L2 traffic (ncu capture) against the L2 read rate measured in this run
            for rec in [line] + list((line.get("other_workloads") or {}).values()):
                dram = rec["roofline"].get("dram")
                if dram and dram.get("l2_bytes_per_launch"):
                    dram["l2_gbs"] = dram["l2_bytes_per_launch"] / (rec["roofline"]["launch_ms"] * 1e-3) / 1e9
                    dram["l2_frac_of_measured_read_rate"] = dram["l2_gbs"] / l2
            line["eval_population"] = [eval_stage(rp, torch, n, dev, l2) for n in ("medium", "large", "wide")]
            line["concurrent_plans"] = [concurrent_plans(rp, torch, "medium", dev, n, 200, pl) for pl in (1, 0) for n in (1, 2, 4)]
            # large: one warp per chain and 7 warps per SM for a single window, so several windows fit the SMs at once
            line["concurrent_plans"] += [concurrent_plans(rp, torch, "large", dev, n, 60, 0) for n in (1, 2, 4)]
            line["single_plan_latency"] = [one_launch_latency(rp, torch, n, dev) for n in ("tiny", "medium")]
            line["seeding_stages"] = [seeding_stages(rp, torch, "medium", dev), seeding_stages(rp, torch, "heavy", dev, per_stage=False)]
            line["mechanism_diagnostics"] = [mechanism_diagnostics(rp, torch, n, dev) for n in ("medium", "large")]
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="heavy", choices=list(SPECS))
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", dest="sweep", action="store_false",
                    help="skip the records of the other four windows and the context figures (N=1 only)")
    ap.add_argument("--eval-only", action="store_true",
                    help="profiling aid: time only rp_eval_population on a population-sized batch of the workload")
    ap.add_argument("--pop", type=int, default=0, help="override the population size (profiling aid)")
    ap.add_argument("--levels", type=int, default=0, help="override the number of temperature levels (profiling aid)")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "cuda":
        args.warmup = 3
    if args.impl == "reference":
        return run_reference(args)
    return run_cuda(args)


if __name__ == "__main__":
    sys.exit(main())
