#!/usr/bin/env python
"""Benchmark of the GoodServe routing hot path on B200.

One step = one pass of the whole hot path over one batch of synthetic input:
gs_route_batch over N pending requests x M instances, then gs_risk_scan over A active
requests (instance prologue, pair scoring, selection, risk test, candidate compaction).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 3] [--impl reference]

Prints ONE JSON line (rank 0).  With N > 1 (launched by torch.distributed.run) every rank
runs the same-size workload on its own GPU with its own seed -- requests are independent, so
the path shards with no collective -- and the reported value is all ranks' units over the
slowest rank's device time ("weak" scaling).
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads as W  # noqa: E402

METRIC = "request-instance pairs scored/sec"
UNIT = "pairs/s"
ROUTE_BYTES_PER_REQUEST = 24      # 3 input columns + 3 output columns, 4 B each
RISK_BYTES_PER_REQUEST = 20.125   # 5 input columns + 1 flag bit (candidate indices added per flag)
KERNEL_NAMES = ("prologue", "route", "advance", "risk_flags", "risk_scatter", "reroute", "ema", "sequential")
ISSUE_PEAK_WARP_INST_PER_S = 148 * 4 * 1.965e9   # SMs x schedulers x 1 warp-instruction per clock

# Counters of one launch on config 3 taken with ncu (profiles/route_kernel_config3.md,
# profiles/risk_flags_kernel_config3.md).  They describe the kernel sources with these hashes;
# after any change to those files they no longer apply and the fields that use them become
# null until the kernel is profiled again.
PROFILED_ROUTE = {"sources_sha1": "bac3726b1cb32d3d74d0cdb6b491727579021779", "config": 3,
                  "dram_bytes_per_launch": 52_352_256 + 7_199_488,
                  "warp_instructions_per_launch": 24_600_939}
PROFILED_RISK_FLAGS = {"sources_sha1": "23376727e5a3e7bc33cc0aaa3cba258afd1240c6", "config": 3,
                       "dram_bytes_per_launch": 335_564_032 + 4_064_256}


def _sources_sha1(names) -> str:
    import hashlib
    h = hashlib.sha1()
    base = os.path.join(ROOT, "paper_2605_16867_b200", "csrc")
    for name in names:
        with open(os.path.join(base, name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def kernel_sources_sha1() -> str:
    return _sources_sha1(("gs_internal.cuh", "prologue.cu", "route.cu"))


def risk_sources_sha1() -> str:
    return _sources_sha1(("gs_internal.cuh", "risk.cu"))


# --------------------------------------------------------------------------------------
# helpers that do not need a GPU (covered by the CPU tests)
# --------------------------------------------------------------------------------------

def rank_seed(cfg_id: int, rank: int) -> int:
    """Every rank draws its own batch: same shape, different seed."""
    return cfg_id + 1000 * rank


def aggregate_over_ranks(local_ms: float, local_units: float, dist=None):
    """(max time over ranks, sum of units over ranks).  `dist` is torch.distributed or None."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return local_ms, local_units
    import torch
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([local_ms], dtype=torch.float64, device=dev)
    u = torch.tensor([local_units], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        if self.thread is not None:
            self.thread.join(timeout=5)
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for r in self.rows:
            if len(r) < 6:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            for name, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons),
                "samples": len(sm)}


# --------------------------------------------------------------------------------------
# reference arm: the CPU oracle, as it stands, on a bounded sample
# --------------------------------------------------------------------------------------

def oracle_step(wl, n_req: int, n_act: int, threads: int):
    """One pass of the oracle over the first n_req requests and n_act active requests."""
    import oracle
    t0 = time.perf_counter()
    tab = oracle.instance_table(wl.types, wl.instances, wl.ema_alpha, "f64")
    r, a = wl.requests, wl.active
    oracle.route(tab, r.prompt_len[:n_req], r.pred_decode_len[:n_req], r.slo_ms[:n_req], threads=threads)
    t1 = time.perf_counter()
    res = oracle.risk(tab, *(c[:n_act] for c in a.columns()), threads=threads)
    oracle.compact(res.flag)
    t2 = time.perf_counter()
    return t1 - t0, t2 - t1


def cpu_baseline(wl, seconds_target: float = 12.0):
    threads = len(os.sched_getaffinity(0))
    M = wl.instances.n_instances
    n_req = min(wl.requests.n, 1 << 18)
    n_act = min(wl.active.n, 1 << 22)
    t_route, t_risk = oracle_step(wl, n_req, n_act, threads)           # also warms the library
    # grow the route sample towards the time target (bounded by the workload)
    scale = max(1.0, min(seconds_target / max(t_route, 1e-3) * 0.5, wl.requests.n / n_req))
    n_req = int(n_req * scale)
    t_route, t_risk = oracle_step(wl, n_req, n_act, threads)
    return {"value": n_req * M / (t_route + t_risk), "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"fp64 oracle, first {n_req} of {wl.requests.n} requests x {M} instances "
                      f"({t_route:.2f} s) + risk scan of first {n_act} of {wl.active.n} active requests "
                      f"({t_risk:.2f} s), {threads} threads over contiguous request ranges",
            "route_pairs_per_s": n_req * M / t_route, "risk_scan_requests_per_s": n_act / t_risk}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = W.CONFIGS[args.config]
    wl = W.make_workload(args.config, n_requests=min(cfg.n_requests, 1 << 20),
                         n_active=min(cfg.n_active, 1 << 22))
    threads = len(os.sched_getaffinity(0))
    M = wl.instances.n_instances
    n_req, n_act = min(wl.requests.n, 1 << 19), wl.active.n
    for _ in range(args.warmup):
        oracle_step(wl, n_req // 8, n_act // 8, threads)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(wl, n_req, n_act, threads)
    dt = time.perf_counter() - t0
    value = args.steps * n_req * M / dt
    sample = (f"each step: fp64 oracle over {n_req} requests x {M} instances + risk scan over {n_act} "
              f"active requests (bounded sample of config {args.config}), {threads} threads")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": workload_name(args.config), "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def workload_name(cfg_id: int) -> str:
    c = W.CONFIGS[cfg_id]
    return (f"config {cfg_id}: {c.n_requests} pending requests x {c.n_instances} instances of "
            f"{c.n_types} GPU types, SLO U[{c.slo_lo},{c.slo_hi}] x ideal; risk scan over {c.n_active} active requests")


# --------------------------------------------------------------------------------------
# GPU arm
# --------------------------------------------------------------------------------------

def run_gpu(args):
    import torch
    from paper_2605_16867_b200 import GoodServe, InstancePool

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)

    cfg = W.CONFIGS[args.config]
    wl = W.make_workload(args.config, seed=rank_seed(args.config, rank))
    N, M, A = wl.requests.n, wl.instances.n_instances, wl.active.n
    alpha = wl.ema_alpha

    gs = GoodServe(local_rank)
    pool = InstancePool.from_host(wl.types, wl.instances, dev)
    req = [torch.from_numpy(c).to(dev) for c in wl.requests.columns()]
    act = [torch.from_numpy(c).to(dev) for c in wl.active.columns()]
    out_idx = torch.empty(N, dtype=torch.int32, device=dev)
    out_est = torch.empty(N, dtype=torch.float32, device=dev)
    out_slack = torch.empty(N, dtype=torch.float32, device=dev)
    flag_bits = torch.empty((A + 31) // 32, dtype=torch.int32, device=dev)
    cand = torch.empty(A, dtype=torch.int32, device=dev)
    count = torch.zeros(1, dtype=torch.int64, device=dev)
    stream = torch.cuda.current_stream(dev)

    # The two halves of a step are independent (the scan reads the same instance snapshot and
    # uses separate scratch), so the scan runs on a second stream beside the routing round: one
    # is bound by instruction issue, the other by HBM.  --serial puts both on one stream.
    side = None if args.serial else torch.cuda.Stream(dev)
    fork, join = torch.cuda.Event(), torch.cuda.Event()

    def step(overlap=True):
        if side is None or not overlap:
            gs.route_batch(*req, pool, alpha, out_idx, out_est, out_slack, None, stream=stream)
            gs.risk_scan(*act, pool, flag_bits, cand, count, stream=stream)
            return
        fork.record(stream)
        side.wait_event(fork)
        gs.risk_scan(*act, pool, flag_bits, cand, count, stream=side)
        gs.route_batch(*req, pool, alpha, out_idx, out_est, out_slack, None, stream=stream)
        join.record(side)
        stream.wait_event(join)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    # clocks are sampled from before the warm-up until a few samples under load exist: the
    # timed region itself lasts only milliseconds, less than one nvidia-smi sampling period
    sampler = ClockSampler(local_rank)
    sampler.start()
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()

    # ---- device-resident timed region: exactly K steps ------------------------------
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = gs.launch_count()
    barrier()
    ev0.record(stream)
    for _ in range(args.steps):
        step()
    ev1.record(stream)
    barrier()
    local_ms = ev0.elapsed_time(ev1)
    launches = gs.launch_count() - launches0

    # ---- per-kernel durations: K more steps, one stream, every launch bracketed by events ----
    # (kernels that share the GPU with another stream's kernel have no duration of their own,
    # so the roofline figures come from this serial pass over the same inputs)
    gs.timing_enable(True)
    barrier()
    ev0.record(stream)
    for _ in range(args.steps):
        step(overlap=False)
    ev1.record(stream)
    barrier()
    serial_ms_per_step = ev0.elapsed_time(ev1) / args.steps
    kernel_ms = {}
    for k, name in enumerate(KERNEL_NAMES):
        ms, n = gs.timing_read(k)
        if n:
            kernel_ms[name] = (ms, n)
    gs.timing_enable(False)

    # ---- the step after the scan (not part of the timed step): re-route its candidates ----
    reroute = None
    if not args.no_reroute:
        a_prompt = torch.from_numpy(W.make_requests(cfg, wl.types, seed=rank_seed(args.config, rank) + 7,
                                                    n=A).prompt_len).to(dev)
        r_inst = torch.empty(A, dtype=torch.int32, device=dev)
        r_est = torch.empty(A, dtype=torch.float32, device=dev)
        r_slack = torch.empty(A, dtype=torch.float32, device=dev)
        gs.reroute_candidates(cand, count, *act, a_prompt, pool, alpha, r_inst, r_est, r_slack, stream=stream)
        barrier()
        gs.timing_enable(True)
        for _ in range(max(3, args.steps // 2)):
            gs.reroute_candidates(cand, count, *act, a_prompt, pool, alpha, r_inst, r_est, r_slack, stream=stream)
        barrier()
        ms, n_l = gs.timing_read(KERNEL_NAMES.index("reroute"))
        gs.timing_enable(False)
        n_cand = int(count.item())
        reroute = {"candidates": n_cand, "avg_us": ms / n_l * 1e3,
                   "candidates_per_s": n_cand / (ms / n_l * 1e-3),
                   "algorithmic_GBps": n_cand * (4 + 24 + 12) / (ms / n_l * 1e-3) / 1e9}
        del a_prompt, r_inst, r_est, r_slack
    # ---- the routing round with Eq. 2's prefix-cache term (not part of the timed step) ----
    prefix = None
    if not args.no_prefix:
        stride = (N + 3) // 4 * 4
        pi, ph = W.make_prefix_hits(wl.requests, M, seed=rank_seed(args.config, rank), n_slots=1)
        pi_d = torch.full((stride,), -1, dtype=torch.int32, device=dev)
        ph_d = torch.zeros(stride, dtype=torch.int32, device=dev)
        pi_d[:N] = torch.from_numpy(pi[0]).to(dev)
        ph_d[:N] = torch.from_numpy(ph[0]).to(dev)
        run = lambda: gs.route_batch_prefix(*req, pi_d, ph_d, 1, stride, pool, alpha, out_idx, out_est,
                                            out_slack, None, stream=stream)
        run()
        barrier()
        gs.timing_enable(True)
        for _ in range(max(3, args.steps // 2)):
            run()
        barrier()
        ms, n_l = gs.timing_read(KERNEL_NAMES.index("route"))
        gs.timing_enable(False)
        prefix = {"n_slots": 1, "hit_share": float((pi[0] >= 0).mean()), "avg_us": ms / n_l * 1e3,
                  "algorithmic_GBps": N * (ROUTE_BYTES_PER_REQUEST + 8) / (ms / n_l * 1e-3) / 1e9}
        del pi_d, ph_d
        gs.route_batch(*req, pool, alpha, out_idx, out_est, out_slack, None, stream=stream)   # outputs of the timed step
    # ---- the routing round against black-box coefficients given per instance (not timed) ----
    direct = None
    if not args.no_direct:
        bb = W.make_blackbox_table(wl.types, wl.instances, seed=rank_seed(args.config, rank))
        tab = [torch.from_numpy(c).to(dev) for c in bb.columns()]
        obs = [torch.from_numpy(W.make_observations(c, seed=rank_seed(args.config, rank), step=k)).to(dev)
               for k, c in enumerate(bb.columns()[:3])]
        run = lambda: (gs.ema_update(alpha, *obs, *tab[:3], stream=stream),
                       gs.route_batch_direct(*req, *tab, out_idx, out_est, out_slack, None, stream=stream))
        run()
        barrier()
        gs.timing_enable(True)
        for _ in range(max(3, args.steps // 2)):
            run()
        barrier()
        t = {name: gs.timing_read(KERNEL_NAMES.index(name)) for name in ("ema", "prologue", "route")}
        gs.timing_enable(False)
        direct = {name + "_avg_us": ms / n_l * 1e3 for name, (ms, n_l) in t.items()}
        direct["groups"] = 8
        del tab, obs
        gs.route_batch(*req, pool, alpha, out_idx, out_est, out_slack, None, stream=stream)   # outputs of the timed step
    # ---- Algorithm 1 one request at a time: a single dependent chain (not timed) ----
    sequential = None
    if not args.no_sequential:
        n_seq = min(N, 262144)
        seq_pool = InstancePool.from_host(wl.types, wl.instances, dev)      # advanced in place
        gs.timing_enable(True)
        gs.route_sequential(*req, seq_pool, alpha, out_idx, out_est, out_slack, None, n_requests=n_seq, stream=stream)
        barrier()
        ms, n_l = gs.timing_read(KERNEL_NAMES.index("sequential"))
        gs.timing_enable(False)
        sequential = {"requests": n_seq, "ms": ms / n_l, "requests_per_s": n_seq / (ms / n_l * 1e-3),
                      "ns_per_request": ms / n_l * 1e6 / n_seq}
        del seq_pool
        gs.route_batch(*req, pool, alpha, out_idx, out_est, out_slack, None, stream=stream)   # outputs of the timed step
    t_wait = time.perf_counter()
    while len(sampler.rows) < 4 and time.perf_counter() - t_wait < 3.0:
        step()                                   # keep the same load up for the sampler (untimed)
        torch.cuda.synchronize(dev)
    clocks = sampler.stop()
    flagged = int(count.item())
    status = gs.device_status()

    total_ms, total_pairs = aggregate_over_ranks(local_ms, float(args.steps) * N * M, dist)
    value = total_pairs / (total_ms * 1e-3)
    ms_per_step = total_ms / args.steps

    # ---- end to end through the host-buffer C ABI ------------------------------------
    pin = lambda a: torch.from_numpy(a).pin_memory()            # noqa: E731
    h_req = [pin(c) for c in wl.requests.columns()]
    h_act = [pin(c) for c in wl.active.columns()]
    h_idx = torch.empty(N, dtype=torch.int32).pin_memory()
    h_est = torch.empty(N, dtype=torch.float32).pin_memory()
    h_slack = torch.empty(N, dtype=torch.float32).pin_memory()
    h_bits = torch.empty((A + 31) // 32, dtype=torch.int32).pin_memory()
    h_cand = torch.empty(A, dtype=torch.int32).pin_memory()

    def e2e_step():
        gs.route_batch_host(*h_req, wl.types, wl.instances, alpha, h_idx, h_est, h_slack, stream=stream)
        return gs.risk_scan_host(*h_act, wl.types, wl.instances, h_bits, h_cand, stream=stream)

    e2e_steps = max(1, min(args.steps, 5))
    n_flag = flagged
    if args.no_e2e:
        e2e_steps, e2e_ms = 0, float("nan")
    else:
        e2e_step()
        barrier()
        t0 = time.perf_counter()
        ev0.record(stream)
        for _ in range(e2e_steps):
            n_flag = e2e_step()
        ev1.record(stream)
        barrier()
        e2e_ms = max(ev0.elapsed_time(ev1), (time.perf_counter() - t0) * 1e3)
    e2e_ms, e2e_pairs = aggregate_over_ranks(e2e_ms, float(e2e_steps) * N * M, dist)
    h2d = 3 * 4 * N + 5 * 4 * A + 2 * (5 * 4 * M + 3 * 4 * wl.types.n_types)
    d2h = 3 * 4 * N + 4 * ((A + 31) // 32) + 8 + 4 * n_flag

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel ---------------------------------------------
    peak, peak_kind = load_peaks()
    per_kernel = {}
    for name, (ms, n) in kernel_ms.items():
        per_kernel[name] = {"launches": n, "avg_us": ms / n * 1e3}
    dominant = max(kernel_ms, key=lambda k: kernel_ms[k][0]) if kernel_ms else None
    alg_bytes = {"route": ROUTE_BYTES_PER_REQUEST * N + 20 * M,
                 "risk_flags": 20 * A + 4 * ((A + 31) // 32) + 4 * ((A + 1023) // 1024),
                 "risk_scatter": 4 * ((A + 31) // 32) + 4 * flagged + 4 * ((A + 1023) // 1024)}
    roofline = None
    issue = None
    profiled = (PROFILED_ROUTE if PROFILED_ROUTE["sources_sha1"] == kernel_sources_sha1()
                and PROFILED_ROUTE["config"] == args.config else None)
    profiled_risk = (PROFILED_RISK_FLAGS if PROFILED_RISK_FLAGS["sources_sha1"] == risk_sources_sha1()
                     and PROFILED_RISK_FLAGS["config"] == args.config else None)
    if dominant in alg_bytes:
        ms, n = kernel_ms[dominant]
        achieved = alg_bytes[dominant] / (ms / n * 1e-3) / 1e9
        roofline = {"bound": "hbm", "kernel": dominant, "achieved": achieved, "peak": peak, "unit": "GB/s",
                    "frac": achieved / peak,
                    "traffic": (profiled["dram_bytes_per_launch"] if profiled and dominant == "route" else
                                profiled_risk["dram_bytes_per_launch"] if profiled_risk and dominant == "risk_flags" else None),
                    "peak_kind": f"of {peak_kind}", "algorithmic_bytes_per_launch": alg_bytes[dominant]}
    if profiled and "route" in kernel_ms:
        ms, n = kernel_ms["route"]
        rate = profiled["warp_instructions_per_launch"] / (ms / n * 1e-3)
        issue = {"kernel": "route", "bound": "alu", "achieved": rate, "peak": ISSUE_PEAK_WARP_INST_PER_S,
                 "unit": "warp-instructions/s", "frac": rate / ISSUE_PEAK_WARP_INST_PER_S,
                 "warp_instructions_per_request": profiled["warp_instructions_per_launch"] / N,
                 "note": "instruction count from ncu; peak = 148 SMs x 4 schedulers x 1.965 GHz"}
    for name in per_kernel:
        if name in alg_bytes:
            gbs = alg_bytes[name] / (per_kernel[name]["avg_us"] * 1e-6) / 1e9
            per_kernel[name]["algorithmic_GBps"] = gbs
            per_kernel[name]["frac_of_hbm_peak"] = gbs / peak
    if profiled and "route" in per_kernel:
        per_kernel["route"]["dram_bytes_per_launch"] = profiled["dram_bytes_per_launch"]
    if profiled_risk and "risk_flags" in per_kernel:
        per_kernel["risk_flags"]["dram_bytes_per_launch"] = profiled_risk["dram_bytes_per_launch"]
    route_ms = sum(kernel_ms[k][0] for k in ("prologue", "route") if k in kernel_ms) / args.steps   # serial pass
    risk_ms = sum(kernel_ms[k][0] for k in ("risk_flags", "risk_scatter") if k in kernel_ms) / args.steps
    step_bytes = ROUTE_BYTES_PER_REQUEST * N + RISK_BYTES_PER_REQUEST * A + 4 * flagged

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_name(args.config), "ema_alpha": alpha,
                   "l2": "inputs larger than L2: one step streams %.0f MB" % (step_bytes / 1e6),
                   "streams": 1 if args.serial else 2,
                   "per_rank_seed": "config id + 1000 * rank", "sharding": "independent batches per rank, no collective"},
        "risk_scan_requests_per_s": world * A / (risk_ms * 1e-3) if risk_ms else None,
        "route_pairs_per_s": world * N * M / (route_ms * 1e-3) if route_ms else None,
        "route_requests_per_s": world * N / (route_ms * 1e-3) if route_ms else None,
        "step_hbm_frac": step_bytes / (ms_per_step * 1e-3) / 1e9 / peak,
        "flagged_fraction": flagged / A, "device_status": status,
        "roofline": roofline, "issue": issue, "kernels": per_kernel, "reroute": reroute, "prefix": prefix, "direct": direct, "sequential": sequential,
        "kernel_timing": "serial pass of %d steps on one stream after the timed region, %.4f ms/step" % (
            args.steps, serial_ms_per_step),
        "e2e": None if args.no_e2e else
               {"value": e2e_pairs / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / e2e_steps, "steps": e2e_steps},
        "gpu_launches": launches, "clocks": clocks,
    }
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(wl)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=3, choices=sorted(W.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=("ours", "reference"))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--no-reroute", action="store_true", help="skip the untimed re-route measurement")
    ap.add_argument("--no-direct", action="store_true", help="skip the untimed black-box-table routing measurement")
    ap.add_argument("--no-sequential", action="store_true", help="skip the untimed one-at-a-time routing measurement")
    ap.add_argument("--no-prefix", action="store_true", help="skip the untimed prefix-cache routing measurement")
    ap.add_argument("--serial", action="store_true", help="route and scan on one stream instead of two")
    ap.add_argument("--print-kernel-hash", action="store_true", help="print the hash PROFILED_ROUTE refers to")
    args = ap.parse_args()
    if args.print_kernel_hash:
        print(kernel_sources_sha1(), risk_sources_sha1())
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
