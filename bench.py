#!/usr/bin/env python
"""Benchmark of the GoodServe routing hot path on B200.

One step = one pass of the whole hot path over one batch of synthetic input:
gs_route_batch over N pending requests x M instances, then gs_risk_scan over A active
requests (instance prologue, pair scoring, selection, risk test, candidate compaction).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 3] [--impl reference]

Besides the step of the largest workload (the headline), rank 0 of a one-GPU run measures
every one of the five workload shapes (`per_config`): each entry point called back to back and
one call at a time, inputs rotated through several device copies so that L2 cannot serve them,
the 64-round stream of config 4 replayed from a CUDA graph, and the work the routing search
does per request (from the library's counting build).

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
SCHEDULERS_PER_SM = 4             # one warp-instruction per scheduler and clock

# Counters of one launch on config 3 taken with ncu (the committed ncu summaries).  They describe
# the kernel sources with these hashes; after any change to those files they no longer apply and
# the fields that use them become null until the kernel is profiled again.
PROFILED_ROUTE = {"sources_sha1": "310620025137156884c78c86c3f55770bea78be7", "config": 3,
                  "dram_bytes_per_launch": 52_239_104 + 7_389_440,
                  "warp_instructions_per_launch": 28_136_474}
PROFILED_RISK_FLAGS = {"sources_sha1": "924a286221ab49a6ca09c606b4dc3cc192a2ea7b", "config": 3,
                       "dram_bytes_per_launch": 335_574_272 + 4_547_840}


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
    # the same plain loop on one thread, on a sample sized for a few seconds
    n1 = max(1024, min(n_req, int(n_req / max(threads, 1) * 0.5)))
    a1 = max(1024, min(n_act, 1 << 20))
    t1_route, t1_risk = oracle_step(wl, n1, a1, 1)
    return {"value": n_req * M / (t_route + t_risk), "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"fp64 oracle, first {n_req} of {wl.requests.n} requests x {M} instances "
                      f"({t_route:.2f} s) + risk scan of first {n_act} of {wl.active.n} active requests "
                      f"({t_risk:.2f} s), {threads} threads over contiguous request ranges",
            "route_pairs_per_s": n_req * M / t_route, "risk_scan_requests_per_s": n_act / t_risk,
            "one_thread": {"route_pairs_per_s": n1 * M / t1_route, "risk_scan_requests_per_s": a1 / t1_risk,
                           "sample": f"first {n1} requests x {M} instances ({t1_route:.2f} s), first {a1} active "
                                     f"requests ({t1_risk:.2f} s)"}}


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
              f"active requests (bounded sample of config {args.config}: the full workload would take the "
              f"oracle seconds per step, so rates, not step times, are what compares), {threads} threads")
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
# timing of one entry point, and the five workload shapes
# --------------------------------------------------------------------------------------

def time_back_to_back(fn, stream, inner: int = 20, outer: int = 7) -> float:
    """Microseconds per call when `inner` calls are enqueued back to back (what a stream of
    rounds sees): one event pair around the batch, median over `outer` batches."""
    import torch
    fn(0)
    out = []
    k = 1
    for _ in range(outer):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(inner):
            fn(k)
            k += 1
        e1.record(stream)
        torch.cuda.synchronize()
        out.append(e0.elapsed_time(e1) / inner * 1e3)
    return statistics.median(out)


def time_isolated(fn, stream, reps: int = 25) -> float:
    """Microseconds of one call on an idle GPU: every call between its own pair of events
    (the pair itself costs a few microseconds), median over `reps` calls."""
    import torch
    fn(0)
    out = []
    for k in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        fn(k + 1)
        e1.record(stream)
        torch.cuda.synchronize()
        out.append(e0.elapsed_time(e1) * 1e3)
    return statistics.median(out)


def n_copies(bytes_per_copy: int) -> int:
    """Device copies of an input set to rotate through: at least four while the set is smaller
    than 256 MB (then L2 could serve a repeated one), enough to reach 512 MB, at most 16."""
    if bytes_per_copy >= 256e6:
        return 2
    return int(max(4, min(16, 512e6 // max(bytes_per_copy, 1) + 1)))


def measure_config(gs, cfg_id: int, seed: int, dev, peak_gbs: float, gs_count=None):
    """Every entry point of the hot path on one workload shape at full size."""
    import torch
    from paper_2605_16867_b200 import InstancePool
    wl = W.make_workload(cfg_id, seed=seed)
    N, M, A, Tn = wl.requests.n, wl.instances.n_instances, wl.active.n, wl.types.n_types
    alpha = wl.ema_alpha
    stream = torch.cuda.current_stream(dev)
    pool = InstancePool.from_host(wl.types, wl.instances, dev)
    res = {"n_requests": N, "n_instances": M, "n_types": Tn, "n_active": A}

    # ---- the routing round -------------------------------------------------------------
    nc = n_copies(24 * N)
    reqs = [[torch.from_numpy(c).to(dev) for c in wl.requests.columns()] for _ in range(nc)]
    outs = [(torch.empty(N, dtype=torch.int32, device=dev), torch.empty(N, dtype=torch.float32, device=dev),
             torch.empty(N, dtype=torch.float32, device=dev)) for _ in range(nc)]
    tier = torch.empty(N, dtype=torch.uint8, device=dev)
    route = lambda k: gs.route_batch(*reqs[k % nc], pool, alpha, *outs[k % nc], None, stream=stream)   # noqa: E731
    for k in range(3):
        route(k)
    t_b2b = time_back_to_back(route, stream)
    t_iso = time_isolated(route, stream)
    gs.timing_enable(True)
    for k in range(20):
        route(k)
    torch.cuda.synchronize(dev)
    t_pro, t_rt = gs.timing_read(KERNEL_NAMES.index("prologue")), gs.timing_read(KERNEL_NAMES.index("route"))
    gs.timing_enable(False)
    gs.route_batch(*reqs[0], pool, alpha, *outs[0], tier, stream=stream)
    torch.cuda.synchronize(dev)
    hist = torch.bincount(tier.to(torch.int64), minlength=4).cpu().tolist()
    by = ROUTE_BYTES_PER_REQUEST * N + 20 * M
    res["route"] = {
        "call_us": t_b2b, "call_us_isolated": t_iso, "input_copies_rotated": nc,
        "requests_per_s": N / (t_b2b * 1e-6), "logical_pairs_per_s": N * M / (t_b2b * 1e-6),
        "algorithmic_GBps": by / (t_b2b * 1e-6) / 1e9, "frac_of_hbm_peak": by / (t_b2b * 1e-6) / 1e9 / peak_gbs,
        "frac_of_hbm_peak_isolated": by / (t_iso * 1e-6) / 1e9 / peak_gbs,
        "kernel_us": {"prologue": t_pro[0] / t_pro[1] * 1e3, "route": t_rt[0] / t_rt[1] * 1e3},
        "tier_histogram": {"just_enough": hist[1], "fallback_kv_ok": hist[2], "fallback_any": hist[3]},
    }
    if gs_count is not None:
        # the search's work per request, from the counting build (same kernels, counters on)
        gs_count.eval_counters(clear=True)
        gs_count.route_batch(*reqs[0], pool, alpha, *outs[0], None, stream=stream)
        c = gs_count.eval_counters(clear=True)
        res["route"]["evaluated_per_request"] = {
            "pairs_scored_exactly": c[0] / N, "row_bounds_tested": c[1] / N, "type_bounds_tested": c[2] / N,
            "logical_pairs": M, "share_left_to_full_search": c[3] / N, "share_fallback": c[4] / N,
            "share_scored_by_a_whole_warp": c[5] / N}
    del reqs, outs, tier

    # ---- the risk scan -------------------------------------------------------------------
    nc = n_copies(20 * A)
    acts = [[torch.from_numpy(c).to(dev) for c in wl.active.columns()] for _ in range(nc)]
    bits = torch.empty((A + 31) // 32, dtype=torch.int32, device=dev)
    cand = torch.empty(A, dtype=torch.int32, device=dev)
    count = torch.zeros(1, dtype=torch.int64, device=dev)
    scan = lambda k: gs.risk_scan(*acts[k % nc], pool, bits, cand, count, stream=stream)   # noqa: E731
    for k in range(3):
        scan(k)
    t_b2b = time_back_to_back(scan, stream)
    t_iso = time_isolated(scan, stream)
    gs.timing_enable(True)
    for k in range(20):
        scan(k)
    torch.cuda.synchronize(dev)
    t_fl, t_sc = gs.timing_read(KERNEL_NAMES.index("risk_flags")), gs.timing_read(KERNEL_NAMES.index("risk_scatter"))
    gs.timing_enable(False)
    flagged = int(count.item())
    by = RISK_BYTES_PER_REQUEST * A + 4 * flagged
    res["risk_scan"] = {
        "call_us": t_b2b, "call_us_isolated": t_iso, "input_copies_rotated": nc, "flagged_fraction": flagged / A,
        "requests_per_s": A / (t_b2b * 1e-6), "algorithmic_GBps": by / (t_b2b * 1e-6) / 1e9,
        "frac_of_hbm_peak": by / (t_b2b * 1e-6) / 1e9 / peak_gbs,
        "frac_of_hbm_peak_isolated": by / (t_iso * 1e-6) / 1e9 / peak_gbs,
        "kernel_us": {"risk_flags": t_fl[0] / t_fl[1] * 1e3, "risk_scatter": t_sc[0] / t_sc[1] * 1e3},
    }

    # ---- config 4: the stream of dependent rounds (route + advance, a scan after every round) ----
    if wl.cfg.n_rounds > 1:
        R = wl.cfg.n_rounds
        rounds = [[torch.from_numpy(c).to(dev) for c in W.make_round_requests(wl, k).columns()] for k in range(R)]
        o_idx = torch.empty(N, dtype=torch.int32, device=dev)
        o_est = torch.empty(N, dtype=torch.float32, device=dev)
        o_slack = torch.empty(N, dtype=torch.float32, device=dev)
        state0 = InstancePool.from_host(wl.types, wl.instances, dev)
        live = InstancePool.from_host(wl.types, wl.instances, dev)

        def reset_state():
            for name in ("queued_prefill_tokens", "decode_batch", "free_kv_tokens", "q_ema_ms"):
                getattr(live, name).copy_(getattr(state0, name))

        def enqueue_stream(st):
            for k in range(R):
                gs.route_batch(*rounds[k], live, alpha, o_idx, o_est, o_slack, None, accumulate=True, stream=st)
                gs.advance_state(live, stream=st)
                gs.risk_scan(*acts[k % nc], live, bits, cand, count, stream=st)

        side = torch.cuda.Stream(dev)
        how = "CUDA graph of the 64 rounds, replayed"
        graph = None
        try:
            reset_state()
            torch.cuda.synchronize(dev)
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                enqueue_stream(side)
        except Exception as exc:                      # capture refused: enqueue the rounds one by one
            graph = None
            how = "rounds enqueued one by one from the host (graph capture failed: %s)" % type(exc).__name__
        torch.cuda.synchronize(dev)

        def time_stream(use_graph):
            times = []
            for _ in range(7):
                reset_state()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize(dev)
                e0.record(stream)
                if use_graph:
                    graph.replay()
                else:
                    enqueue_stream(stream)
                e1.record(stream)
                torch.cuda.synchronize(dev)
                times.append(e0.elapsed_time(e1))
            return statistics.median(times)

        ms_host = time_stream(False)                  # enqueued call by call from Python
        ms = time_stream(True) if graph is not None else ms_host
        res["stream"] = {"rounds": R, "ms": ms, "us_per_round": ms / R * 1e3, "how": how,
                         "ms_enqueued_from_host": ms_host,
                         "requests_per_s": R * N / (ms * 1e-3), "logical_pairs_per_s": R * N * M / (ms * 1e-3),
                         "scans": R, "scan_requests_per_s": R * A / (ms * 1e-3),
                         "what": "per round: gs_route_batch(ACCUMULATE) + gs_advance_state + gs_risk_scan over the advanced state"}
    status = gs.device_status()
    res["device_status"] = status
    return res


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
    props = torch.cuda.get_device_properties(dev)
    n_sm = int(props.multi_processor_count)
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
    # ---- every workload shape, each entry point by itself (rank 0 of a one-GPU run) ----
    peak, peak_kind = load_peaks()
    per_config = None
    if world == 1 and not args.no_per_config:
        gs_count = None
        if not args.no_count:
            try:
                gs_count = GoodServe(local_rank, counting=True)
            except Exception as exc:                   # the counting build is optional equipment
                print(f"counting build unavailable: {exc}", file=sys.stderr)
        per_config = {}
        for cid in sorted(W.CONFIGS):
            per_config[str(cid)] = measure_config(gs, cid, rank_seed(cid, rank), dev, peak, gs_count)
            torch.cuda.empty_cache()
        if gs_count is not None:
            gs_count.close()
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

    # (the routing round's results travel back while the scan's inputs arrive: the first call
    # returns once it is enqueued, the second one waits for both)
    def e2e_step():
        gs.route_batch_host(*h_req, wl.types, wl.instances, alpha, h_idx, h_est, h_slack, stream=stream, wait=False)
        n_flagged = gs.risk_scan_host(*h_act, wl.types, wl.instances, h_bits, h_cand, stream=stream)
        gs.host_wait(stream)
        return n_flagged

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
    sm_max_hz = (clocks.get("sm_max_mhz") or 1965.0) * 1e6
    issue_peak = n_sm * SCHEDULERS_PER_SM * sm_max_hz      # SM count from the device, clock from nvidia-smi
    per_kernel = {}
    for name, (ms, n) in kernel_ms.items():
        per_kernel[name] = {"launches": n, "avg_us": ms / n * 1e3}
    dominant = max(kernel_ms, key=lambda k: kernel_ms[k][0]) if kernel_ms else None
    alg_bytes = {"route": ROUTE_BYTES_PER_REQUEST * N + 20 * M,
                 "risk_flags": 20 * A + 4 * ((A + 31) // 32),
                 "risk_scatter": 4 * ((A + 31) // 32) + 4 * flagged}
    roofline = None
    issue = None
    profiled = (PROFILED_ROUTE if PROFILED_ROUTE["sources_sha1"] == kernel_sources_sha1()
                and PROFILED_ROUTE["config"] == args.config else None)
    profiled_risk = (PROFILED_RISK_FLAGS if PROFILED_RISK_FLAGS["sources_sha1"] == risk_sources_sha1()
                     and PROFILED_RISK_FLAGS["config"] == args.config else None)
    if dominant in alg_bytes:
        ms, n = kernel_ms[dominant]
        in_step_order_us = ms / n * 1e3
        how = ("every launch between its own pair of CUDA events, serial pass in the step's order "
               "(prologue, route, risk_flags, risk_scatter)")
        us = in_step_order_us
        pc = (per_config or {}).get(str(args.config))
        loop_of = {"risk_flags": "risk_scan", "risk_scatter": "risk_scan", "route": "route", "prologue": "route"}
        if pc and dominant in pc[loop_of[dominant]]["kernel_us"]:
            # the same event pairs in a loop of calls of the kernel's own entry point (inputs rotated):
            # there the kernel does not also wait for the other entry point's dirty L2 lines to drain
            us = pc[loop_of[dominant]]["kernel_us"][dominant]
            how = ("every launch between its own pair of CUDA events, in a loop of %s calls with rotated inputs; "
                   "in the step's order, behind the other entry point's kernel: %.1f us" % (
                       "gs_" + ("risk_scan" if loop_of[dominant] == "risk_scan" else "route_batch"), in_step_order_us))
        achieved = alg_bytes[dominant] / (us * 1e-6) / 1e9
        roofline = {"bound": "hbm", "kernel": dominant, "achieved": achieved, "peak": peak, "unit": "GB/s",
                    "frac": achieved / peak, "launch_us": us, "how": how,
                    "traffic": (profiled["dram_bytes_per_launch"] if profiled and dominant == "route" else
                                profiled_risk["dram_bytes_per_launch"] if profiled_risk and dominant == "risk_flags" else None),
                    "peak_kind": f"of {peak_kind}", "algorithmic_bytes_per_launch": alg_bytes[dominant]}
    if profiled and "route" in kernel_ms:
        ms, n = kernel_ms["route"]
        rate = profiled["warp_instructions_per_launch"] / (ms / n * 1e-3)
        issue = {"kernel": "route", "bound": "alu", "achieved": rate, "peak": issue_peak,
                 "unit": "warp-instructions/s", "frac": rate / issue_peak,
                 "warp_instructions_per_request": profiled["warp_instructions_per_launch"] / N,
                 "note": "instruction count from ncu; peak = %d SMs x %d schedulers x %.3f GHz" % (
                     n_sm, SCHEDULERS_PER_SM, sm_max_hz / 1e9)}
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
        "value_note": "logical pairs: N x M per routing round -- pairs decided, not pairs scored; the search scores "
                      "about one pair per request exactly (per_config.*.route.evaluated_per_request)",
        "route_logical_pairs_per_s": world * N * M / (route_ms * 1e-3) if route_ms else None,
        "route_requests_per_s": world * N / (route_ms * 1e-3) if route_ms else None,
        "step_hbm_frac": step_bytes / (ms_per_step * 1e-3) / 1e9 / peak,
        "flagged_fraction": flagged / A, "device_status": status,
        "roofline": roofline, "issue": issue, "kernels": per_kernel,
        "route_call": None if not per_config else {
            "us": per_config[str(args.config)]["route"]["call_us"],
            "algorithmic_GBps": per_config[str(args.config)]["route"]["algorithmic_GBps"],
            "frac_of_hbm_peak": per_config[str(args.config)]["route"]["frac_of_hbm_peak"],
            "what": "gs_route_batch (prologue + route kernel) called back to back, inputs rotated"},
        "scan_call": None if not per_config else {
            "us": per_config[str(args.config)]["risk_scan"]["call_us"],
            "algorithmic_GBps": per_config[str(args.config)]["risk_scan"]["algorithmic_GBps"],
            "frac_of_hbm_peak": per_config[str(args.config)]["risk_scan"]["frac_of_hbm_peak"],
            "what": "gs_risk_scan (both passes) called back to back, inputs rotated"},
        "per_config": per_config, "reroute": reroute, "prefix": prefix, "direct": direct, "sequential": sequential,
        "kernel_timing": "serial pass of %d steps on one stream after the timed region, every launch between its own "
                         "pair of CUDA events (the pair adds about 3 us to each duration), %.4f ms/step" % (
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
    ap.add_argument("--no-per-config", action="store_true", help="skip the per-config block (all five workload shapes)")
    ap.add_argument("--no-count", action="store_true", help="skip the counting build (work per request)")
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
