"""CPU oracle for the routing hot path -- TEST INFRASTRUCTURE ONLY.

Thin ctypes wrapper over ``goodserve_oracle.c`` (plain C, built here with gcc).  Only the
tests, the smoke check and the benchmark's CPU-baseline leg may import this package; the
product (the CUDA library and its Python binding) never does, and this package never
imports the product.

The functions follow the paper's notation: ``q, p, d`` are the per-instance coefficients
of Eq. 2, ``x = L_in``, ``y = L_out``, ``D`` the E2E-SLO.  ``precision`` selects the
arithmetic: ``"f64"`` (authority for values) or ``"f32"`` (single precision in the fixed
operation order in which the kernels take their decisions).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "goodserve_oracle.c")

BAD_INSTANCE, BAD_TYPE, BAD_VALUE = 1, 2, 4


def _cpu_has_fma() -> bool:
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    return " fma " in (line + " ")
    except OSError:
        pass
    return False


def lib_path() -> str:
    tag = "fma" if _cpu_has_fma() else "nofma"
    return os.path.join(_HERE, "_build", f"libgoodserve_oracle_{tag}.so")


def build(force: bool = False) -> str:
    """Compile the C oracle (no contraction, no fast-math, so every operation rounds once)."""
    out = lib_path()
    if (not force and os.path.exists(out)
            and os.path.getmtime(out) >= os.path.getmtime(_SRC)):
        return out
    os.makedirs(os.path.dirname(out), exist_ok=True)
    cmd = ["gcc", "-O2", "-fPIC", "-shared", "-ffp-contract=off", "-fno-fast-math",
           "-Wall", "-Wextra"]
    if _cpu_has_fma():
        cmd.append("-mfma")           # fmaf() becomes one correctly-rounded instruction
    tmp = out + f".tmp{os.getpid()}"
    subprocess.run(cmd + [_SRC, "-lm", "-o", tmp], check=True)
    os.replace(tmp, out)
    return out


_lib = None


def _L():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.gso_compact.restype = C.c_int64
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


@dataclass
class InstanceTable:
    """Per-instance coefficients of Eq. 2 for one routing round."""
    q: np.ndarray      # queue delay after the EMA step (ms)
    p: np.ndarray      # per-token prefill latency (ms)
    d: np.ndarray      # per-token decode latency under load (ms)
    kv: np.ndarray     # free KV tokens, int64
    status: int
    precision: str

    @property
    def n_instances(self) -> int:
        return int(self.q.shape[0])


def instance_table(types, inst, ema_alpha: float, precision: str = "f64") -> InstanceTable:
    M = inst.n_instances
    real = np.float64 if precision == "f64" else np.float32
    q = np.empty(M, real); p = np.empty(M, real); d = np.empty(M, real)
    kv = np.empty(M, np.int64)
    status = C.c_uint(0)
    fn = getattr(_L(), f"gso_instance_table_{precision}")
    fn(C.c_int32(M), C.c_int32(types.n_types),
       _p(_c(inst.type_id, np.int32)), _p(_c(inst.queued_prefill_tokens, np.int32)),
       _p(_c(inst.decode_batch, np.int32)), _p(_c(inst.free_kv_tokens, np.int32)),
       _p(_c(inst.q_ema_ms, np.float32)),
       _p(_c(types.prefill_ms_per_tok, np.float32)), _p(_c(types.tpot_a_ms, np.float32)),
       _p(_c(types.tpot_b_ms, np.float32)), C.c_float(ema_alpha),
       _p(q), _p(p), _p(d), _p(kv), C.byref(status))
    return InstanceTable(q, p, d, kv, status.value, precision)


def direct_table(q_ms, p_ms_per_tok, d_ms_per_tok, free_kv_tokens, precision: str = "f64") -> InstanceTable:
    """The table of a round from coefficients given directly (black-box estimates, Sec. 3.3)."""
    qi = _c(q_ms, np.float32); pi = _c(p_ms_per_tok, np.float32); di = _c(d_ms_per_tok, np.float32)
    kvi = _c(free_kv_tokens, np.int32)
    M = qi.shape[0]
    real = np.float64 if precision == "f64" else np.float32
    q = np.empty(M, real); p = np.empty(M, real); d = np.empty(M, real); kv = np.empty(M, np.int64)
    status = C.c_uint(0)
    getattr(_L(), f"gso_direct_table_{precision}")(C.c_int32(M), _p(qi), _p(pi), _p(di), _p(kvi),
                                                   _p(q), _p(p), _p(d), _p(kv), C.byref(status))
    return InstanceTable(q, p, d, kv, status.value, precision)


def ema_update(alpha: float, observed, state, precision: str = "f64"):
    """One EMA step of a coefficient column: returns (new state, status)."""
    obs = _c(observed, np.float32)
    real = np.float64 if precision == "f64" else np.float32
    c_in = _c(state, real)
    c_out = np.empty_like(c_in)
    status = C.c_uint(0)
    getattr(_L(), f"gso_ema_update_{precision}")(C.c_int32(obs.shape[0]), C.c_float(alpha), _p(obs), _p(c_in),
                                                 _p(c_out), C.byref(status))
    return c_out, status.value


@dataclass
class RouteResult:
    instance_idx: np.ndarray   # int32[N]
    est_e2e_ms: np.ndarray     # real[N]
    slack_ms: np.ndarray       # real[N]
    tier: np.ndarray           # uint8[N]: 1 just-enough, 2 fallback among KV-ok, 3 fallback among all
    status: int


def _route_range(table: InstanceTable, x, y, D, out: RouteResult, lo: int, hi: int, status):
    fn = getattr(_L(), f"gso_route_{table.precision}")
    fn(C.c_int64(hi - lo), _p(x[lo:hi]), _p(y[lo:hi]), _p(D[lo:hi]),
       C.c_int32(table.n_instances), _p(table.q), _p(table.p), _p(table.d), _p(table.kv),
       _p(out.instance_idx[lo:hi]), _p(out.est_e2e_ms[lo:hi]), _p(out.slack_ms[lo:hi]),
       _p(out.tier[lo:hi]), C.byref(status))


def route(table: InstanceTable, prompt_len, pred_decode_len, slo_ms, threads: int = 1) -> RouteResult:
    """Algorithm 1 for every request.  ``threads > 1`` only splits the request range into
    contiguous chunks run by the same plain loop (requests are independent)."""
    x = _c(prompt_len, np.int32); y = _c(pred_decode_len, np.int32); D = _c(slo_ms, np.float32)
    N = x.shape[0]
    real = np.float64 if table.precision == "f64" else np.float32
    out = RouteResult(np.empty(N, np.int32), np.empty(N, real), np.empty(N, real),
                      np.empty(N, np.uint8), 0)
    if N == 0:
        return out
    threads = max(1, min(int(threads), N))
    bounds = np.linspace(0, N, threads + 1).astype(np.int64)
    stats = [C.c_uint(0) for _ in range(threads)]
    if threads == 1:
        _route_range(table, x, y, D, out, 0, N, stats[0])
    else:
        with ThreadPoolExecutor(threads) as ex:
            list(ex.map(lambda i: _route_range(table, x, y, D, out, int(bounds[i]),
                                               int(bounds[i + 1]), stats[i]), range(threads)))
    for s in stats:
        out.status |= s.value
    return out


def route_prefix(table: InstanceTable, prompt_len, pred_decode_len, slo_ms, prefix_inst, prefix_hit_len,
                 threads: int = 1) -> RouteResult:
    """Algorithm 1 with the prefix-cache term of Eq. 2.  ``prefix_inst`` / ``prefix_hit_len`` are
    int32 arrays of shape (n_slots, N): the instances on which request r has a cached prefix and
    the hit lengths (see the C file for the reading of empty, invalid and duplicate slots)."""
    x = _c(prompt_len, np.int32); y = _c(pred_decode_len, np.int32); D = _c(slo_ms, np.float32)
    N = x.shape[0]
    pi = _c(prefix_inst, np.int32).reshape(-1, N) if N else np.zeros((0, 0), np.int32)
    ph = _c(prefix_hit_len, np.int32).reshape(-1, N) if N else np.zeros((0, 0), np.int32)
    assert pi.shape == ph.shape
    K = pi.shape[0]
    real = np.float64 if table.precision == "f64" else np.float32
    out = RouteResult(np.empty(N, np.int32), np.empty(N, real), np.empty(N, real),
                      np.empty(N, np.uint8), 0)
    if N == 0:
        return out
    fn = getattr(_L(), f"gso_route_prefix_{table.precision}")
    threads = max(1, min(int(threads), N))
    bounds = np.linspace(0, N, threads + 1).astype(np.int64)
    stats = [C.c_uint(0) for _ in range(threads)]

    def run(i):
        lo, hi = int(bounds[i]), int(bounds[i + 1])
        pi_c = np.ascontiguousarray(pi[:, lo:hi]); ph_c = np.ascontiguousarray(ph[:, lo:hi])
        fn(C.c_int64(hi - lo), _p(x[lo:hi]), _p(y[lo:hi]), _p(D[lo:hi]), C.c_int32(K), _p(pi_c), _p(ph_c),
           C.c_int32(table.n_instances), _p(table.q), _p(table.p), _p(table.d), _p(table.kv),
           _p(out.instance_idx[lo:hi]), _p(out.est_e2e_ms[lo:hi]), _p(out.slack_ms[lo:hi]),
           _p(out.tier[lo:hi]), C.byref(stats[i]))

    if threads == 1:
        run(0)
    else:
        with ThreadPoolExecutor(threads) as ex:
            list(ex.map(run, range(threads)))
    for s in stats:
        out.status |= s.value
    return out


def route_sequential(types, inst, ema_alpha: float, prompt_len, pred_decode_len, slo_ms) -> RouteResult:
    """Algorithm 1 one request at a time, each seeing the state left by the ones before it.
    ``inst`` (a workloads.InstanceState) is advanced in place.  Single precision."""
    x = _c(prompt_len, np.int32); y = _c(pred_decode_len, np.int32); D = _c(slo_ms, np.float32)
    N = x.shape[0]
    for a in inst.columns():
        assert a.flags.c_contiguous
    out = RouteResult(np.empty(N, np.int32), np.empty(N, np.float32), np.empty(N, np.float32),
                      np.empty(N, np.uint8), 0)
    status = C.c_uint(0)
    _L().gso_route_sequential_f32(
        C.c_int64(N), _p(x), _p(y), _p(D), C.c_int32(inst.n_instances), C.c_int32(types.n_types),
        _p(_c(inst.type_id, np.int32)), _p(inst.queued_prefill_tokens), _p(inst.decode_batch),
        _p(inst.free_kv_tokens), _p(inst.q_ema_ms),
        _p(_c(types.prefill_ms_per_tok, np.float32)), _p(_c(types.tpot_a_ms, np.float32)),
        _p(_c(types.tpot_b_ms, np.float32)), C.c_float(ema_alpha),
        _p(out.instance_idx), _p(out.est_e2e_ms), _p(out.slack_ms), _p(out.tier), C.byref(status))
    out.status = status.value
    return out


@dataclass
class RiskResult:
    flag: np.ndarray        # uint8[A]
    finish_ms: np.ndarray   # real[A]
    status: int


def risk(table: InstanceTable, assigned_inst, generated_tokens, pred_len, elapsed_ms, slo_ms,
         threads: int = 1) -> RiskResult:
    g = _c(assigned_inst, np.int32); gen = _c(generated_tokens, np.int32)
    tot = _c(pred_len, np.int32); el = _c(elapsed_ms, np.float32); slo = _c(slo_ms, np.float32)
    A = g.shape[0]
    real = np.float64 if table.precision == "f64" else np.float32
    out = RiskResult(np.empty(A, np.uint8), np.empty(A, real), 0)
    if A == 0:
        return out
    fn = getattr(_L(), f"gso_risk_{table.precision}")
    threads = max(1, min(int(threads), A))
    bounds = np.linspace(0, A, threads + 1).astype(np.int64)
    stats = [C.c_uint(0) for _ in range(threads)]

    def run(i):
        lo, hi = int(bounds[i]), int(bounds[i + 1])
        fn(C.c_int64(hi - lo), _p(g[lo:hi]), _p(gen[lo:hi]), _p(tot[lo:hi]), _p(el[lo:hi]),
           _p(slo[lo:hi]), C.c_int32(table.n_instances), _p(table.d),
           _p(out.flag[lo:hi]), _p(out.finish_ms[lo:hi]), C.byref(stats[i]))

    if threads == 1:
        run(0)
    else:
        with ThreadPoolExecutor(threads) as ex:
            list(ex.map(run, range(threads)))
    for s in stats:
        out.status |= s.value
    return out


def compact(flag: np.ndarray, capacity: Optional[int] = None):
    """Packed flag words, ascending candidate list (at most ``capacity`` entries) and the
    true number of flagged requests."""
    flag = _c(flag, np.uint8)
    A = flag.shape[0]
    cap = A if capacity is None else int(capacity)
    bits = np.zeros((A + 31) // 32, np.uint32)
    cand = np.empty(max(cap, 0), np.int32)
    count = _L().gso_compact(C.c_int64(A), _p(flag), _p(bits), _p(cand), C.c_int64(cap))
    return bits, cand[:min(count, cap)], int(count)


def advance(inst, table_f32: InstanceTable, instance_idx, prompt_len, pred_decode_len):
    """Apply one round's assignments to the instance state, in place (see the C source)."""
    assert table_f32.precision == "f32", "the carried EMA state is single precision"
    idx = _c(instance_idx, np.int32); x = _c(prompt_len, np.int32); y = _c(pred_decode_len, np.int32)
    for a in inst.columns():
        assert a.flags.c_contiguous
    _L().gso_advance(C.c_int32(inst.n_instances), C.c_int64(idx.shape[0]), _p(idx), _p(x), _p(y),
                     _p(inst.queued_prefill_tokens), _p(inst.decode_batch),
                     _p(inst.free_kv_tokens), _p(inst.q_ema_ms), _p(table_f32.q))


@dataclass
class RerouteResult:
    new_instance: np.ndarray   # int32[n_cand], -1 = no strictly faster instance exists
    est_ms: np.ndarray         # real[n_cand]: estimated remaining time on the target
    slack_ms: np.ndarray       # real[n_cand]: (slo - elapsed) - est
    tier: np.ndarray           # uint8[n_cand]: 0 no move, 1 just-enough, 2 / 3 fallback
    status: int


def reroute(table: InstanceTable, cand_idx, assigned_inst, generated_tokens, pred_len, elapsed_ms,
            slo_ms, prompt_len) -> RerouteResult:
    """Re-routing of flagged requests among strictly faster instances (see the C source)."""
    cand = _c(cand_idx, np.int32)
    g = _c(assigned_inst, np.int32); gen = _c(generated_tokens, np.int32)
    tot = _c(pred_len, np.int32); el = _c(elapsed_ms, np.float32); slo = _c(slo_ms, np.float32)
    x = _c(prompt_len, np.int32)
    n = cand.shape[0]
    real = np.float64 if table.precision == "f64" else np.float32
    out = RerouteResult(np.empty(n, np.int32), np.empty(n, real), np.empty(n, real), np.empty(n, np.uint8), 0)
    status = C.c_uint(0)
    if n:
        fn = getattr(_L(), f"gso_reroute_{table.precision}")
        fn(C.c_int64(n), _p(cand), _p(g), _p(gen), _p(tot), _p(el), _p(slo), _p(x),
           C.c_int32(table.n_instances), _p(table.q), _p(table.p), _p(table.d), _p(table.kv),
           _p(out.new_instance), _p(out.est_ms), _p(out.slack_ms), _p(out.tier), C.byref(status))
    out.status = status.value
    return out
