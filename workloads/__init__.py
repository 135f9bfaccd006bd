"""Seeded synthetic inputs for the routing hot path.

This module only *draws inputs*: request columns, the GPU-type table, per-instance
serving state and the active-request population.  It holds none of the routing
method's arithmetic (no latency estimate, no selection, no risk test) so that the
CPU oracle and the CUDA path can both consume exactly the same arrays without
sharing any code of the method itself.

The distributions stand in for the paper's evaluation workload (a mix of agentic
benchmarks replayed on a production arrival trace, Sec. 4.1 "Workloads"), which is
not available offline; nothing of those datasets is reproduced.  Every array is a
NumPy array in host memory; integer columns are int32, real columns float32.

Streams: every column draws from its own Philox stream keyed by
``(seed, stream_id)`` so that changing the number of requests never reshuffles
another column.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Optional, Tuple

import numpy as np

# --------------------------------------------------------------------------------------
# configuration table (the five workload shapes)
# --------------------------------------------------------------------------------------

#: per-type constants of the smallest pool: prefill rate (tokens/ms), and the decode
#: time-per-output-token model  tpot_ms = a + b * decode_batch.
BASE_TYPES: Tuple[Tuple[float, float, float], ...] = (
    (40.0, 8.0, 0.05),
    (20.0, 14.0, 0.08),
    (10.0, 25.0, 0.15),
)


@dataclass(frozen=True)
class Config:
    cfg_id: int
    n_requests: int          # N, pending requests per routing round
    n_instances: int         # M
    n_types: int             # Tn
    n_active: int            # A, active requests per risk scan
    slo_lo: float = 1.5      # SLO = U[slo_lo, slo_hi] * ideal
    slo_hi: float = 5.0
    decode: str = "lognormal"        # "lognormal" | "bimodal"
    active_sigma: float = 1.0        # sigma of the active population's decode lengths
    n_rounds: int = 1                # >1: a stream of dependent rounds
    ema_alpha: float = 0.5


CONFIGS: Dict[int, Config] = {
    0: Config(0, 256, 8, 3, 1024),
    1: Config(1, 65_536, 64, 4, 262_144),
    2: Config(2, 1_048_576, 256, 6, 4_194_304, decode="bimodal"),
    3: Config(3, 4_194_304, 1024, 8, 16_777_216, slo_lo=1.1, slo_hi=2.0),
    4: Config(4, 131_072, 512, 6, 2_097_152, active_sigma=1.5, n_rounds=64),
}

# stream ids (second word of the Philox key)
_S_TYPES, _S_INST, _S_PROMPT, _S_DECODE, _S_SLO, _S_MIX = 1, 2, 3, 4, 5, 6
_S_A_INST, _S_A_PRED, _S_A_GEN, _S_A_PROMPT, _S_A_SLO, _S_A_ELAPSED = 10, 11, 12, 13, 14, 15
_S_PFX_HAS, _S_PFX_INST, _S_PFX_LEN = 20, 21, 22
_S_BB_Q, _S_BB_P, _S_BB_D, _S_BB_OBS = 60, 61, 62, 63
_ROUND_STRIDE = 1000  # stream ids of round k are offset by k * _ROUND_STRIDE


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed) & (2**64 - 1), int(stream)]))


# --------------------------------------------------------------------------------------
# containers
# --------------------------------------------------------------------------------------

@dataclass
class TypeTable:
    prefill_ms_per_tok: np.ndarray   # f32[Tn]   p_t = 1 / prefill rate
    tpot_a_ms: np.ndarray            # f32[Tn]
    tpot_b_ms: np.ndarray            # f32[Tn]

    @property
    def n_types(self) -> int:
        return int(self.prefill_ms_per_tok.shape[0])


@dataclass
class InstanceState:
    type_id: np.ndarray                 # i32[M]
    queued_prefill_tokens: np.ndarray   # i32[M]
    decode_batch: np.ndarray            # i32[M]
    free_kv_tokens: np.ndarray          # i32[M]
    q_ema_ms: np.ndarray                # f32[M]

    @property
    def n_instances(self) -> int:
        return int(self.type_id.shape[0])

    def copy(self) -> "InstanceState":
        return InstanceState(*(a.copy() for a in self.columns()))

    def columns(self):
        return (self.type_id, self.queued_prefill_tokens, self.decode_batch,
                self.free_kv_tokens, self.q_ema_ms)


@dataclass
class RequestBatch:
    prompt_len: np.ndarray        # i32[N]
    pred_decode_len: np.ndarray   # i32[N]
    slo_ms: np.ndarray            # f32[N]

    @property
    def n(self) -> int:
        return int(self.prompt_len.shape[0])

    def columns(self):
        return (self.prompt_len, self.pred_decode_len, self.slo_ms)


@dataclass
class ActiveSet:
    assigned_inst: np.ndarray     # i32[A]
    generated_tokens: np.ndarray  # i32[A]
    pred_len: np.ndarray          # i32[A]  re-estimated TOTAL output length
    elapsed_ms: np.ndarray        # f32[A]
    slo_ms: np.ndarray            # f32[A]

    @property
    def n(self) -> int:
        return int(self.assigned_inst.shape[0])

    def columns(self):
        return (self.assigned_inst, self.generated_tokens, self.pred_len,
                self.elapsed_ms, self.slo_ms)


@dataclass
class Workload:
    cfg: Config
    seed: int
    types: TypeTable
    instances: InstanceState
    requests: RequestBatch           # round 0 (the only round unless cfg.n_rounds > 1)
    active: ActiveSet
    ema_alpha: float = 0.5
    extra: dict = field(default_factory=dict)


# --------------------------------------------------------------------------------------
# draws
# --------------------------------------------------------------------------------------

def make_types(n_types: int, seed: int, perturb: bool) -> TypeTable:
    """Type ``t`` takes base triple ``t mod 3``; with ``perturb`` each of its three
    constants is multiplied by an independent U[0.5, 2] factor."""
    rate = np.empty(n_types, np.float64)
    a = np.empty(n_types, np.float64)
    b = np.empty(n_types, np.float64)
    rng = _rng(seed, _S_TYPES)
    for t in range(n_types):
        r0, a0, b0 = BASE_TYPES[t % len(BASE_TYPES)]
        f = rng.uniform(0.5, 2.0, size=3) if perturb else np.ones(3)
        rate[t], a[t], b[t] = r0 * f[0], a0 * f[1], b0 * f[2]
    rate32 = rate.astype(np.float32)
    p = (np.float32(1.0) / rate32).astype(np.float32)       # computed once, passed as data
    return TypeTable(p, a.astype(np.float32), b.astype(np.float32))


def make_instances(n_instances: int, types: TypeTable, seed: int) -> InstanceState:
    rng = _rng(seed, _S_INST)
    g = np.arange(n_instances, dtype=np.int64)
    type_id = (g % types.n_types).astype(np.int32)
    queued = rng.integers(0, 20_001, size=n_instances, dtype=np.int64).astype(np.int32)
    batch = rng.integers(0, 65, size=n_instances, dtype=np.int64).astype(np.int32)
    free_kv = rng.integers(0, 200_001, size=n_instances, dtype=np.int64).astype(np.int32)
    jitter = rng.uniform(0.8, 1.2, size=n_instances)
    q_ema = (queued.astype(np.float64) * types.prefill_ms_per_tok[type_id].astype(np.float64)
             * jitter).astype(np.float32)
    return InstanceState(type_id, queued, batch, free_kv, q_ema)


def _lognormal_tokens(rng: np.random.Generator, n: int, mu, sigma, lo: int, hi: int) -> np.ndarray:
    z = rng.standard_normal(n)
    v = np.rint(np.exp(mu + sigma * z))
    return np.clip(v, lo, hi).astype(np.int32)


def _decode_lengths(rng_len, rng_mix, n: int, mode: str, sigma_override: Optional[float] = None):
    if mode == "bimodal":
        pick = rng_mix.random(n) < 0.5
        mu = np.where(pick, 4.0, 7.0)
        return _lognormal_tokens(rng_len, n, mu, 0.8, 8, 8192)
    sigma = 1.0 if sigma_override is None else sigma_override
    return _lognormal_tokens(rng_len, n, 5.5, sigma, 8, 8192)


def _unloaded_latency_ms(types: TypeTable, prompt_len: np.ndarray, decode_len: np.ndarray) -> np.ndarray:
    """Base latency used only to *scale the SLO draw*: the smallest, over GPU types, of
    prompt_len * p_t + decode_len * a_t (an empty, idle instance of that type).  This mirrors
    how the paper sets deadlines: a base latency measured with the request running alone,
    times a relaxation factor (Sec. 4.1)."""
    p = types.prefill_ms_per_tok.astype(np.float64)[:, None]
    a = types.tpot_a_ms.astype(np.float64)[:, None]
    x = prompt_len.astype(np.float64)[None, :]
    y = decode_len.astype(np.float64)[None, :]
    # chunk to bound the temporary for large N
    out = np.empty(prompt_len.shape[0], np.float64)
    step = 1 << 20
    for s in range(0, out.shape[0], step):
        e = min(s + step, out.shape[0])
        out[s:e] = np.min(p * x[:, s:e] + a * y[:, s:e], axis=0)
    return out


def make_requests(cfg: Config, types: TypeTable, seed: int, n: Optional[int] = None,
                  round_idx: int = 0) -> RequestBatch:
    n = cfg.n_requests if n is None else int(n)
    off = round_idx * _ROUND_STRIDE
    prompt = _lognormal_tokens(_rng(seed, _S_PROMPT + off), n, 6.5, 1.0, 16, 16384)
    decode = _decode_lengths(_rng(seed, _S_DECODE + off), _rng(seed, _S_MIX + off), n, cfg.decode)
    scale = _rng(seed, _S_SLO + off).uniform(cfg.slo_lo, cfg.slo_hi, size=n)
    slo = (scale * _unloaded_latency_ms(types, prompt, decode)).astype(np.float32)
    return RequestBatch(prompt, decode, slo)


@dataclass
class BlackBoxTable:
    """Per-instance coefficients of Eq. 2 as a monitor would report them (Sec. 3.3)."""
    q_ms: np.ndarray            # f32[M]
    p_ms_per_tok: np.ndarray    # f32[M]
    d_ms_per_tok: np.ndarray    # f32[M]
    free_kv_tokens: np.ndarray  # i32[M]

    @property
    def n_instances(self) -> int:
        return int(self.q_ms.shape[0])

    def columns(self):
        return self.q_ms, self.p_ms_per_tok, self.d_ms_per_tok, self.free_kv_tokens


def make_blackbox_table(types: TypeTable, inst: InstanceState, seed: int, jitter: float = 0.05) -> BlackBoxTable:
    """What black-box monitoring of the pool ``(types, inst)`` would hand to the router: the
    pool's nominal per-instance values, each with its own multiplicative measurement jitter
    (so no two instances share p exactly, unlike the typed description)."""
    M = inst.n_instances
    t = inst.type_id
    u = lambda sid: _rng(seed, sid).uniform(1.0 - jitter, 1.0 + jitter, size=M)
    p = types.prefill_ms_per_tok[t].astype(np.float64) * u(_S_BB_P)
    d = (types.tpot_a_ms[t].astype(np.float64)
         + types.tpot_b_ms[t].astype(np.float64) * inst.decode_batch.astype(np.float64)) * u(_S_BB_D)
    q = inst.q_ema_ms.astype(np.float64) * u(_S_BB_Q)
    return BlackBoxTable(q.astype(np.float32), p.astype(np.float32), d.astype(np.float32),
                         inst.free_kv_tokens.copy())


def make_observations(column: np.ndarray, seed: int, step: int, jitter: float = 0.2) -> np.ndarray:
    """A fresh noisy observation of a coefficient column (input of one EMA step)."""
    u = _rng(seed, _S_BB_OBS + 7 * step).uniform(1.0 - jitter, 1.0 + jitter, size=column.shape[0])
    return (column.astype(np.float64) * u).astype(np.float32)


def make_prefix_hits(requests: RequestBatch, n_instances: int, seed: int, n_slots: int = 1,
                     hit_share: float = 0.35, block: int = 16) -> Tuple[np.ndarray, np.ndarray]:
    """Sparse prefix-cache state for a batch: ``(prefix_inst, prefix_hit_len)``, int32 arrays
    of shape (n_slots, N).  A share ``hit_share`` of the requests has a cached prefix in slot 0
    (system prompts and multi-turn sessions); each further slot is filled for half of the
    requests that filled the one before (replicated prefixes).  The instance is uniform over
    the pool, the hit a uniform fraction of the prompt rounded down to whole KV blocks of
    ``block`` tokens.  Empty slots hold instance -1 and length 0."""
    n = requests.prompt_len.shape[0]
    pi = np.full((n_slots, n), -1, np.int32)
    ph = np.zeros((n_slots, n), np.int32)
    has = np.ones(n, bool)
    for k in range(n_slots):
        u = _rng(seed, _S_PFX_HAS + 10 * k).random(n)
        has = has & (u < (hit_share if k == 0 else 0.5))
        g = _rng(seed, _S_PFX_INST + 10 * k).integers(0, n_instances, size=n, dtype=np.int64)
        frac = _rng(seed, _S_PFX_LEN + 10 * k).random(n)
        length = (np.floor(frac * requests.prompt_len.astype(np.float64)) // block * block).astype(np.int32)
        pi[k] = np.where(has, g, -1).astype(np.int32)
        ph[k] = np.where(has, length, 0).astype(np.int32)
    return pi, ph


def make_active(cfg: Config, types: TypeTable, n_instances: int, seed: int,
                n: Optional[int] = None) -> ActiveSet:
    n = cfg.n_active if n is None else int(n)
    assigned = _rng(seed, _S_A_INST).integers(0, n_instances, size=n, dtype=np.int64).astype(np.int32)
    sigma = cfg.active_sigma
    if cfg.decode == "bimodal":
        pred = _decode_lengths(_rng(seed, _S_A_PRED), _rng(seed, _S_A_PRED + 50), n, "bimodal")
    else:
        pred = _decode_lengths(_rng(seed, _S_A_PRED), None, n, "lognormal", sigma)
    u = _rng(seed, _S_A_GEN).random(n)
    generated = np.minimum(np.floor(u * (pred.astype(np.float64) + 1.0)), pred).astype(np.int32)
    prompt = _lognormal_tokens(_rng(seed, _S_A_PROMPT), n, 6.5, 1.0, 16, 16384)  # private, not passed on
    scale = _rng(seed, _S_A_SLO).uniform(cfg.slo_lo, cfg.slo_hi, size=n)
    slo = (scale * _unloaded_latency_ms(types, prompt, pred)).astype(np.float32)
    elapsed = (_rng(seed, _S_A_ELAPSED).random(n) * slo.astype(np.float64)).astype(np.float32)
    return ActiveSet(assigned, generated, pred, elapsed, slo)


def make_workload(cfg_id: int, seed: Optional[int] = None, n_requests: Optional[int] = None,
                  n_active: Optional[int] = None) -> Workload:
    """Draw the full input set of configuration ``cfg_id`` (seed defaults to ``cfg_id``).
    ``n_requests`` / ``n_active`` shrink or grow the populations without touching the
    pool (types and instances)."""
    cfg = CONFIGS[cfg_id]
    seed = cfg_id if seed is None else int(seed)
    types = make_types(cfg.n_types, seed, perturb=(cfg_id != 0))
    inst = make_instances(cfg.n_instances, types, seed)
    req = make_requests(cfg, types, seed, n_requests)
    act = make_active(cfg, types, cfg.n_instances, seed, n_active)
    return Workload(cfg, seed, types, inst, req, act, cfg.ema_alpha)


def make_round_requests(wl: Workload, round_idx: int, n: Optional[int] = None) -> RequestBatch:
    """Requests of round ``round_idx`` of a multi-round stream (round 0 == ``wl.requests``
    when sizes agree)."""
    return make_requests(wl.cfg, wl.types, wl.seed, n, round_idx)


def make_pool(n_instances: int, n_types: int, seed: int, perturb: bool = True):
    """A free-form pool (types + instances) for edge-size tests."""
    types = make_types(n_types, seed, perturb)
    return types, make_instances(n_instances, types, seed)
