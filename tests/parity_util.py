"""Helpers of the GPU parity tests: run the CUDA path through the binding, run the oracle,
and compare under the documented rules."""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

import oracle

REL_TOL = 1e-5     # tolerance for fp32 latency estimates against the fp64 oracle


@dataclass
class GpuRoute:
    instance_idx: np.ndarray
    est_e2e_ms: np.ndarray
    slack_ms: np.ndarray
    tier: np.ndarray


def gpu_route(gs, pool, req, alpha, accumulate=False, with_tier=True):
    import torch
    dev = gs.device
    n = req.n
    x = torch.from_numpy(req.prompt_len).to(dev)
    y = torch.from_numpy(req.pred_decode_len).to(dev)
    D = torch.from_numpy(req.slo_ms).to(dev)
    idx = torch.full((n,), -7, dtype=torch.int32, device=dev)
    est = torch.full((n,), float("nan"), dtype=torch.float32, device=dev)
    slack = torch.full((n,), float("nan"), dtype=torch.float32, device=dev)
    tier = torch.zeros(n, dtype=torch.uint8, device=dev) if with_tier else None
    gs.route_batch(x, y, D, pool, alpha, idx, est, slack, tier, accumulate=accumulate)
    torch.cuda.synchronize(dev)
    return GpuRoute(idx.cpu().numpy(), est.cpu().numpy(), slack.cpu().numpy(),
                    tier.cpu().numpy() if with_tier else None)


def gpu_route_prefix(gs, pool, req, alpha, prefix_inst, prefix_hit_len, pad_to=None):
    """prefix_inst / prefix_hit_len: int32 arrays (n_slots, N); columns are padded to a stride
    that is a multiple of 4 (``pad_to`` forces a larger one)."""
    import torch
    dev = gs.device
    n = req.n
    K = prefix_inst.shape[0]
    stride = max((n + 3) // 4 * 4, pad_to or 0)
    pi = np.full((K, stride), 12345, np.int32)          # padding must never be read as a slot
    ph = np.full((K, stride), 999, np.int32)
    pi[:, :n] = prefix_inst
    ph[:, :n] = prefix_hit_len
    x = torch.from_numpy(req.prompt_len).to(dev)
    y = torch.from_numpy(req.pred_decode_len).to(dev)
    D = torch.from_numpy(req.slo_ms).to(dev)
    pi_d = torch.from_numpy(pi.reshape(-1)).to(dev)
    ph_d = torch.from_numpy(ph.reshape(-1)).to(dev)
    idx = torch.full((n,), -7, dtype=torch.int32, device=dev)
    est = torch.full((n,), float("nan"), dtype=torch.float32, device=dev)
    slack = torch.full((n,), float("nan"), dtype=torch.float32, device=dev)
    tier = torch.zeros(n, dtype=torch.uint8, device=dev)
    gs.route_batch_prefix(x, y, D, pi_d, ph_d, K, stride, pool, alpha, idx, est, slack, tier)
    torch.cuda.synchronize(dev)
    return GpuRoute(idx.cpu().numpy(), est.cpu().numpy(), slack.cpu().numpy(), tier.cpu().numpy())


def gpu_route_direct(gs, bb, req):
    """bb: workloads.BlackBoxTable (or anything with .columns() -> q, p, d, kv as numpy)."""
    import torch
    dev = gs.device
    n = req.n
    q, p, d, kv = (torch.from_numpy(np.ascontiguousarray(c)).to(dev) for c in bb.columns())
    x = torch.from_numpy(req.prompt_len).to(dev)
    y = torch.from_numpy(req.pred_decode_len).to(dev)
    D = torch.from_numpy(req.slo_ms).to(dev)
    idx = torch.full((n,), -7, dtype=torch.int32, device=dev)
    est = torch.full((n,), float("nan"), dtype=torch.float32, device=dev)
    slack = torch.full((n,), float("nan"), dtype=torch.float32, device=dev)
    tier = torch.zeros(n, dtype=torch.uint8, device=dev)
    gs.route_batch_direct(x, y, D, q, p, d, kv, idx, est, slack, tier)
    torch.cuda.synchronize(dev)
    return GpuRoute(idx.cpu().numpy(), est.cpu().numpy(), slack.cpu().numpy(), tier.cpu().numpy())


@dataclass
class GpuRisk:
    flag_bits: np.ndarray     # uint32 words
    cand_idx: np.ndarray
    count: int


def gpu_risk(gs, pool, act, capacity=None):
    import torch
    dev = gs.device
    n = act.n
    cols = [torch.from_numpy(c).to(dev) for c in act.columns()]
    words = (n + 31) // 32
    bits = torch.full((max(words, 1),), -1, dtype=torch.int32, device=dev)
    cap = n if capacity is None else capacity
    cand = torch.full((max(cap, 1),), -9, dtype=torch.int32, device=dev)
    count = torch.full((1,), -1, dtype=torch.int64, device=dev)
    gs.risk_scan(*cols, pool, bits, cand, count, cand_capacity=cap)
    torch.cuda.synchronize(dev)
    c = int(count.item())
    return GpuRisk(bits.cpu().numpy().view(np.uint32)[:words], cand.cpu().numpy()[:min(c, cap)], c), \
        cand.cpu().numpy()


def unpack_bits(words: np.ndarray, n: int) -> np.ndarray:
    return np.unpackbits(words.view(np.uint8), bitorder="little")[:n]


def assert_route_matches_f32_oracle(got: GpuRoute, ref):
    """Decisions are taken in the same single-precision operation order on both sides, so
    every output must be bit-identical."""
    np.testing.assert_array_equal(got.instance_idx, ref.instance_idx)
    if got.tier is not None:
        np.testing.assert_array_equal(got.tier, ref.tier)
    np.testing.assert_array_equal(got.est_e2e_ms.view(np.uint32), ref.est_e2e_ms.view(np.uint32))
    np.testing.assert_array_equal(got.slack_ms.view(np.uint32), ref.slack_ms.view(np.uint32))


def check_route_against_f64(got: GpuRoute, tab64, req, max_explain=5):
    """fp64 authority: estimates within REL_TOL where the index agrees; an index that differs
    must be a documented near-tie.  Returns the number of accepted near-tie mismatches."""
    ref = oracle.route(tab64, *req.columns(), threads=8)
    same = got.instance_idx == ref.instance_idx
    err = np.abs(got.est_e2e_ms[same] - ref.est_e2e_ms[same]) / np.maximum(np.abs(ref.est_e2e_ms[same]), 1e-30)
    assert err.size == 0 or err.max() <= REL_TOL, f"est_e2e relative error {err.max()}"
    D = req.slo_ms.astype(np.float64)
    serr = np.abs(got.slack_ms[same] - ref.slack_ms[same])
    assert (serr <= REL_TOL * np.maximum(np.abs(ref.est_e2e_ms[same]), np.abs(D[same])) + 1e-30).all()
    bad = np.nonzero(~same)[0]
    kv = tab64.kv
    for r in bad:
        x, y = float(req.prompt_len[r]), float(req.pred_decode_len[r])
        T = tab64.q + tab64.p * x + tab64.d * y
        ok = (int(req.prompt_len[r]) + int(req.pred_decode_len[r])) <= kv
        amb = np.abs(T - D[r]) <= REL_TOL * np.maximum(np.abs(T), abs(D[r]))
        definitely = ok & (T <= D[r]) & ~amb
        maybe = ok & ((T <= D[r]) | amb)
        g = int(got.instance_idx[r])
        order = np.arange(len(T))
        preferred = (tab64.d > tab64.d[g]) | ((tab64.d == tab64.d[g]) & (order < g))
        tier1_ok = maybe[g] and not (definitely & preferred).any()
        pool = ok if ok.any() else np.ones_like(ok)
        tmin = T[pool].min()
        fb_ok = (not definitely.any()) and pool[g] and (T[g] - tmin) <= REL_TOL * abs(tmin)
        assert tier1_ok or fb_ok, f"request {r}: GPU chose {g}, oracle {ref.instance_idx[r]}, not a near-tie"
    return len(bad)


def check_risk_against_f64(flags: np.ndarray, tab64, act):
    ref = oracle.risk(tab64, *act.columns(), threads=8)
    diff = np.nonzero(flags != ref.flag)[0]
    slo = act.slo_ms.astype(np.float64)
    for i in diff:
        f = ref.finish_ms[i]
        assert abs(f - slo[i]) <= REL_TOL * max(abs(f), abs(slo[i])), f"risk flag {i} differs away from a tie"
    return len(diff)
