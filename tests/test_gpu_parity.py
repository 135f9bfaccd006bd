"""GPU parity: the CUDA path, called through the C ABI (ctypes binding), against the CPU
oracle on the same seeded inputs.  Integer results (instance index, tier, flag bits,
candidate list, advanced state) are compared bit for bit with the oracle's fixed-order
single-precision mode; latency estimates are compared with the fp64 oracle within 1e-5
relative, and any index that differs from the fp64 oracle must be a documented near-tie."""
import numpy as np
import pytest

import oracle
import workloads as W
from parity_util import (REL_TOL, GpuRoute, assert_route_matches_f32_oracle, check_risk_against_f64,
                         check_route_against_f64, gpu_risk, gpu_route, gpu_route_direct, gpu_route_prefix,
                         unpack_bits)

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def gs():
    from paper_2605_16867_b200 import GoodServe
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    ctx = GoodServe(0)
    yield ctx
    ctx.close()


def pool_of(gs, types, inst):
    from paper_2605_16867_b200 import InstancePool
    return InstancePool.from_host(types, inst, gs.device)


def run_config(gs, wl, threads=8):
    alpha = wl.ema_alpha
    pool = pool_of(gs, wl.types, wl.instances)
    t32 = oracle.instance_table(wl.types, wl.instances, alpha, "f32")
    t64 = oracle.instance_table(wl.types, wl.instances, alpha, "f64")
    got = gpu_route(gs, pool, wl.requests, alpha)
    ref = oracle.route(t32, *wl.requests.columns(), threads=threads)
    assert_route_matches_f32_oracle(got, ref)
    n_tie = check_route_against_f64(got, t64, wl.requests)
    # invariant: whenever any instance meets deadline and KV, the chosen one does
    t1 = got.tier == 1
    assert (got.slack_ms[t1] >= 0).all() and (got.slack_ms[got.tier == 2] < 0).all()

    risk, _ = gpu_risk(gs, pool, wl.active)
    rref = oracle.risk(t32, *wl.active.columns(), threads=threads)
    bits, cand, count = oracle.compact(rref.flag)
    np.testing.assert_array_equal(risk.flag_bits, bits)
    assert risk.count == count
    np.testing.assert_array_equal(risk.cand_idx, cand)
    n_flag_tie = check_risk_against_f64(unpack_bits(risk.flag_bits, wl.active.n), t64, wl.active)
    assert gs.device_status() == 0
    print(f"cfg {wl.cfg.cfg_id}: N={wl.requests.n} M={wl.instances.n_instances} A={wl.active.n} "
          f"tiers={[int((got.tier == k).sum()) for k in (1, 2, 3)]} flagged={count} "
          f"near-tie index mismatches vs fp64={n_tie}, flag mismatches vs fp64={n_flag_tie}")


@pytest.mark.parametrize("cfg_id", [0, 1, 2])
def test_config_full_size(gs, cfg_id):
    run_config(gs, W.make_workload(cfg_id))


def test_config3_full_size(gs):
    """Largest shape: 4,194,304 requests x 1,024 instances, 16,777,216 active requests."""
    run_config(gs, W.make_workload(3))


def test_config4_stream(gs):
    """64 dependent rounds with state advance on the device, a risk scan after every 8th
    round against the advanced state; the whole trajectory must match the oracle's."""
    wl = W.make_workload(4)
    alpha = wl.ema_alpha
    pool = pool_of(gs, wl.types, wl.instances)
    state = wl.instances.copy()
    for k in range(wl.cfg.n_rounds):
        req = W.make_round_requests(wl, k)
        got = gpu_route(gs, pool, req, alpha, accumulate=True)
        gs.advance_state(pool)
        t32 = oracle.instance_table(wl.types, state, alpha, "f32")
        ref = oracle.route(t32, *req.columns(), threads=8)
        assert_route_matches_f32_oracle(got, ref)
        if k % 16 == 0:
            check_route_against_f64(got, oracle.instance_table(wl.types, state, alpha, "f64"), req)
        oracle.advance(state, t32, ref.instance_idx, req.prompt_len, req.pred_decode_len)
        for dev_col, host_col in zip((pool.queued_prefill_tokens, pool.decode_batch, pool.free_kv_tokens),
                                     (state.queued_prefill_tokens, state.decode_batch, state.free_kv_tokens)):
            np.testing.assert_array_equal(dev_col.cpu().numpy(), host_col, err_msg=f"round {k}")
        np.testing.assert_array_equal(pool.q_ema_ms.cpu().numpy().view(np.uint32),
                                      state.q_ema_ms.view(np.uint32), err_msg=f"round {k}")
        if k % 8 == 7:
            risk, _ = gpu_risk(gs, pool, wl.active)
            t32n = oracle.instance_table(wl.types, state, alpha, "f32")
            rref = oracle.risk(t32n, *wl.active.columns(), threads=8)
            bits, cand, count = oracle.compact(rref.flag)
            np.testing.assert_array_equal(risk.flag_bits, bits)
            np.testing.assert_array_equal(risk.cand_idx, cand)
            assert risk.count == count
    assert gs.device_status() == 0


def test_runs_are_deterministic(gs):
    wl = W.make_workload(2, n_requests=300_000, n_active=1_000_000)
    pool = pool_of(gs, wl.types, wl.instances)
    a = gpu_route(gs, pool, wl.requests, 0.5)
    b = gpu_route(gs, pool, wl.requests, 0.5)
    for u, v in ((a.instance_idx, b.instance_idx), (a.est_e2e_ms, b.est_e2e_ms), (a.tier, b.tier)):
        assert u.tobytes() == v.tobytes()
    ra, _ = gpu_risk(gs, pool, wl.active)
    rb, _ = gpu_risk(gs, pool, wl.active)
    assert ra.flag_bits.tobytes() == rb.flag_bits.tobytes() and ra.cand_idx.tobytes() == rb.cand_idx.tobytes()


# --------------------------------------------------------------------------------------
# edge sizes
# --------------------------------------------------------------------------------------

@pytest.mark.parametrize("M", [1, 2, 3, 31, 32, 33, 127, 1023, 1024])
@pytest.mark.parametrize("N", [1, 3, 4, 5, 31, 32, 33, 1000, 4099])
def test_ragged_sizes(gs, M, N):
    types, inst = W.make_pool(M, min(M, 8), seed=100 + M)
    cfg = W.CONFIGS[3]
    req = W.make_requests(cfg, types, seed=7 * M + N, n=N)
    act = W.make_active(cfg, types, M, seed=11 * M + N, n=N)
    pool = pool_of(gs, types, inst)
    t32 = oracle.instance_table(types, inst, 0.25, "f32")
    assert_route_matches_f32_oracle(gpu_route(gs, pool, req, 0.25), oracle.route(t32, *req.columns()))
    risk, _ = gpu_risk(gs, pool, act)
    bits, cand, count = oracle.compact(oracle.risk(t32, *act.columns()).flag)
    np.testing.assert_array_equal(risk.flag_bits, bits)
    np.testing.assert_array_equal(risk.cand_idx, cand)
    assert risk.count == count


def test_empty_inputs(gs):
    types, inst = W.make_pool(16, 4, seed=1)
    pool = pool_of(gs, types, inst)
    e_i = torch.empty(0, dtype=torch.int32, device=gs.device)
    e_f = torch.empty(0, dtype=torch.float32, device=gs.device)
    gs.route_batch(e_i, e_i, e_f, pool, 0.5, e_i, e_f, e_f)
    count = torch.full((1,), -1, dtype=torch.int64, device=gs.device)
    gs.risk_scan(e_i, e_i, e_i, e_f, e_f, pool, e_i, None, count, cand_capacity=0)
    assert int(count.item()) == 0 and gs.device_status() == 0


def test_all_tiers_and_boundaries(gs):
    """The hand-worked pool: every tier, KV exactly enough, deadline exactly met."""
    from test_oracle_pins import fixture_pool, read_rows
    for name, D, k0, k1, k2, g, est, slack, tier in read_rows("handworked_routing.txt"):
        types, inst = fixture_pool((int(k0), int(k1), int(k2)))
        pool = pool_of(gs, types, inst)
        req = W.RequestBatch(np.array([1000], np.int32), np.array([200], np.int32), np.array([float(D)], np.float32))
        got = gpu_route(gs, pool, req, 0.5)
        assert got.instance_idx[0] == int(g) and got.tier[0] == int(tier), name
        assert got.est_e2e_ms[0] == pytest.approx(float(est), rel=REL_TOL), name
    types, inst = fixture_pool()
    pool = pool_of(gs, types, inst)
    for name, pred, gen, elapsed, slo, finish, flag in read_rows("handworked_risk.txt"):
        act = W.ActiveSet(np.array([1], np.int32), np.array([int(gen)], np.int32), np.array([int(pred)], np.int32),
                          np.array([float(elapsed)], np.float32), np.array([float(slo)], np.float32))
        risk, _ = gpu_risk(gs, pool, act)
        assert risk.count == int(flag), name


def test_extreme_values(gs):
    """Huge token counts (L_in + L_out above 2^31), infinite / NaN / negative deadlines."""
    types, inst = W.make_pool(64, 4, seed=3)
    inst.free_kv_tokens[:8] = 2 ** 31 - 1
    pool = pool_of(gs, types, inst)
    x = np.array([2 ** 31 - 1, 2 ** 30, 16, 16, 16, 2 ** 31 - 1, 0, 5], np.int32)
    y = np.array([2 ** 31 - 1, 2 ** 30, 8, 8, 8, 0, 0, 7], np.int32)
    D = np.array([1e30, np.inf, np.nan, -1.0, 0.0, 1e12, 1.0, np.inf], np.float32)
    req = W.RequestBatch(x, y, D)
    t32 = oracle.instance_table(types, inst, 0.5, "f32")
    got = gpu_route(gs, pool, req, 0.5)
    ref = oracle.route(t32, x, y, D)
    np.testing.assert_array_equal(got.instance_idx, ref.instance_idx)
    np.testing.assert_array_equal(got.tier, ref.tier)
    np.testing.assert_array_equal(got.est_e2e_ms.view(np.uint32), ref.est_e2e_ms.view(np.uint32))
    assert {1, 2, 3} <= set(got.tier.tolist())
    assert gs.device_status() == 0


def test_invalid_data_sets_status_bits(gs):
    from paper_2605_16867_b200 import DeviceStatus
    types, inst = W.make_pool(32, 4, seed=5)
    inst.type_id[3] = 99
    inst.decode_batch[4] = -2
    inst.q_ema_ms[5] = np.nan
    pool = pool_of(gs, types, inst)
    cfg = W.CONFIGS[1]
    req = W.make_requests(cfg, types, seed=1, n=500)
    req.prompt_len[17] = -40
    t32 = oracle.instance_table(types, inst, 0.5, "f32")
    got = gpu_route(gs, pool, req, 0.5)
    assert_route_matches_f32_oracle(got, oracle.route(t32, *req.columns()))
    st = gs.device_status()
    assert st & DeviceStatus.BAD_TYPE and st & DeviceStatus.BAD_VALUE
    act = W.make_active(cfg, types, 32, seed=2, n=700)
    act.assigned_inst[5] = 32
    act.assigned_inst[6] = -1
    act.generated_tokens[7] = -3
    risk, _ = gpu_risk(gs, pool, act)
    rref = oracle.risk(t32, *act.columns())
    np.testing.assert_array_equal(unpack_bits(risk.flag_bits, act.n), rref.flag)
    st = gs.device_status()
    assert st & DeviceStatus.BAD_INSTANCE and st & DeviceStatus.BAD_VALUE
    assert gs.device_status() == 0         # reading clears


def test_candidate_buffer_too_small(gs):
    from paper_2605_16867_b200 import DeviceStatus
    wl = W.make_workload(1, n_requests=16, n_active=50_000)
    pool = pool_of(gs, wl.types, wl.instances)
    t32 = oracle.instance_table(wl.types, wl.instances, 0.5, "f32")
    flag = oracle.risk(t32, *wl.active.columns()).flag
    _, cand, count = oracle.compact(flag)
    cap = count // 3
    risk, raw = gpu_risk(gs, pool, wl.active, capacity=cap)
    assert risk.count == count                      # the true count is still reported
    np.testing.assert_array_equal(raw[:cap], cand[:cap])
    assert gs.device_status() & DeviceStatus.CAND_TRUNCATED
    # and nothing is written past the capacity
    dev = gs.device
    cols = [torch.from_numpy(c).to(dev) for c in wl.active.columns()]
    bits = torch.zeros((wl.active.n + 31) // 32, dtype=torch.int32, device=dev)
    buf = torch.full((cap + 64,), -9, dtype=torch.int32, device=dev)
    cnt = torch.zeros(1, dtype=torch.int64, device=dev)
    gs.risk_scan(*cols, pool, bits, buf, cnt, cand_capacity=cap)
    torch.cuda.synchronize()
    assert (buf[cap:].cpu().numpy() == -9).all()
    gs.device_status()


def test_accumulate_and_advance_saturate(gs):
    types, inst = W.make_pool(4, 2, seed=9)
    inst.free_kv_tokens[:] = 2 ** 31 - 1
    inst.queued_prefill_tokens[:] = 5
    pool = pool_of(gs, types, inst)
    n = 64
    req = W.RequestBatch(np.full(n, 2 ** 30, np.int32), np.full(n, 100, np.int32), np.full(n, np.inf, np.float32))
    t32 = oracle.instance_table(types, inst, 0.5, "f32")
    got = gpu_route(gs, pool, req, 0.5, accumulate=True)
    gs.advance_state(pool)
    ref = oracle.route(t32, *req.columns())
    np.testing.assert_array_equal(got.instance_idx, ref.instance_idx)
    state = inst.copy()
    oracle.advance(state, t32, ref.instance_idx, req.prompt_len, req.pred_decode_len)
    assert state.queued_prefill_tokens.max() == 2 ** 31 - 1 and state.free_kv_tokens.min() == 0
    np.testing.assert_array_equal(pool.queued_prefill_tokens.cpu().numpy(), state.queued_prefill_tokens)
    np.testing.assert_array_equal(pool.decode_batch.cpu().numpy(), state.decode_batch)
    np.testing.assert_array_equal(pool.free_kv_tokens.cpu().numpy(), state.free_kv_tokens)
    # a second advance with nothing pending changes only nothing
    gs.advance_state(pool)
    np.testing.assert_array_equal(pool.decode_batch.cpu().numpy(), state.decode_batch)


def test_accumulate_with_the_most_types(gs):
    """Sixteen GPU types make the route kernel's tables as large as they get; with the
    per-instance sums of the accumulate variant beside them the CTA's shared memory is at its
    fullest.  Decisions and the advanced state must still be the oracle's."""
    rng = np.random.default_rng(16)
    types, inst = _random_pool(rng, 1024, 16)
    pool = pool_of(gs, types, inst)
    t32 = oracle.instance_table(types, inst, 0.5, "f32")
    req = _boundary_requests(rng, t32, 9000)
    got = gpu_route(gs, pool, req, 0.5, accumulate=True)
    gs.advance_state(pool)
    ref = oracle.route(t32, *req.columns(), threads=4)
    assert_route_matches_f32_oracle(got, ref)
    state = inst.copy()
    oracle.advance(state, t32, ref.instance_idx, req.prompt_len, req.pred_decode_len)
    np.testing.assert_array_equal(pool.queued_prefill_tokens.cpu().numpy(), state.queued_prefill_tokens)
    np.testing.assert_array_equal(pool.decode_batch.cpu().numpy(), state.decode_batch)
    np.testing.assert_array_equal(pool.free_kv_tokens.cpu().numpy(), state.free_kv_tokens)
    assert gs.device_status() == 0


def test_route_without_accumulate_leaves_state_alone(gs):
    wl = W.make_workload(1, n_requests=4096, n_active=16)
    pool = pool_of(gs, wl.types, wl.instances)
    gpu_route(gs, pool, wl.requests, 0.5)
    gs.advance_state(pool)
    np.testing.assert_array_equal(pool.queued_prefill_tokens.cpu().numpy(), wl.instances.queued_prefill_tokens)
    np.testing.assert_array_equal(pool.decode_batch.cpu().numpy(), wl.instances.decode_batch)


def test_advance_carries_the_queue_delay_of_the_accumulate_round_only(gs):
    """gs_advance_state writes back q_g of the latest ACCUMULATE round.  Routing calls that do not
    accumulate (another alpha, another pool) between that round and the advance must not change
    what is carried, and an advance with no round pending leaves q_ema alone."""
    import torch
    wl = W.make_workload(1, n_requests=3000, n_active=16)
    pool = pool_of(gs, wl.types, wl.instances)
    q0 = pool.q_ema_ms.cpu().numpy().copy()
    gs.advance_state(pool)                                     # nothing pending
    np.testing.assert_array_equal(pool.q_ema_ms.cpu().numpy().view(np.uint32), q0.view(np.uint32))
    gpu_route(gs, pool, wl.requests, 0.25)                     # no accumulate: nothing to carry
    gs.advance_state(pool)
    np.testing.assert_array_equal(pool.q_ema_ms.cpu().numpy().view(np.uint32), q0.view(np.uint32))
    t32 = oracle.instance_table(wl.types, wl.instances, 0.5, "f32")
    got = gpu_route(gs, pool, wl.requests, 0.5, accumulate=True)
    # other rounds in between: a plain one with another alpha, and one against a smaller pool
    gpu_route(gs, pool, wl.requests, 0.9)
    other = W.make_workload(0, n_requests=64, n_active=16)
    gpu_route(gs, pool_of(gs, other.types, other.instances), other.requests, 0.1)
    gs.advance_state(pool)
    torch.cuda.synchronize()
    ref = oracle.route(t32, *wl.requests.columns())
    assert_route_matches_f32_oracle(got, ref)
    state = wl.instances.copy()
    oracle.advance(state, t32, ref.instance_idx, wl.requests.prompt_len, wl.requests.pred_decode_len)
    np.testing.assert_array_equal(pool.q_ema_ms.cpu().numpy().view(np.uint32), state.q_ema_ms.view(np.uint32))
    np.testing.assert_array_equal(pool.decode_batch.cpu().numpy(), state.decode_batch)
    assert gs.device_status() == 0


@pytest.mark.parametrize("n_req,n_act", [(20_001, 70_003), (700_001, 1_000_003)])
def test_host_entry_points_match_device_ones(gs, n_req, n_act):
    """The host-buffer entry points work through their input in pieces (copies in, kernels and
    copies out overlap); the larger size spans several pieces with a ragged last one.  Results
    must equal the device entry points' bit for bit, also with a candidate buffer that ends
    inside a piece."""
    wl = W.make_workload(1, n_requests=n_req, n_active=n_act)
    pool = pool_of(gs, wl.types, wl.instances)
    dev = gpu_route(gs, pool, wl.requests, 0.5)
    n = wl.requests.n
    idx = np.empty(n, np.int32); est = np.empty(n, np.float32); slack = np.empty(n, np.float32)
    tier = np.empty(n, np.uint8)
    gs.route_batch_host(*wl.requests.columns(), wl.types, wl.instances, 0.5, idx, est, slack, tier)
    np.testing.assert_array_equal(idx, dev.instance_idx)
    np.testing.assert_array_equal(est, dev.est_e2e_ms)
    np.testing.assert_array_equal(slack, dev.slack_ms)
    np.testing.assert_array_equal(tier, dev.tier)
    risk, _ = gpu_risk(gs, pool, wl.active)
    bits = np.empty((wl.active.n + 31) // 32, np.uint32)
    cand = np.empty(wl.active.n, np.int32)
    count = gs.risk_scan_host(*wl.active.columns(), wl.types, wl.instances, bits, cand)
    assert count == risk.count
    np.testing.assert_array_equal(bits, risk.flag_bits)
    np.testing.assert_array_equal(cand[:count], risk.cand_idx)
    assert gs.device_status() == 0
    # a candidate buffer that holds two thirds of the list: the true count, the list's head
    small = np.full(2 * count // 3, -5, np.int32)
    count2 = gs.risk_scan_host(*wl.active.columns(), wl.types, wl.instances, bits, small)
    assert count2 == risk.count
    np.testing.assert_array_equal(small, risk.cand_idx[:small.size])
    assert gs.device_status() == 16                              # GS_DEV_CAND_TRUNCATED


def test_deferred_host_routing_overlaps_the_scan_and_changes_nothing(gs):
    """gs_route_batch_host_deferred returns once its work is enqueued; the scan's host call that
    follows sends its inputs while the round's results come back.  Pinned buffers (the copies are
    then really asynchronous); twice in a row, so that the second round meets the first one's
    buffers; the results are the blocking calls', and the oracle's."""
    wl = W.make_workload(2, n_requests=600_001, n_active=900_003)
    t32 = oracle.instance_table(wl.types, wl.instances, 0.5, "f32")
    ref = oracle.route(t32, *wl.requests.columns(), threads=8)
    flags = oracle.risk(t32, *wl.active.columns(), threads=8).flag
    rbits, rcand, rcount = oracle.compact(flags)
    pin = lambda a: torch.from_numpy(a).pin_memory()            # noqa: E731
    req = [pin(c) for c in wl.requests.columns()]
    act = [pin(c) for c in wl.active.columns()]
    n, a = wl.requests.n, wl.active.n
    for rep in range(2):
        idx = torch.full((n,), -7, dtype=torch.int32).pin_memory()
        est = torch.zeros(n, dtype=torch.float32).pin_memory()
        slack = torch.zeros(n, dtype=torch.float32).pin_memory()
        tier = torch.zeros(n, dtype=torch.uint8).pin_memory()
        bits = torch.zeros((a + 31) // 32, dtype=torch.int32).pin_memory()
        cand = torch.zeros(a, dtype=torch.int32).pin_memory()
        gs.route_batch_host(*req, wl.types, wl.instances, 0.5, idx, est, slack, tier, wait=False)
        if rep == 1:       # a second deferred round right behind the first
            gs.route_batch_host(*req, wl.types, wl.instances, 0.5, idx, est, slack, tier, wait=False)
        count = gs.risk_scan_host(*act, wl.types, wl.instances, bits, cand)
        gs.host_wait()
        got = GpuRoute(idx.numpy(), est.numpy(), slack.numpy(), tier.numpy())
        assert_route_matches_f32_oracle(got, ref)
        assert count == rcount
        np.testing.assert_array_equal(bits.numpy().view(np.uint32), rbits)
        np.testing.assert_array_equal(cand.numpy()[:count], rcand)
    assert gs.device_status() == 0


def test_work_counters_of_the_counting_build(gs):
    """The measuring build (-DGS_COUNT_EVALS) runs the same kernels with its counters on: its
    answers are still the oracle's, every request is scored exactly at least once, far fewer
    pairs are scored than the N x M the definition names, and the regular build counts nothing."""
    from paper_2605_16867_b200 import GoodServe
    wl = W.make_workload(1, n_requests=30_000, n_active=16)
    t32 = oracle.instance_table(wl.types, wl.instances, wl.ema_alpha, "f32")
    ref = oracle.route(t32, *wl.requests.columns())
    counting = GoodServe(0, counting=True)
    try:
        counting.eval_counters(clear=True)
        got = gpu_route(counting, pool_of(counting, wl.types, wl.instances), wl.requests, wl.ema_alpha)
        assert_route_matches_f32_oracle(got, ref)
        c = counting.eval_counters(clear=True)
        n, M = wl.requests.n, wl.instances.n_instances
        assert n <= c[0] < n * M // 4                      # pairs scored exactly
        assert c[1] >= c[0] and c[2] >= n                  # row bounds, type bounds
        assert 0 <= c[3] < n and c[4] <= c[3]              # left to the full search, of which fallback
        assert counting.eval_counters() == [0] * 8         # cleared
    finally:
        counting.close()
    gpu_route(gs, pool_of(gs, wl.types, wl.instances), wl.requests, wl.ema_alpha)
    assert gs.eval_counters() == [0] * 8


def test_error_codes(gs):
    from paper_2605_16867_b200 import GoodServe, GoodServeError, InstancePool
    types, inst = W.make_pool(16, 4, seed=1)
    pool = pool_of(gs, types, inst)
    dev = gs.device
    n = 64
    xi = torch.zeros(n + 4, dtype=torch.int32, device=dev)
    xf = torch.zeros(n + 4, dtype=torch.float32, device=dev)
    with pytest.raises(GoodServeError) as e:      # misaligned view
        gs.route_batch(xi[1:n + 1], xi[:n], xf[:n], pool, 0.5, xi[:n].clone(), xf[:n].clone(), xf[:n].clone())
    assert e.value.code == -4
    small = GoodServe(0, max_instances=8, max_types=2)
    with pytest.raises(GoodServeError) as e:      # pool larger than the context
        small.route_batch(xi[:n], xi[:n], xf[:n], pool, 0.5, xi[:n].clone(), xf[:n].clone(), xf[:n].clone())
    assert e.value.code == -2
    small.close()
    with pytest.raises(GoodServeError) as e:
        GoodServe(0, max_instances=4096)
    assert e.value.code == -2
    with pytest.raises((TypeError, ValueError)):  # wrong dtype is caught by the binding
        gs.route_batch(xf[:n], xi[:n], xf[:n], pool, 0.5, xi[:n].clone(), xf[:n].clone(), xf[:n].clone())
    # the context is still usable
    cfg = W.CONFIGS[0]
    req = W.make_requests(cfg, types, seed=0, n=100)
    t32 = oracle.instance_table(types, inst, 0.5, "f32")
    assert_route_matches_f32_oracle(gpu_route(gs, pool, req, 0.5), oracle.route(t32, *req.columns()))


# --------------------------------------------------------------------------------------
# adversarial pools for the pruned search: the result must stay exactly the definition's
# --------------------------------------------------------------------------------------

def _canonical_T(tab32, x, y):
    """T(r, g) for all (r, g) in the kernels' single-precision operation order (a product of
    two floats is exact in double, so rounding the double sum once gives the fused result)."""
    t1 = (np.outer(x.astype(np.float64), tab32.p.astype(np.float64)) + tab32.q.astype(np.float64)).astype(np.float32)
    return (np.outer(y.astype(np.float64), tab32.d.astype(np.float64)) + t1.astype(np.float64)).astype(np.float32)


def _random_pool(rng, M, Tn, scale_p=1.0, scale_d=1.0, equal_batches=False, zero_queue=False, scarce_kv=False):
    types = W.TypeTable((rng.uniform(0.01, 0.2, Tn) * scale_p).astype(np.float32),
                        (rng.uniform(4, 50, Tn) * scale_d).astype(np.float32),
                        (rng.uniform(0.02, 0.3, Tn) * scale_d).astype(np.float32))
    type_id = rng.integers(0, Tn, M).astype(np.int32)
    queued = (np.zeros(M) if zero_queue else rng.integers(0, 20001, M)).astype(np.int32)
    batch = (np.full(M, 7) if equal_batches else rng.integers(0, 65, M)).astype(np.int32)
    kv = (rng.integers(0, 3000, M) if scarce_kv else rng.integers(0, 200001, M)).astype(np.int32)
    q_ema = (queued * types.prefill_ms_per_tok[type_id] * rng.uniform(0.8, 1.2, M)).astype(np.float32)
    return types, W.InstanceState(type_id, queued, batch, kv, q_ema)


def _boundary_requests(rng, tab32, n):
    """Requests whose deadline sits exactly on, one ulp below and one ulp above the estimate
    of some instance, mixed with loose and hopeless ones."""
    x = np.clip(np.rint(np.exp(rng.normal(6.5, 1.0, n))), 1, 1 << 20).astype(np.int32)
    y = np.clip(np.rint(np.exp(rng.normal(5.0, 1.5, n))), 1, 1 << 20).astype(np.int32)
    y[rng.random(n) < 0.02] = 0
    x[rng.random(n) < 0.02] = 0
    T = _canonical_T(tab32, x, y)
    g = rng.integers(0, T.shape[1], n)
    D = T[np.arange(n), g].copy()
    kind = rng.integers(0, 6, n)
    D = np.where(kind == 1, np.nextafter(D, np.float32(-np.inf)), D)
    D = np.where(kind == 2, np.nextafter(D, np.float32(np.inf)), D)
    D = np.where(kind == 3, D * rng.uniform(0.3, 3.0, n).astype(np.float32), D)
    D = np.where(kind == 4, T.min(axis=1) * np.float32(0.999), D)
    D = np.where(kind == 5, T.max(axis=1) * np.float32(1.001), D)
    return W.RequestBatch(x, y, D.astype(np.float32))


FUZZ_CASES = [
    dict(M=1024, Tn=1), dict(M=1024, Tn=16), dict(M=1000, Tn=3), dict(M=513, Tn=8, scarce_kv=True),
    dict(M=300, Tn=16, equal_batches=True), dict(M=128, Tn=1, equal_batches=True, zero_queue=True),
    dict(M=64, Tn=2, zero_queue=True), dict(M=17, Tn=1), dict(M=16, Tn=1), dict(M=40, Tn=5, scarce_kv=True),
    dict(M=777, Tn=7, scale_p=1e-6, scale_d=1e-5), dict(M=777, Tn=7, scale_p=1e4, scale_d=1e3),
    dict(M=1024, Tn=8, scale_d=1e-3), dict(M=257, Tn=4, scale_p=0.0),
]


@pytest.mark.parametrize("case", range(len(FUZZ_CASES)))
def test_pruned_search_is_exact_on_adversarial_pools(gs, case):
    rng = np.random.default_rng(1000 + case)
    types, inst = _random_pool(rng, **FUZZ_CASES[case])
    pool = pool_of(gs, types, inst)
    for alpha in (0.0, 0.5):
        t32 = oracle.instance_table(types, inst, alpha, "f32")
        req = _boundary_requests(rng, t32, 6000)
        got = gpu_route(gs, pool, req, alpha)
        ref = oracle.route(t32, *req.columns(), threads=4)
        assert_route_matches_f32_oracle(got, ref)
    assert gs.device_status() == 0


RECORD_LIST_CASES = [
    dict(M=1024, Tn=8),                    # the benchmark's shape: every type gets a share of the pool
    dict(M=1024, Tn=1),                    # one type of 1,024 rows: long lists, the pool runs out at some bucket
    dict(M=1024, Tn=2, scarce_kv=True),    # picks that lack KV room leave the lists' promise
    dict(M=600, Tn=3, zero_queue=True),    # equal q: a type's records collapse to its first row
    dict(M=96, Tn=16),                     # six rows a type: lists shorter than the window
]


@pytest.mark.parametrize("case", range(len(RECORD_LIST_CASES)))
def test_record_lists_at_bucket_edges_and_row_deadlines(gs, case):
    """The first attempt of the route kernel looks at a few entries of a per-type, per-bucket
    list of rows; what it cannot prove goes to the full search.  L_out on, just below and just
    above every bucket edge (powers of two and 1.5 times them, up to beyond the last bucket),
    deadlines exactly on, one ulp below and one ulp above the estimate of every instance of a
    request's row, so that each list entry is the pick of some request and each of its
    neighbours is refused by one ulp."""
    rng = np.random.default_rng(7000 + case)
    types, inst = _random_pool(rng, **RECORD_LIST_CASES[case])
    pool = pool_of(gs, types, inst)
    t32 = oracle.instance_table(types, inst, 0.5, "f32")
    M = inst.n_instances
    edges = []
    for e in range(0, 19):
        for base in (1 << e, 3 << e >> 1):
            edges += [base - 1, base, base + 1]
    y_vals = np.array(sorted({v for v in edges if v >= 1}), np.int32)
    reps = -(-3 * M // len(y_vals))                     # every instance gets on/below/above deadlines
    y = np.tile(y_vals, reps * 8)[: 24 * M]
    n = y.size
    x = np.clip(np.rint(np.exp(rng.normal(6.0, 1.5, n))), 0, 1 << 18).astype(np.int32)
    T = _canonical_T(t32, x, y)
    g = np.arange(n) % M
    D = T[np.arange(n), g].copy()
    kind = (np.arange(n) // M) % 3
    D = np.where(kind == 1, np.nextafter(D, np.float32(-np.inf)), D)
    D = np.where(kind == 2, np.nextafter(D, np.float32(np.inf)), D)
    req = W.RequestBatch(x, y.astype(np.int32), D.astype(np.float32))
    got = gpu_route(gs, pool, req, 0.5)
    ref = oracle.route(t32, *req.columns(), threads=4)
    assert_route_matches_f32_oracle(got, ref)
    assert gs.device_status() == 0


@pytest.mark.parametrize("variant", ["plain", "accumulate", "prefix", "direct"])
def test_large_batches_take_the_wide_kernel(gs, variant):
    """From 2,097,152 requests on, the route kernel reads four requests per lane with 128-bit
    loads (below: one per lane).  Every variant of it runs here on a batch just over that size,
    ragged at the end, with a tenth of the deadlines out of reach so that the queue and the
    fallback see traffic too."""
    n = (1 << 21) + 37
    wl = W.make_workload(3, n_requests=n, n_active=1024)
    req = wl.requests
    rng = np.random.default_rng(99)
    hopeless = rng.random(n) < 0.1
    req = W.RequestBatch(req.prompt_len, req.pred_decode_len,
                         np.where(hopeless, req.slo_ms * np.float32(0.3), req.slo_ms).astype(np.float32))
    t32 = oracle.instance_table(wl.types, wl.instances, wl.ema_alpha, "f32")
    if variant == "direct":
        bb = W.make_blackbox_table(wl.types, wl.instances, seed=3)
        t32 = oracle.direct_table(*bb.columns(), "f32")
        got = gpu_route_direct(gs, bb, req)
        ref = oracle.route(t32, *req.columns(), threads=8)
    elif variant == "prefix":
        pool = pool_of(gs, wl.types, wl.instances)
        pi, ph = W.make_prefix_hits(req, t32.n_instances, seed=3, n_slots=2)
        got = gpu_route_prefix(gs, pool, req, wl.ema_alpha, pi, ph)
        ref = oracle.route_prefix(t32, *req.columns(), pi, ph, threads=8)
    else:
        pool = pool_of(gs, wl.types, wl.instances)
        got = gpu_route(gs, pool, req, wl.ema_alpha, accumulate=variant == "accumulate")
        ref = oracle.route(t32, *req.columns(), threads=8)
        if variant == "accumulate":
            gs.advance_state(pool)
            state = wl.instances.copy()
            oracle.advance(state, t32, ref.instance_idx, req.prompt_len, req.pred_decode_len)
            np.testing.assert_array_equal(pool.queued_prefill_tokens.cpu().numpy(), state.queued_prefill_tokens)
            np.testing.assert_array_equal(pool.decode_batch.cpu().numpy(), state.decode_batch)
            np.testing.assert_array_equal(pool.free_kv_tokens.cpu().numpy(), state.free_kv_tokens)
    assert_route_matches_f32_oracle(got, ref)
    assert (ref.tier >= 2).mean() > 0.05
    assert gs.device_status() == 0


@pytest.mark.parametrize("share", [1.0, 0.3, 0.01])
@pytest.mark.parametrize("scarce_kv", [False, True])
def test_fallback_heavy_and_sparse_batches(gs, share, scarce_kv):
    """Batches in which all, many or only a few requests have no feasible instance: the
    fallback's minimum of T (with and without KV room) is the definition's whichever way the
    kernel chooses to compute it, ties to the smallest index."""
    rng = np.random.default_rng(4242)
    types, inst = _random_pool(rng, 1024, 8, scarce_kv=scarce_kv)
    inst.queued_prefill_tokens[::3] = 0            # groups of instances with equal estimates
    inst.q_ema_ms[::3] = 0.0
    inst.decode_batch[::3] = 5
    pool = pool_of(gs, types, inst)
    t32 = oracle.instance_table(types, inst, 0.5, "f32")
    n = 20000
    x = np.clip(np.rint(np.exp(rng.normal(6.5, 1.0, n))), 1, 1 << 18).astype(np.int32)
    y = np.clip(np.rint(np.exp(rng.normal(5.0, 1.5, n))), 1, 1 << 18).astype(np.int32)
    T = _canonical_T(t32, x, y)
    hopeless = rng.random(n) < share
    D = np.where(hopeless, T.min(axis=1) * np.float32(0.9), T.max(axis=1) * np.float32(1.1)).astype(np.float32)
    req = W.RequestBatch(x, y, D)
    got = gpu_route(gs, pool, req, 0.5)
    ref = oracle.route(t32, *req.columns(), threads=4)
    assert_route_matches_f32_oracle(got, ref)
    assert (ref.tier[hopeless] >= 2).all() and (3 in set(ref.tier.tolist())) == scarce_kv


def test_coefficients_the_bounds_cannot_use_take_the_exhaustive_path(gs):
    """A negative type constant makes lower bounds meaningless; the kernel then scores every
    instance for every request and still returns the definition's answer."""
    from paper_2605_16867_b200 import DeviceStatus
    rng = np.random.default_rng(77)
    types, inst = _random_pool(rng, 200, 4)
    types.tpot_a_ms[1] = -3.0
    pool = pool_of(gs, types, inst)
    t32 = oracle.instance_table(types, inst, 0.5, "f32")
    cfg = W.CONFIGS[1]
    req = W.make_requests(cfg, types, seed=3, n=5000)
    req.slo_ms[:] = np.abs(req.slo_ms)
    got = gpu_route(gs, pool, req, 0.5)
    ref = oracle.route(t32, *req.columns())
    np.testing.assert_array_equal(got.instance_idx, ref.instance_idx)
    np.testing.assert_array_equal(got.tier, ref.tier)
    assert gs.device_status() & DeviceStatus.BAD_VALUE


# --------------------------------------------------------------------------------------
# re-routing of the scan's candidates (Sec. 3.4)
# --------------------------------------------------------------------------------------

def gpu_scan_and_reroute(gs, pool, act, prompt, alpha):
    dev = gs.device
    cols = [torch.from_numpy(c).to(dev) for c in act.columns()]
    x = torch.from_numpy(prompt).to(dev)
    n = act.n
    bits = torch.zeros(max((n + 31) // 32, 1), dtype=torch.int32, device=dev)
    cand = torch.full((max(n, 1),), -9, dtype=torch.int32, device=dev)
    count = torch.zeros(1, dtype=torch.int64, device=dev)
    gs.risk_scan(*cols, pool, bits, cand, count)
    new_inst = torch.full((max(n, 1),), -7, dtype=torch.int32, device=dev)
    est = torch.full((max(n, 1),), float("nan"), dtype=torch.float32, device=dev)
    slack = torch.full((max(n, 1),), float("nan"), dtype=torch.float32, device=dev)
    tier = torch.full((max(n, 1),), 9, dtype=torch.uint8, device=dev)
    gs.reroute_candidates(cand, count, *cols, x, pool, alpha, new_inst, est, slack, tier)
    torch.cuda.synchronize(dev)
    c = int(count.item())
    return (cand.cpu().numpy()[:c], new_inst.cpu().numpy(), est.cpu().numpy(), slack.cpu().numpy(),
            tier.cpu().numpy(), c)


def check_reroute(gs, types, inst, act, prompt, alpha=0.5):
    pool = pool_of(gs, types, inst)
    t32 = oracle.instance_table(types, inst, alpha, "f32")
    t64 = oracle.instance_table(types, inst, alpha, "f64")
    cand, new_inst, est, slack, tier, c = gpu_scan_and_reroute(gs, pool, act, prompt, alpha)
    ref_cand = np.nonzero(oracle.risk(t32, *act.columns(), threads=8).flag)[0].astype(np.int32)
    np.testing.assert_array_equal(cand, ref_cand)
    ref = oracle.reroute(t32, ref_cand, *act.columns(), prompt)
    np.testing.assert_array_equal(new_inst[:c], ref.new_instance)
    np.testing.assert_array_equal(tier[:c], ref.tier)
    np.testing.assert_array_equal(est[:c].view(np.uint32), ref.est_ms.view(np.uint32))
    np.testing.assert_array_equal(slack[:c].view(np.uint32), ref.slack_ms.view(np.uint32))
    assert (new_inst[c:] == -7).all() and (tier[c:] == 9).all()       # nothing past the count is touched
    ref64 = oracle.reroute(t64, ref_cand, *act.columns(), prompt)
    agree = ref64.new_instance == ref.new_instance
    same = agree & (ref.tier > 0)
    err = np.abs(est[:c][same] - ref64.est_ms[same]) / np.maximum(np.abs(ref64.est_ms[same]), 1e-30)
    assert err.size == 0 or err.max() <= REL_TOL
    assert agree.size == 0 or agree.mean() > 0.999       # the two precisions part only at near-ties
    return ref


@pytest.mark.parametrize("cfg_id", [0, 1, 2])
def test_reroute_full_size(gs, cfg_id):
    wl = W.make_workload(cfg_id)
    prompt = W.make_requests(wl.cfg, wl.types, seed=500 + cfg_id, n=wl.active.n).prompt_len
    ref = check_reroute(gs, wl.types, wl.instances, wl.active, prompt)
    print(f"cfg {cfg_id}: {len(ref.tier)} candidates, tiers 0..3 = {[int((ref.tier == k).sum()) for k in range(4)]}")
    assert gs.device_status() == 0


def test_reroute_config3_sample(gs):
    """Largest pool (1,024 instances of 8 types) on 2,097,152 active requests."""
    wl = W.make_workload(3, n_requests=16, n_active=2_097_152)
    prompt = W.make_requests(wl.cfg, wl.types, seed=503, n=wl.active.n).prompt_len
    ref = check_reroute(gs, wl.types, wl.instances, wl.active, prompt)
    assert {0, 1, 2} <= set(ref.tier.tolist())


def test_reroute_handworked(gs):
    from test_oracle_pins import fixture_pool, read_rows
    for name, cur, elapsed, slo, k0, k1, g, est, slack, tier in read_rows("handworked_reroute.txt"):
        types, inst = fixture_pool((int(k0), int(k1), 100000))
        act = W.ActiveSet(np.array([int(cur)], np.int32), np.array([50], np.int32), np.array([200], np.int32),
                          np.array([float(elapsed)], np.float32), np.array([float(slo)], np.float32))
        pool = pool_of(gs, types, inst)
        cand, new_inst, e, s, t, c = gpu_scan_and_reroute(gs, pool, act, np.array([1000], np.int32), 0.5)
        if c == 0:          # the request is not at risk where it runs: nothing to re-route
            continue
        assert new_inst[0] == int(g) and t[0] == int(tier), name
        assert e[0] == pytest.approx(float(est), rel=REL_TOL), name


@pytest.mark.parametrize("case", [0, 3, 4, 7, 8, 10])
def test_reroute_on_adversarial_pools(gs, case):
    rng = np.random.default_rng(2000 + case)
    types, inst = _random_pool(rng, **FUZZ_CASES[case])
    cfg = W.CONFIGS[3]
    act = W.make_active(cfg, types, inst.n_instances, seed=case, n=20_000)
    act.generated_tokens[::7] = 0
    act.generated_tokens[1::11] = act.pred_len[1::11]            # nothing left to decode
    prompt = np.clip(np.rint(np.exp(rng.normal(6.5, 1.2, act.n))), 0, 1 << 20).astype(np.int32)
    check_reroute(gs, types, inst, act, prompt, alpha=0.25)
    assert gs.device_status() == 0


def gpu_reroute_listed(gs, pool, act, prompt, alpha, cand_idx):
    """Re-routes the listed active requests (a caller-made list: the scan is not involved)."""
    dev = gs.device
    cols = [torch.from_numpy(c).to(dev) for c in act.columns()]
    x = torch.from_numpy(prompt).to(dev)
    c = len(cand_idx)
    cand = torch.from_numpy(np.ascontiguousarray(cand_idx, np.int32)).to(dev)
    count = torch.tensor([c], dtype=torch.int64, device=dev)
    new_inst = torch.full((c + 3,), -7, dtype=torch.int32, device=dev)
    est = torch.full((c + 3,), float("nan"), dtype=torch.float32, device=dev)
    slack = torch.full((c + 3,), float("nan"), dtype=torch.float32, device=dev)
    tier = torch.full((c + 3,), 9, dtype=torch.uint8, device=dev)
    gs.reroute_candidates(cand, count, *cols, x, pool, alpha, new_inst, est, slack, tier, cand_capacity=c)
    torch.cuda.synchronize(dev)
    assert (new_inst[c:] == -7).all() and (tier[c:] == 9).all()
    return new_inst.cpu().numpy()[:c], est.cpu().numpy()[:c], slack.cpu().numpy()[:c], tier.cpu().numpy()[:c]


def assert_reroute_matches(got, ref):
    new_inst, est, slack, tier = got
    np.testing.assert_array_equal(new_inst, ref.new_instance)
    np.testing.assert_array_equal(tier, ref.tier)
    np.testing.assert_array_equal(est.view(np.uint32), ref.est_ms.view(np.uint32))
    np.testing.assert_array_equal(slack.view(np.uint32), ref.slack_ms.view(np.uint32))


@pytest.mark.parametrize("case", [0, 2, 3, 5, 8, 10])
def test_reroute_of_requests_that_are_not_at_risk(gs, case):
    """The candidate list is the caller's: requests with time to spare, whose unrestricted pick is
    often an instance no faster than the current one, must still be held to faster instances."""
    rng = np.random.default_rng(2100 + case)
    types, inst = _random_pool(rng, **FUZZ_CASES[case])
    act = W.make_active(W.CONFIGS[3], types, inst.n_instances, seed=40 + case, n=30_000)
    act.slo_ms[:] = act.elapsed_ms + np.exp(rng.uniform(np.log(5.0), np.log(4.0e5), act.n)).astype(np.float32)
    act.generated_tokens[::13] = act.pred_len[::13]              # nothing left to decode
    prompt = np.clip(np.rint(np.exp(rng.normal(6.0, 1.5, act.n))), 0, 1 << 20).astype(np.int32)
    cand = np.sort(rng.choice(act.n, size=act.n * 3 // 4, replace=False)).astype(np.int32)
    pool = pool_of(gs, types, inst)
    t32 = oracle.instance_table(types, inst, 0.25, "f32")
    ref = oracle.reroute(t32, cand, *act.columns(), prompt)
    assert_reroute_matches(gpu_reroute_listed(gs, pool, act, prompt, 0.25, cand), ref)
    if case == 5:                  # identical instances: nothing is strictly faster, nobody moves
        assert (ref.tier == 0).all() and (ref.new_instance == -1).all()
    else:
        assert (ref.tier == 1).any() and (ref.tier != 1).any()
    cur_d = t32.d[act.assigned_inst[cand]]
    assert (t32.d[ref.new_instance[ref.tier > 0]] < cur_d[ref.tier > 0]).all()   # only strictly faster instances
    assert gs.device_status() == 0


@pytest.mark.parametrize("case", [0, 4, 7, 9])
def test_reroute_with_time_left_on_instance_estimates(gs, case):
    """Time left equal to, one ulp below and one ulp above the exact T of some instance for the
    re-posed request: the feasibility tests and every bound before them sit on their edge."""
    rng = np.random.default_rng(2200 + case)
    types, inst = _random_pool(rng, **FUZZ_CASES[case])
    t32 = oracle.instance_table(types, inst, 0.5, "f32")
    n = 24_000
    act = W.make_active(W.CONFIGS[3], types, inst.n_instances, seed=60 + case, n=n)
    prompt = np.clip(np.rint(np.exp(rng.normal(6.0, 1.0, n))), 1, 1 << 18).astype(np.int32)
    x = (prompt.astype(np.int64) + act.generated_tokens).astype(np.float32)
    y = np.maximum(act.pred_len - act.generated_tokens, 0).astype(np.float32)
    target = rng.integers(0, inst.n_instances, n)
    t1 = (x.astype(np.float64) * t32.p[target].astype(np.float64) + t32.q[target].astype(np.float64)).astype(np.float32)
    T = (y.astype(np.float64) * t32.d[target].astype(np.float64) + t1.astype(np.float64)).astype(np.float32)   # see _canonical_T
    step = rng.integers(-1, 2, n)
    T = np.where(step < 0, np.nextafter(T, np.float32(-np.inf)), np.where(step > 0, np.nextafter(T, np.float32(np.inf)), T))
    act.elapsed_ms[:] = 0.0                                      # time left = slo, bit for bit
    act.slo_ms[:] = T.astype(np.float32)
    cand = np.arange(n, dtype=np.int32)
    pool = pool_of(gs, types, inst)
    ref = oracle.reroute(t32, cand, *act.columns(), prompt)
    assert_reroute_matches(gpu_reroute_listed(gs, pool, act, prompt, 0.5, cand), ref)
    assert gs.device_status() == 0


def test_reroute_invalid_data_and_unusable_coefficients(gs):
    """Bad entries in the active columns are read as the oracle reads them (status bits); a pool
    whose coefficients the bounds cannot take (an infinite decode time) is still served exactly,
    every candidate scored against every instance."""
    from paper_2605_16867_b200 import DeviceStatus
    rng = np.random.default_rng(31)
    types, inst = _random_pool(rng, 300, 5)
    act = W.make_active(W.CONFIGS[3], types, inst.n_instances, seed=77, n=6000)
    act.pred_len[:] = np.maximum(act.pred_len, act.generated_tokens + 1)      # something left to decode everywhere
    prompt = np.clip(np.rint(np.exp(rng.normal(6.0, 1.0, act.n))), 1, 1 << 18).astype(np.int32)
    act.assigned_inst[5] = inst.n_instances; act.assigned_inst[6] = -1
    act.generated_tokens[7] = -3; prompt[9] = -20
    cand = np.arange(act.n, dtype=np.int32)
    for unusable in (False, True):
        if unusable:
            types.tpot_a_ms[2] = np.inf
        pool = pool_of(gs, types, inst)
        t32 = oracle.instance_table(types, inst, 0.5, "f32")
        ref = oracle.reroute(t32, cand, *act.columns(), prompt)
        assert_reroute_matches(gpu_reroute_listed(gs, pool, act, prompt, 0.5, cand), ref)
        st = gs.device_status()
        assert st & DeviceStatus.BAD_INSTANCE and st & DeviceStatus.BAD_VALUE
        assert ref.status & DeviceStatus.BAD_INSTANCE and ref.status & DeviceStatus.BAD_VALUE


# --------------------------------------------------------------------------------------
# routing with the prefix-cache term of Eq. 2
# --------------------------------------------------------------------------------------

@pytest.mark.parametrize("cfg_id,n_slots", [(0, 1), (1, 1), (1, 3), (2, 2)])
def test_prefix_config_full_size(gs, cfg_id, n_slots):
    wl = W.make_workload(cfg_id)
    pool = pool_of(gs, wl.types, wl.instances)
    t32 = oracle.instance_table(wl.types, wl.instances, wl.ema_alpha, "f32")
    pi, ph = W.make_prefix_hits(wl.requests, t32.n_instances, seed=cfg_id, n_slots=n_slots)
    got = gpu_route_prefix(gs, pool, wl.requests, wl.ema_alpha, pi, ph)
    ref = oracle.route_prefix(t32, *wl.requests.columns(), pi, ph, threads=8)
    assert_route_matches_f32_oracle(got, ref)
    plain = oracle.route(t32, *wl.requests.columns(), threads=8)
    print(f"cfg {cfg_id}, {n_slots} slot(s): {int((plain.instance_idx != ref.instance_idx).sum())} of "
          f"{len(ref.tier)} answers moved by the hits")
    assert gs.device_status() == 0


def test_prefix_config3_sample(gs):
    """Full-size launch; the oracle checks a strided sample of the requests."""
    wl = W.make_workload(3)
    pool = pool_of(gs, wl.types, wl.instances)
    t32 = oracle.instance_table(wl.types, wl.instances, wl.ema_alpha, "f32")
    pi, ph = W.make_prefix_hits(wl.requests, t32.n_instances, seed=3, n_slots=1)
    got = gpu_route_prefix(gs, pool, wl.requests, wl.ema_alpha, pi, ph)
    sel = np.arange(0, wl.requests.n, 61)
    x, y, D = (c[sel] for c in wl.requests.columns())
    ref = oracle.route_prefix(t32, x, y, D, pi[:, sel], ph[:, sel], threads=8)
    np.testing.assert_array_equal(got.instance_idx[sel], ref.instance_idx)
    np.testing.assert_array_equal(got.tier[sel], ref.tier)
    np.testing.assert_array_equal(got.est_e2e_ms[sel], ref.est_e2e_ms)


@pytest.mark.parametrize("n_slots", [0, 1, 2])
def test_prefix_without_hits_equals_plain_routing(gs, n_slots):
    wl = W.make_workload(1, n_requests=10001)
    pool = pool_of(gs, wl.types, wl.instances)
    n = wl.requests.n
    pi = np.full((n_slots, n), -1, np.int32)
    ph = np.full((n_slots, n), 50, np.int32)
    a = gpu_route_prefix(gs, pool, wl.requests, 0.5, pi, ph)
    b = gpu_route(gs, pool, wl.requests, 0.5)
    for u, v in ((a.instance_idx, b.instance_idx), (a.est_e2e_ms, b.est_e2e_ms), (a.slack_ms, b.slack_ms), (a.tier, b.tier)):
        np.testing.assert_array_equal(u, v)


def test_prefix_handworked(gs):
    from test_oracle_pins import fixture_pool, parse_slots, read_rows
    for name, x, y, D, k0, k1, k2, slots, g, est, slack, tier in read_rows("handworked_prefix.txt"):
        types, inst = fixture_pool((int(k0), int(k1), int(k2)))
        pool = pool_of(gs, types, inst)
        pi, ph = parse_slots(slots)
        req = W.RequestBatch(np.array([int(x)], np.int32), np.array([int(y)], np.int32), np.array([float(D)], np.float32))
        got = gpu_route_prefix(gs, pool, req, 0.5, pi, ph)
        assert got.instance_idx[0] == int(g) and got.tier[0] == int(tier), name
        assert got.est_e2e_ms[0] == pytest.approx(float(est), rel=1e-5), name
        assert got.slack_ms[0] == pytest.approx(float(slack), rel=1e-4, abs=2e-3), name
        gs.device_status()


@pytest.mark.parametrize("case", [0, 1, 3, 5, 9, 13])
def test_prefix_on_adversarial_pools(gs, case):
    """Boundary deadlines, equal estimates, scarce KV, slots that are empty, unknown,
    duplicated, negative or longer than the prompt; ragged batch size and padded stride."""
    from paper_2605_16867_b200 import DeviceStatus
    rng = np.random.default_rng(2000 + case)
    types, inst = _random_pool(rng, **FUZZ_CASES[case])
    pool = pool_of(gs, types, inst)
    t32 = oracle.instance_table(types, inst, 0.5, "f32")
    M = t32.n_instances
    n = 6001
    req = _boundary_requests(rng, t32, n)
    K = 3
    pi = rng.integers(-1, M + 1, (K, n)).astype(np.int32)
    pi[2] = np.where(rng.random(n) < 0.5, pi[0], pi[2])                 # duplicates
    ph = (rng.random((K, n)) * 1.2 * req.prompt_len - 2).astype(np.int32)
    # deadlines that the hit decides: just below the hit-free estimate of the first slot's instance
    g0 = np.clip(pi[0], 0, M - 1)
    T0 = _canonical_T(t32, req.prompt_len, req.pred_decode_len)[np.arange(n), g0]
    req.slo_ms[::4] = np.nextafter(T0, np.float32(-np.inf))[::4]
    got = gpu_route_prefix(gs, pool, req, 0.5, pi, ph, pad_to=n + 37 + (4 - (n + 37) % 4) % 4)
    ref = oracle.route_prefix(t32, *req.columns(), pi, ph, threads=4)
    assert_route_matches_f32_oracle(got, ref)
    assert gs.device_status() == ref.status == (DeviceStatus.BAD_VALUE | DeviceStatus.BAD_INSTANCE)


def test_prefix_error_codes(gs):
    from paper_2605_16867_b200 import GoodServeError
    wl = W.make_workload(0, n_requests=64)
    pool = pool_of(gs, wl.types, wl.instances)
    dev = gs.device
    x = torch.from_numpy(wl.requests.prompt_len).to(dev)
    y = torch.from_numpy(wl.requests.pred_decode_len).to(dev)
    D = torch.from_numpy(wl.requests.slo_ms).to(dev)
    hits = torch.zeros(9 * 64 + 4, dtype=torch.int32, device=dev)
    o_i = torch.zeros(64, dtype=torch.int32, device=dev)
    o_f = torch.zeros(64, dtype=torch.float32, device=dev)
    o_s = torch.zeros(64, dtype=torch.float32, device=dev)
    for kwargs, code in ((dict(n_slots=9, slot_stride=64), -1),        # more slots than supported
                         (dict(n_slots=-1, slot_stride=64), -1),
                         (dict(n_slots=1, slot_stride=60), -1),        # stride shorter than the batch
                         (dict(n_slots=1, slot_stride=66), -4)):       # stride not a multiple of 4
        with pytest.raises(GoodServeError) as e:
            gs.route_batch_prefix(x, y, D, hits, hits, kwargs["n_slots"], kwargs["slot_stride"], pool, 0.5, o_i, o_f, o_s)
        assert e.value.code == code, kwargs
    with pytest.raises(GoodServeError) as e:                            # misaligned hit column
        gs.route_batch_prefix(x, y, D, hits[1:], hits, 1, 64, pool, 0.5, o_i, o_f, o_s)
    assert e.value.code == -4


# --------------------------------------------------------------------------------------
# black-box coefficients: directly given tables and their EMA step (Sec. 3.3)
# --------------------------------------------------------------------------------------

@pytest.mark.parametrize("cfg_id", [0, 1, 2])
def test_direct_config_full_size(gs, cfg_id):
    wl = W.make_workload(cfg_id)
    bb = W.make_blackbox_table(wl.types, wl.instances, seed=cfg_id)
    t32 = oracle.direct_table(*bb.columns(), "f32")
    got = gpu_route_direct(gs, bb, wl.requests)
    ref = oracle.route(t32, *wl.requests.columns(), threads=8)
    assert_route_matches_f32_oracle(got, ref)
    t64 = oracle.direct_table(*bb.columns(), "f64")
    n_tie = check_route_against_f64(got, t64, wl.requests)
    print(f"cfg {cfg_id} direct: tiers={[int((got.tier == k).sum()) for k in (1, 2, 3)]} near-ties vs fp64={n_tie}")
    assert gs.device_status() == 0


def test_direct_config3_sample(gs):
    wl = W.make_workload(3)
    bb = W.make_blackbox_table(wl.types, wl.instances, seed=3)
    t32 = oracle.direct_table(*bb.columns(), "f32")
    got = gpu_route_direct(gs, bb, wl.requests)
    sel = np.arange(0, wl.requests.n, 37)
    ref = oracle.route(t32, *(c[sel] for c in wl.requests.columns()), threads=8)
    np.testing.assert_array_equal(got.instance_idx[sel], ref.instance_idx)
    np.testing.assert_array_equal(got.tier[sel], ref.tier)
    np.testing.assert_array_equal(got.est_e2e_ms[sel], ref.est_e2e_ms)


def test_direct_table_of_typed_coefficients_equals_typed_routing(gs):
    """Feeding the typed path's own coefficients through the direct interface must not change
    a single output, although the search then runs on groups of p instead of GPU types."""
    wl = W.make_workload(2, n_requests=200000)
    pool = pool_of(gs, wl.types, wl.instances)
    typed = gpu_route(gs, pool, wl.requests, wl.ema_alpha)
    t32 = oracle.instance_table(wl.types, wl.instances, wl.ema_alpha, "f32")
    bb = W.BlackBoxTable(t32.q, t32.p, t32.d, t32.kv.astype(np.int32))
    direct = gpu_route_direct(gs, bb, wl.requests)
    for u, v in ((typed.instance_idx, direct.instance_idx), (typed.est_e2e_ms, direct.est_e2e_ms),
                 (typed.slack_ms, direct.slack_ms), (typed.tier, direct.tier)):
        np.testing.assert_array_equal(u, v)


@pytest.mark.parametrize("case", range(8))
def test_direct_on_adversarial_tables(gs, case):
    """Continuous p (no two instances alike), all p equal, p spanning orders of magnitude, zeros,
    a single instance; deadlines on, one ulp below and one ulp above instance estimates."""
    rng = np.random.default_rng(3000 + case)
    M = [1024, 1000, 513, 64, 1, 17, 300, 1024][case]
    q = rng.uniform(0, 500, M)
    p = [rng.uniform(0.01, 0.2, M), np.full(M, 0.05), 10.0 ** rng.uniform(-6, 2, M), rng.uniform(0.01, 0.2, M),
         np.array([0.03]), np.zeros(M), rng.choice([0.02, 0.05, 0.11], M) * rng.uniform(0.97, 1.03, M),
         rng.uniform(0.01, 0.2, M)][case]
    d = rng.uniform(4, 60, M)
    if case == 3:
        q[:] = 0.0; d[::2] = d[0]                      # equal d: ties go to the smaller index
    if case == 7:
        d[rng.random(M) < 0.3] = 0.0; q[rng.random(M) < 0.3] = 0.0
    kv = rng.integers(0, 3000 if case in (2, 6) else 200001, M)
    bb = W.BlackBoxTable(q.astype(np.float32), p.astype(np.float32), d.astype(np.float32), kv.astype(np.int32))
    t32 = oracle.direct_table(*bb.columns(), "f32")
    req = _boundary_requests(rng, t32, 6000)
    got = gpu_route_direct(gs, bb, req)
    ref = oracle.route(t32, *req.columns(), threads=4)
    assert_route_matches_f32_oracle(got, ref)
    assert gs.device_status() == 0


def test_direct_invalid_coefficients(gs):
    from paper_2605_16867_b200 import DeviceStatus
    rng = np.random.default_rng(9)
    M = 200
    q = rng.uniform(0, 500, M).astype(np.float32); p = rng.uniform(0.01, 0.2, M).astype(np.float32)
    d = rng.uniform(4, 60, M).astype(np.float32); kv = rng.integers(0, 200001, M).astype(np.int32)
    q[3] = -1.0; p[5] = np.nan; d[7] = -2.0; kv[9] = -5
    bb = W.BlackBoxTable(q, p, d, kv)
    t32 = oracle.direct_table(*bb.columns(), "f32")
    req = W.make_requests(W.CONFIGS[1], W.make_types(3, 0, perturb=False), seed=5, n=5000)
    got = gpu_route_direct(gs, bb, req)
    ref = oracle.route(t32, *req.columns())
    assert_route_matches_f32_oracle(got, ref)
    assert gs.device_status() == t32.status == DeviceStatus.BAD_VALUE
    d[11] = np.inf                                     # bounds unusable: exhaustive path, still exact
    bb = W.BlackBoxTable(q, p, d, kv)
    t32 = oracle.direct_table(*bb.columns(), "f32")
    got = gpu_route_direct(gs, bb, req)
    ref = oracle.route(t32, *req.columns())
    np.testing.assert_array_equal(got.instance_idx, ref.instance_idx)
    np.testing.assert_array_equal(got.tier, ref.tier)
    assert gs.device_status() & DeviceStatus.BAD_VALUE


def test_ema_update_matches_oracle(gs):
    from paper_2605_16867_b200 import DeviceStatus, GoodServeError
    wl = W.make_workload(3, n_requests=8, n_active=8)
    bb = W.make_blackbox_table(wl.types, wl.instances, seed=3)
    dev = gs.device
    M = bb.n_instances
    state = [torch.from_numpy(c.copy()).to(dev) for c in (bb.q_ms, bb.p_ms_per_tok, bb.d_ms_per_tok)]
    want = [c.copy() for c in (bb.q_ms, bb.p_ms_per_tok, bb.d_ms_per_tok)]
    for step in range(5):
        obs = [W.make_observations(c, seed=3 + k, step=step) for k, c in enumerate((bb.q_ms, bb.p_ms_per_tok, bb.d_ms_per_tok))]
        if step == 2:
            obs[1][4] = np.nan; obs[2][6] = -1.0
        alpha = (0.3, 0.0, 0.5, 1.0, 0.125)[step]
        skip_p = step == 3                            # a column without observations stays as it is
        gs.ema_update(alpha, *(torch.from_numpy(o).to(dev) if not (skip_p and k == 1) else None for k, o in enumerate(obs)), *state)
        st = 0
        for k in range(3):
            if skip_p and k == 1:
                continue
            want[k], s_k = oracle.ema_update(alpha, obs[k], want[k], "f32")
            st |= s_k
        for k in range(3):
            np.testing.assert_array_equal(state[k].cpu().numpy(), want[k])
        assert gs.device_status() == st == (DeviceStatus.BAD_VALUE if step == 2 else 0)
    # the smoothed table routes like the oracle's
    bb2 = W.BlackBoxTable(want[0], want[1], want[2], bb.free_kv_tokens)
    req = W.make_requests(wl.cfg, wl.types, seed=3, n=20000)
    got = gpu_route_direct(gs, bb2, req)
    ref = oracle.route(oracle.direct_table(*bb2.columns(), "f32"), *req.columns(), threads=4)
    assert_route_matches_f32_oracle(got, ref)
    with pytest.raises(GoodServeError) as e:          # observations without a state column
        gs.ema_update(0.5, state[0], None, None, None, None, None)
    assert e.value.code == -1


# --------------------------------------------------------------------------------------
# Algorithm 1 one request at a time
# --------------------------------------------------------------------------------------

def gpu_sequential(gs, types, inst, req, alpha):
    pool = pool_of(gs, types, inst)
    dev = gs.device
    n = req.n
    x = torch.from_numpy(req.prompt_len).to(dev)
    y = torch.from_numpy(req.pred_decode_len).to(dev)
    D = torch.from_numpy(req.slo_ms).to(dev)
    idx = torch.full((max(n, 1),), -7, dtype=torch.int32, device=dev)
    est = torch.zeros(max(n, 1), dtype=torch.float32, device=dev)
    slack = torch.zeros(max(n, 1), dtype=torch.float32, device=dev)
    tier = torch.zeros(max(n, 1), dtype=torch.uint8, device=dev)
    gs.route_sequential(x, y, D, pool, alpha, idx, est, slack, tier, n_requests=n)
    torch.cuda.synchronize(dev)
    state = W.InstanceState(pool.type_id.cpu().numpy(), pool.queued_prefill_tokens.cpu().numpy(),
                            pool.decode_batch.cpu().numpy(), pool.free_kv_tokens.cpu().numpy(),
                            pool.q_ema_ms.cpu().numpy())
    return (idx.cpu().numpy()[:n], est.cpu().numpy()[:n], slack.cpu().numpy()[:n], tier.cpu().numpy()[:n]), state


def assert_sequential_matches(got, state, ref, ref_state):
    for u, v in zip(got, (ref.instance_idx, ref.est_e2e_ms, ref.slack_ms, ref.tier)):
        np.testing.assert_array_equal(u, v)
    for u, v in zip(state.columns(), ref_state.columns()):
        np.testing.assert_array_equal(u, v)


@pytest.mark.parametrize("cfg_id,n", [(0, 256), (1, 65536), (2, 150000), (3, 100000)])
def test_sequential_configs(gs, cfg_id, n):
    wl = W.make_workload(cfg_id, n_requests=n)
    req = wl.requests
    req.slo_ms[::7] *= 0.3                                   # some requests fall back
    ref_state = wl.instances.copy()
    ref = oracle.route_sequential(wl.types, ref_state, wl.ema_alpha, *req.columns())
    got, state = gpu_sequential(gs, wl.types, wl.instances, req, wl.ema_alpha)
    assert_sequential_matches(got, state, ref, ref_state)
    snap = oracle.route(oracle.instance_table(wl.types, wl.instances, wl.ema_alpha, "f32"), *req.columns(), threads=8)
    print(f"cfg {cfg_id}: {n} requests one at a time, tiers={[int((ref.tier == k).sum()) for k in (1, 2, 3)]}; "
          f"busiest instance takes {np.bincount(ref.instance_idx).max()} (snapshot round: {np.bincount(snap.instance_idx).max()})")
    assert gs.device_status() == 0


@pytest.mark.parametrize("M", [1, 31, 33, 1000])
@pytest.mark.parametrize("n", [0, 1, 255, 257, 3000])
def test_sequential_ragged_sizes(gs, M, n):
    rng = np.random.default_rng(M * 7 + n)
    types, inst = _random_pool(rng, M, 3, scarce_kv=(M == 33))
    t32 = oracle.instance_table(types, inst, 0.5, "f32")
    req = _boundary_requests(rng, t32, max(n, 1))
    req = W.RequestBatch(req.prompt_len[:n], req.pred_decode_len[:n], req.slo_ms[:n])
    ref_state = inst.copy()
    ref = oracle.route_sequential(types, ref_state, 0.5, *req.columns())
    got, state = gpu_sequential(gs, types, inst, req, 0.5)
    assert_sequential_matches(got, state, ref, ref_state)
    assert gs.device_status() == 0


def test_sequential_equals_rounds_of_one_request_on_the_gpu(gs):
    """What the header promises: n rounds of gs_route_batch(ACCUMULATE) + gs_advance_state with
    one request each give the same assignments and the same final state."""
    wl = W.make_workload(1, n_requests=200)
    req = wl.requests
    got, state = gpu_sequential(gs, wl.types, wl.instances, req, 0.5)
    pool = pool_of(gs, wl.types, wl.instances)
    dev = gs.device
    x = torch.from_numpy(req.prompt_len).to(dev); y = torch.from_numpy(req.pred_decode_len).to(dev)
    D = torch.from_numpy(req.slo_ms).to(dev)
    idx = torch.zeros(req.n, dtype=torch.int32, device=dev)
    est = torch.zeros(req.n, dtype=torch.float32, device=dev)
    slack = torch.zeros(req.n, dtype=torch.float32, device=dev)
    for r in range(req.n):
        one_i = torch.zeros(4, dtype=torch.int32, device=dev); one_e = torch.zeros(4, device=dev); one_s = torch.zeros(4, device=dev)
        gs.route_batch(x[r:r + 1].clone(), y[r:r + 1].clone(), D[r:r + 1].clone(), pool, 0.5, one_i, one_e, one_s,
                       None, accumulate=True, n_requests=1)
        gs.advance_state(pool)
        idx[r] = one_i[0]; est[r] = one_e[0]
    torch.cuda.synchronize(dev)
    np.testing.assert_array_equal(idx.cpu().numpy(), got[0])
    np.testing.assert_array_equal(est.cpu().numpy(), got[1])
    np.testing.assert_array_equal(pool.queued_prefill_tokens.cpu().numpy(), state.queued_prefill_tokens)
    np.testing.assert_array_equal(pool.q_ema_ms.cpu().numpy(), state.q_ema_ms)


def test_sequential_invalid_data(gs):
    from paper_2605_16867_b200 import DeviceStatus
    rng = np.random.default_rng(12)
    types, inst = _random_pool(rng, 100, 3)
    inst.type_id[3] = 9; inst.queued_prefill_tokens[5] = -4; inst.q_ema_ms[7] = np.nan; inst.free_kv_tokens[9] = -1
    t32 = oracle.instance_table(types, inst, 0.5, "f32")
    req = _boundary_requests(rng, t32, 500)
    req.prompt_len[11] = -3
    ref_state = inst.copy()
    ref = oracle.route_sequential(types, ref_state, 0.5, *req.columns())
    got, state = gpu_sequential(gs, types, inst, req, 0.5)
    assert_sequential_matches(got, state, ref, ref_state)
    assert gs.device_status() == ref.status == (DeviceStatus.BAD_TYPE | DeviceStatus.BAD_VALUE)
