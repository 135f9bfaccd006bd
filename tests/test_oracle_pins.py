"""Pins for the CPU oracle: everything here checks the oracle against something other than
itself -- hand-worked fixtures, a declarative restatement of Algorithm 1's post-condition
evaluated on exhaustive tiny grids, textbook special cases (numpy argmax/argmin/bincount),
closed forms and invariants.  No GPU."""
import itertools
import os

import numpy as np
import pytest

import oracle
import workloads as W

GOLD = os.path.join(os.path.dirname(__file__), "golden")
PRECS = ("f64", "f32")


# --------------------------------------------------------------------------------------
# helpers
# --------------------------------------------------------------------------------------

def base_types():
    return W.make_types(3, seed=0, perturb=False)


def fixture_pool(kv=(100000, 100000, 100000)):
    types = base_types()
    type_id = np.array([0, 1, 2], np.int32)
    queued = np.array([4000, 2000, 1000], np.int32)
    batch = np.array([20, 10, 10], np.int32)
    q_ema = (queued.astype(np.float64) * types.prefill_ms_per_tok[type_id]).astype(np.float32)
    inst = W.InstanceState(type_id, queued, batch, np.array(kv, np.int32), q_ema)
    return types, inst


def read_rows(name):
    rows = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


def latency_all_instances(q, p, d, x, y, prec):
    """T(r, .) of Eq. 2 for one request.  In single precision each fused step rounds once;
    a product of two floats is exact in double, so rounding the double sum gives that."""
    if prec == "f64":
        return q + p * float(x) + d * float(y)
    t1 = (p.astype(np.float64) * float(x) + q).astype(np.float32)
    return (d.astype(np.float64) * float(y) + t1).astype(np.float32).astype(np.float64)


def check_postcondition(q, p, d, kv, x, y, D, idx, tier, prec="f64"):
    """Declarative statement of what Algorithm 1 (with the adopted tie/KV readings) must
    return, written as set conditions instead of a scan."""
    q, p, d = (np.asarray(a, np.float64) for a in (q, p, d))
    kv = np.asarray(kv, np.int64)
    for r in range(len(x)):
        T = latency_all_instances(q, p, d, x[r], y[r], prec)
        ok = (int(x[r]) + int(y[r])) <= kv
        feas = ok & (T <= float(D[r]))
        g = int(idx[r])
        if feas.any():
            assert tier[r] == 1
            assert feas[g]
            better = feas & ((d > d[g]) | ((d == d[g]) & (np.arange(len(d)) < g)))
            assert not better.any()
        else:
            pool = ok if ok.any() else np.ones_like(ok)
            assert tier[r] == (2 if ok.any() else 3)
            assert pool[g]
            better = pool & ((T < T[g]) | ((T == T[g]) & (np.arange(len(d)) < g)))
            assert not better.any()


# --------------------------------------------------------------------------------------
# hand-worked fixtures
# --------------------------------------------------------------------------------------

@pytest.mark.parametrize("prec", PRECS)
@pytest.mark.parametrize("alpha", [0.0, 0.3, 0.5, 1.0])
def test_handworked_routing(prec, alpha):
    for name, D, k0, k1, k2, g, est, slack, tier in read_rows("handworked_routing.txt"):
        types, inst = fixture_pool((int(k0), int(k1), int(k2)))
        tab = oracle.instance_table(types, inst, alpha, prec)
        np.testing.assert_allclose(tab.q, [100, 100, 100], rtol=1e-6, err_msg=name)
        np.testing.assert_allclose(tab.d, [9.0, 14.8, 26.5], rtol=1e-6, err_msg=name)
        res = oracle.route(tab, [1000], [200], [float(D)])
        assert res.instance_idx[0] == int(g), name
        assert res.tier[0] == int(tier), name
        assert res.est_e2e_ms[0] == pytest.approx(float(est), rel=1e-5), name
        assert res.slack_ms[0] == pytest.approx(float(slack), rel=1e-4, abs=2e-3), name


@pytest.mark.parametrize("prec", PRECS)
def test_handworked_risk(prec):
    types, inst = fixture_pool()
    tab = oracle.instance_table(types, inst, 0.5, prec)
    for name, pred, gen, elapsed, slo, finish, flag in read_rows("handworked_risk.txt"):
        res = oracle.risk(tab, [1], [int(gen)], [int(pred)], [float(elapsed)], [float(slo)])
        assert res.finish_ms[0] == pytest.approx(float(finish), rel=1e-6), name
        assert res.flag[0] == int(flag), name


# --------------------------------------------------------------------------------------
# closed form of Eq. 2 and of the instance coefficients
# --------------------------------------------------------------------------------------

@pytest.mark.parametrize("prec", PRECS)
def test_eq2_closed_form_and_linearity(prec):
    wl = W.make_workload(1, n_requests=64, n_active=8)
    tab = oracle.instance_table(wl.types, wl.instances, 0.5, prec)
    # a single-instance pool makes route() return T(r,g) itself
    for g in (0, 17, 63):
        one = oracle.InstanceTable(tab.q[g:g + 1], tab.p[g:g + 1], tab.d[g:g + 1],
                                   tab.kv[g:g + 1], 0, prec)
        x = np.array([0, 1, 0, 1000, 2000, 1000], np.int32)
        y = np.array([0, 0, 1, 200, 200, 400], np.int32)
        T = oracle.route(one, x, y, np.zeros(6, np.float32)).est_e2e_ms.astype(np.float64)
        q, p, d = float(tab.q[g]), float(tab.p[g]), float(tab.d[g])
        rel = 1e-12 if prec == "f64" else 1e-6
        assert T[0] == pytest.approx(q, rel=rel)                      # intercept
        assert T[1] - T[0] == pytest.approx(p, rel=1e-3, abs=1e-4)    # one more prompt token
        assert T[2] - T[0] == pytest.approx(d, rel=1e-3, abs=1e-4)    # one more output token
        assert T[3] == pytest.approx(q + 1000 * p + 200 * d, rel=rel)
        assert T[4] - T[3] == pytest.approx(1000 * p, rel=1e-4)       # linear in L_in
        assert T[5] - T[3] == pytest.approx(200 * d, rel=1e-4)        # linear in L_out


@pytest.mark.parametrize("prec", PRECS)
def test_instance_coefficients(prec):
    types, inst = fixture_pool()
    inst.q_ema_ms[:] = [10.0, 20.0, 30.0]
    w = np.array([100.0, 100.0, 100.0])
    for alpha in (0.0, 0.25, 1.0):
        tab = oracle.instance_table(types, inst, alpha, prec)
        np.testing.assert_allclose(tab.q, alpha * w + (1 - alpha) * inst.q_ema_ms, rtol=1e-6)
        np.testing.assert_allclose(tab.p, [0.025, 0.05, 0.1], rtol=1e-6)
        assert list(tab.kv) == [100000] * 3
    # alpha = 1 forgets the state, alpha = 0 keeps it
    assert np.allclose(oracle.instance_table(types, inst, 1.0, prec).q, w, rtol=1e-6)
    assert np.allclose(oracle.instance_table(types, inst, 0.0, prec).q, inst.q_ema_ms, rtol=1e-6)


def test_invalid_data_is_clamped_and_reported():
    types, inst = fixture_pool()
    inst.type_id[1] = 7
    inst.decode_batch[0] = -5
    inst.q_ema_ms[2] = np.nan
    tab = oracle.instance_table(types, inst, 0.5, "f64")
    assert tab.status & oracle.BAD_TYPE and tab.status & oracle.BAD_VALUE
    assert tab.d[0] == pytest.approx(8.0)             # batch read as 0
    assert tab.p[1] == pytest.approx(0.025)           # type read as 0
    assert tab.q[2] == pytest.approx(0.5 * 100.0)     # q_ema read as 0
    res = oracle.route(tab, [-3], [10], [1e9])
    assert res.status & oracle.BAD_VALUE
    rk = oracle.risk(tab, [99, -1], [0, 0], [10, 10], [0.0, 0.0], [1e9, 1e9])
    assert rk.status & oracle.BAD_INSTANCE
    assert rk.finish_ms[0] == pytest.approx(10 * tab.d[2]) and rk.finish_ms[1] == pytest.approx(10 * tab.d[0])
    # NaN deadline: nothing is feasible, the request falls back to the fastest instance
    res = oracle.route(tab, [1000], [200], [np.nan])
    assert res.tier[0] == 2 and res.instance_idx[0] == int(np.argmin(tab.q + 1000 * tab.p + 200 * tab.d))


# --------------------------------------------------------------------------------------
# Algorithm 1's post-condition on exhaustive tiny grids (brute force)
# --------------------------------------------------------------------------------------

@pytest.mark.parametrize("prec", PRECS)
def test_postcondition_exhaustive_tiny(prec):
    types = base_types()
    p_t = types.prefill_ms_per_tok
    n_cases = 0
    for M in (1, 2, 3, 4):
        for tids in itertools.product(range(3), repeat=M):
            if M == 4 and tids[0] != 0:
                continue                                   # keep the run short
            for code in range(2 ** M):                     # per instance: (batch, queue) pattern
                batch = np.array([(code >> g) & 1 for g in range(M)], np.int32)
                queued = np.array([20000 * ((code >> ((g + 1) % M)) & 1) for g in range(M)], np.int32)
                kvs = np.array([0, 300, 100000, 100000][:M], np.int32)
                tid = np.array(tids, np.int32)
                q_ema = (queued * p_t[tid]).astype(np.float32)
                inst = W.InstanceState(tid, queued, batch, kvs, q_ema)
                tab = oracle.instance_table(types, inst, 0.5, prec)
                x0, y0 = 200, 50
                T = tab.q.astype(np.float64) + tab.p * x0 + tab.d * y0
                # deadlines on, just below and just above every T value, plus extremes
                Ds = np.concatenate([T, T * (1 - 1e-3), T * (1 + 1e-3), [0.0, 1e9]]).astype(np.float32)
                x = np.full(len(Ds), x0, np.int32)
                y = np.full(len(Ds), y0, np.int32)
                x[-1], y[-1] = 400, 50                      # need 450 > kv 300 on g1
                res = oracle.route(tab, x, y, Ds)
                check_postcondition(tab.q, tab.p, tab.d, tab.kv, x, y, Ds, res.instance_idx, res.tier, prec)
                n_cases += len(Ds)
    assert n_cases > 5000


@pytest.mark.parametrize("prec", PRECS)
@pytest.mark.parametrize("cfg_id", [0, 1])
def test_postcondition_on_workload_sample(prec, cfg_id):
    wl = W.make_workload(cfg_id, n_requests=256, n_active=8)
    tab = oracle.instance_table(wl.types, wl.instances, wl.ema_alpha, prec)
    r = wl.requests
    res = oracle.route(tab, *r.columns())
    check_postcondition(tab.q, tab.p, tab.d, tab.kv, r.prompt_len, r.pred_decode_len, r.slo_ms,
                        res.instance_idx, res.tier, prec)
    assert set(np.unique(res.tier)) <= {1, 2, 3}


# --------------------------------------------------------------------------------------
# special cases that reduce to library routines
# --------------------------------------------------------------------------------------

@pytest.mark.parametrize("prec", PRECS)
def test_infinite_deadline_picks_slowest_with_room(prec):
    wl = W.make_workload(2, n_requests=512, n_active=8)
    tab = oracle.instance_table(wl.types, wl.instances, 0.5, prec)
    r = wl.requests
    res = oracle.route(tab, r.prompt_len, r.pred_decode_len, np.full(r.n, np.inf, np.float32))
    need = r.prompt_len.astype(np.int64) + r.pred_decode_len
    for i in range(r.n):
        ok = need[i] <= tab.kv
        assert ok.any()
        expect = int(np.argmax(np.where(ok, tab.d, -np.inf)))     # first max = smallest index
        assert res.instance_idx[i] == expect and res.tier[i] == 1


@pytest.mark.parametrize("prec", PRECS)
def test_zero_deadline_is_min_latency_router(prec):
    wl = W.make_workload(2, n_requests=512, n_active=8)
    tab = oracle.instance_table(wl.types, wl.instances, 0.5, prec)
    r = wl.requests
    res = oracle.route(tab, r.prompt_len, r.pred_decode_len, np.zeros(r.n, np.float32))
    need = r.prompt_len.astype(np.int64) + r.pred_decode_len
    real = np.float64 if prec == "f64" else np.float32
    for i in range(r.n):
        x, y = real(r.prompt_len[i]), real(r.pred_decode_len[i])
        if prec == "f64":
            T = tab.q + tab.p * x + tab.d * y
        else:   # products of two floats are exact in double; one rounding per fused step
            t1 = (tab.p.astype(np.float64) * np.float64(x) + tab.q).astype(np.float32)
            T = (tab.d.astype(np.float64) * np.float64(y) + t1).astype(np.float32)
        ok = need[i] <= tab.kv
        expect = int(np.argmin(np.where(ok, T, np.inf)))
        assert res.instance_idx[i] == expect and res.tier[i] == 2
        assert res.est_e2e_ms[i] == T[expect]
        assert res.slack_ms[i] == -T[expect]


@pytest.mark.parametrize("prec", PRECS)
def test_single_type_equal_batches_first_short_queue(prec):
    """One type, equal batches: p and d are common, so the feasible set is a threshold on q
    and the just-enough pick is the first (smallest-index) instance whose queue fits."""
    types = W.TypeTable(np.array([0.05], np.float32), np.array([14.0], np.float32),
                        np.array([0.08], np.float32))
    M = 16
    rng = np.random.default_rng(5)
    queued = rng.integers(0, 20000, M).astype(np.int32)
    inst = W.InstanceState(np.zeros(M, np.int32), queued, np.full(M, 10, np.int32),
                           np.full(M, 10 ** 6, np.int32), (queued * 0.05).astype(np.float32))
    tab = oracle.instance_table(types, inst, 0.5, prec)
    x, y = 500, 100
    const = 500 * float(tab.p[0]) + 100 * float(tab.d[0])
    for D in np.linspace(const - 10, const + 1100, 57):
        res = oracle.route(tab, [x], [y], [D])
        fits = np.nonzero(tab.q.astype(np.float64) <= np.float32(D) - const - 1e-3)[0]
        tight = np.nonzero(np.abs(tab.q.astype(np.float64) - (np.float32(D) - const)) <= 1e-3)[0]
        if len(tight):
            continue                       # rounding decides; skip the knife edge
        if len(fits):
            assert res.tier[0] == 1 and res.instance_idx[0] == fits[0]
        else:
            assert res.tier[0] == 2 and res.instance_idx[0] == int(np.argmin(tab.q))


# --------------------------------------------------------------------------------------
# invariants
# --------------------------------------------------------------------------------------

@pytest.mark.parametrize("prec", PRECS)
def test_invariants_on_tight_workload(prec):
    wl = W.make_workload(3, n_requests=2048, n_active=8)
    tab = oracle.instance_table(wl.types, wl.instances, 0.5, prec)
    r = wl.requests
    res = oracle.route(tab, *r.columns())
    need = r.prompt_len.astype(np.int64) + r.pred_decode_len
    x = r.prompt_len.astype(np.float64); y = r.pred_decode_len.astype(np.float64)
    T = tab.q[None, :] + np.outer(x, tab.p) + np.outer(y, tab.d)
    ok = need[:, None] <= tab.kv[None, :]
    feas = ok & (T <= r.slo_ms[:, None].astype(np.float64) * (1 + (0 if prec == "f64" else 1e-6)))
    strictly = ok & (T <= r.slo_ms[:, None].astype(np.float64) * (1 - 1e-6))
    g = res.instance_idx
    rows = np.arange(r.n)
    # whenever some instance clearly meets the deadline, the chosen one meets it too
    has = strictly.any(axis=1)
    assert (res.tier[has] == 1).all()
    assert feas[rows[has], g[has]].all() and (res.slack_ms[has] >= 0).all()
    # fallback slack is the best achievable (largest) slack and is negative in tier 2
    fb = res.tier == 2
    assert fb.any() and (res.tier == 1).any()
    best = np.max(np.where(ok, r.slo_ms[:, None].astype(np.float64) - T, -np.inf), axis=1)
    np.testing.assert_allclose(res.slack_ms[fb], best[fb], rtol=1e-5, atol=1e-2)
    assert (res.slack_ms[fb] < 0).all()
    # est + slack = D
    np.testing.assert_allclose(res.est_e2e_ms + res.slack_ms, r.slo_ms, rtol=1e-5)


@pytest.mark.parametrize("prec", PRECS)
def test_chosen_capability_monotone_in_deadline(prec):
    wl = W.make_workload(1, n_requests=8, n_active=8)
    tab = oracle.instance_table(wl.types, wl.instances, 0.5, prec)
    for i in range(8):
        x, y = wl.requests.prompt_len[i], wl.requests.pred_decode_len[i]
        Ds = np.linspace(0, 6 * float(wl.requests.slo_ms[i]), 200).astype(np.float32)
        res = oracle.route(tab, np.full(200, x), np.full(200, y), Ds)
        t1 = res.tier == 1
        dsel = tab.d[res.instance_idx]
        assert (np.diff(dsel[t1]) >= 0).all()          # looser deadline -> never a faster pick
        assert (np.diff(res.tier.astype(int)) <= 0).all()


@pytest.mark.parametrize("prec", PRECS)
def test_permutation_and_degenerate_pools(prec):
    wl = W.make_workload(1, n_requests=300, n_active=8)
    tab = oracle.instance_table(wl.types, wl.instances, 0.5, prec)
    r = wl.requests
    res = oracle.route(tab, *r.columns())
    perm = np.random.default_rng(1).permutation(r.n)
    res_p = oracle.route(tab, r.prompt_len[perm], r.pred_decode_len[perm], r.slo_ms[perm])
    assert (res_p.instance_idx == res.instance_idx[perm]).all()
    assert (res_p.est_e2e_ms == res.est_e2e_ms[perm]).all()
    # relabelling instances (distinct d and distinct T almost surely) relabels the answer
    gperm = np.random.default_rng(2).permutation(tab.n_instances)
    tab_p = oracle.InstanceTable(tab.q[gperm], tab.p[gperm], tab.d[gperm], tab.kv[gperm], 0, prec)
    res_g = oracle.route(tab_p, *r.columns())
    same_d = tab.d[gperm[res_g.instance_idx]] == tab.d[res.instance_idx]
    assert same_d.all()
    np.testing.assert_array_equal(res_g.est_e2e_ms, res.est_e2e_ms)
    # one instance: always 0; identical instances: always 0
    one = oracle.InstanceTable(tab.q[:1], tab.p[:1], tab.d[:1], tab.kv[:1], 0, prec)
    assert (oracle.route(one, *r.columns()).instance_idx == 0).all()
    rep = oracle.InstanceTable(*(np.repeat(a[:1], 9) for a in (tab.q, tab.p, tab.d, tab.kv)), 0, prec)
    assert (oracle.route(rep, *r.columns()).instance_idx == 0).all()


def test_power_of_two_scaling_is_exact_in_f32():
    """Scaling every time-valued input by 2^k is exact in binary floating point, so the
    decisions are unchanged and the outputs scale exactly."""
    wl = W.make_workload(1, n_requests=512, n_active=512)
    s = np.float32(8.0)
    t2 = W.TypeTable(wl.types.prefill_ms_per_tok * s, wl.types.tpot_a_ms * s, wl.types.tpot_b_ms * s)
    i2 = wl.instances.copy(); i2.q_ema_ms *= s
    tab = oracle.instance_table(wl.types, wl.instances, 0.5, "f32")
    tab2 = oracle.instance_table(t2, i2, 0.5, "f32")
    r = wl.requests
    a = oracle.route(tab, *r.columns())
    b = oracle.route(tab2, r.prompt_len, r.pred_decode_len, r.slo_ms * s)
    np.testing.assert_array_equal(a.instance_idx, b.instance_idx)
    np.testing.assert_array_equal(a.tier, b.tier)
    np.testing.assert_array_equal(a.est_e2e_ms * s, b.est_e2e_ms)
    np.testing.assert_array_equal(a.slack_ms * s, b.slack_ms)
    act = wl.active
    ra = oracle.risk(tab, *act.columns())
    rb = oracle.risk(tab2, act.assigned_inst, act.generated_tokens, act.pred_len,
                     act.elapsed_ms * s, act.slo_ms * s)
    np.testing.assert_array_equal(ra.flag, rb.flag)


def test_f32_and_f64_agree_away_from_ties():
    wl = W.make_workload(2, n_requests=4096, n_active=4096)
    t64 = oracle.instance_table(wl.types, wl.instances, 0.5, "f64")
    t32 = oracle.instance_table(wl.types, wl.instances, 0.5, "f32")
    np.testing.assert_allclose(t32.q, t64.q, rtol=3e-7)
    np.testing.assert_allclose(t32.d, t64.d, rtol=3e-7)
    r = wl.requests
    a = oracle.route(t64, *r.columns()); b = oracle.route(t32, *r.columns())
    agree = a.instance_idx == b.instance_idx
    assert agree.mean() > 0.999
    np.testing.assert_allclose(b.est_e2e_ms[agree], a.est_e2e_ms[agree], rtol=1e-6)
    ra = oracle.risk(t64, *wl.active.columns()); rb = oracle.risk(t32, *wl.active.columns())
    assert (ra.flag == rb.flag).mean() > 0.9999


# --------------------------------------------------------------------------------------
# goodput objective (Eq. 1) on tiny inputs
# --------------------------------------------------------------------------------------

def test_single_request_attains_objective_optimum():
    """For one request Eq. 1's optimum is 1 exactly when some instance with room meets the
    deadline; the heuristic must reach indicator 1 in exactly those cases (brute force)."""
    rng = np.random.default_rng(11)
    types = base_types()
    for _ in range(300):
        M = int(rng.integers(1, 5))
        tid = rng.integers(0, 3, M).astype(np.int32)
        queued = rng.integers(0, 20000, M).astype(np.int32)
        inst = W.InstanceState(tid, queued, rng.integers(0, 64, M).astype(np.int32),
                               rng.integers(0, 3000, M).astype(np.int32),
                               (queued * types.prefill_ms_per_tok[tid]).astype(np.float32))
        tab = oracle.instance_table(types, inst, 0.5, "f64")
        x, y = int(rng.integers(16, 2000)), int(rng.integers(8, 800))
        D = np.float32(rng.uniform(500, 30000))
        T = tab.q + tab.p * x + tab.d * y
        optimum = int(any(T[g] <= D and x + y <= tab.kv[g] for g in range(M)))   # enumerate x_{r,g}
        res = oracle.route(tab, [x], [y], [D])
        g = res.instance_idx[0]
        achieved = int(T[g] <= D and x + y <= tab.kv[g])
        assert achieved == optimum


# --------------------------------------------------------------------------------------
# risk scan, compaction, state advance
# --------------------------------------------------------------------------------------

@pytest.mark.parametrize("prec", PRECS)
def test_risk_special_cases(prec):
    wl = W.make_workload(1, n_requests=8, n_active=4096)
    tab = oracle.instance_table(wl.types, wl.instances, 0.5, prec)
    a = wl.active
    # nothing left to generate: flag <=> elapsed > slo
    res = oracle.risk(tab, a.assigned_inst, a.pred_len, a.pred_len, a.elapsed_ms, a.slo_ms)
    np.testing.assert_array_equal(res.flag, (a.elapsed_ms > a.slo_ms).astype(np.uint8))
    res = oracle.risk(tab, a.assigned_inst, a.pred_len, a.pred_len, a.slo_ms * 2 + 1, a.slo_ms)
    assert res.flag.all()
    # not started: flag <=> d * y > D  (products of floats are exact in double)
    zero = np.zeros(a.n, np.int32)
    res = oracle.risk(tab, a.assigned_inst, zero, a.pred_len, np.zeros(a.n, np.float32), a.slo_ms)
    dy = tab.d[a.assigned_inst].astype(np.float64) * a.pred_len
    if prec == "f32":
        dy = dy.astype(np.float32)
    np.testing.assert_array_equal(res.flag, (dy > a.slo_ms).astype(np.uint8))
    # flags are monotone: more elapsed time never clears a flag
    base = oracle.risk(tab, *a.columns())
    later = oracle.risk(tab, a.assigned_inst, a.generated_tokens, a.pred_len, a.elapsed_ms * 1.5, a.slo_ms)
    assert (later.flag >= base.flag).all()
    assert 0 < base.flag.mean() < 1


def test_compaction_matches_numpy():
    rng = np.random.default_rng(3)
    for A in (0, 1, 31, 32, 33, 1000, 4097):
        flag = (rng.random(A) < 0.3).astype(np.uint8)
        bits, cand, count = oracle.compact(flag)
        ref = np.nonzero(flag)[0]
        np.testing.assert_array_equal(cand, ref)
        assert count == len(ref)
        unpacked = np.unpackbits(bits.view(np.uint8), bitorder="little")[:A]
        np.testing.assert_array_equal(unpacked, flag)
        _, cand_small, count_small = oracle.compact(flag, capacity=len(ref) // 2)
        assert count_small == len(ref)
        np.testing.assert_array_equal(cand_small, ref[:len(ref) // 2])


def test_advance_matches_bincount_and_saturates():
    wl = W.make_workload(1, n_requests=5000, n_active=8)
    tab = oracle.instance_table(wl.types, wl.instances, 0.5, "f32")
    r = wl.requests
    res = oracle.route(tab, *r.columns())
    before = wl.instances.copy()
    oracle.advance(wl.instances, tab, res.instance_idx, r.prompt_len, r.pred_decode_len)
    M = before.n_instances
    dq = np.bincount(res.instance_idx, weights=r.prompt_len.astype(np.float64), minlength=M).astype(np.int64)
    db = np.bincount(res.instance_idx, minlength=M)
    dk = np.bincount(res.instance_idx, weights=(r.prompt_len.astype(np.float64) + r.pred_decode_len),
                     minlength=M).astype(np.int64)
    np.testing.assert_array_equal(wl.instances.queued_prefill_tokens, before.queued_prefill_tokens + dq)
    np.testing.assert_array_equal(wl.instances.decode_batch, before.decode_batch + db)
    np.testing.assert_array_equal(wl.instances.free_kv_tokens,
                                  np.maximum(before.free_kv_tokens - dk, 0))
    np.testing.assert_array_equal(wl.instances.q_ema_ms, tab.q)
    # saturation, by hand: 3 requests of 2^30 prompt tokens onto one instance
    types, inst = fixture_pool()
    tabh = oracle.instance_table(types, inst, 0.5, "f32")
    big = np.full(3, 2 ** 30, np.int32)
    oracle.advance(inst, tabh, np.zeros(3, np.int32), big, np.full(3, 5, np.int32))
    assert inst.queued_prefill_tokens[0] == 2 ** 31 - 1
    assert inst.decode_batch[0] == 23 and inst.free_kv_tokens[0] == 0
    assert inst.queued_prefill_tokens[1] == 2000 and inst.free_kv_tokens[1] == 100000


def test_threaded_split_is_identical():
    wl = W.make_workload(1, n_requests=10007, n_active=10007)
    tab = oracle.instance_table(wl.types, wl.instances, 0.5, "f32")
    a = oracle.route(tab, *wl.requests.columns(), threads=1)
    b = oracle.route(tab, *wl.requests.columns(), threads=5)
    np.testing.assert_array_equal(a.instance_idx, b.instance_idx)
    np.testing.assert_array_equal(a.est_e2e_ms, b.est_e2e_ms)
    ra = oracle.risk(tab, *wl.active.columns(), threads=1)
    rb = oracle.risk(tab, *wl.active.columns(), threads=3)
    np.testing.assert_array_equal(ra.flag, rb.flag)


# --------------------------------------------------------------------------------------
# re-routing of flagged requests
# --------------------------------------------------------------------------------------

@pytest.mark.parametrize("prec", PRECS)
def test_handworked_reroute(prec):
    for name, cur, elapsed, slo, k0, k1, g, est, slack, tier in read_rows("handworked_reroute.txt"):
        types, inst = fixture_pool((int(k0), int(k1), 100000))
        tab = oracle.instance_table(types, inst, 0.5, prec)
        res = oracle.reroute(tab, [0], [int(cur)], [50], [200], [float(elapsed)], [float(slo)], [1000])
        assert res.new_instance[0] == int(g), name
        assert res.tier[0] == int(tier), name
        assert res.est_ms[0] == pytest.approx(float(est), rel=1e-5), name
        assert res.slack_ms[0] == pytest.approx(float(slack), rel=1e-4, abs=2e-3), name


@pytest.mark.parametrize("prec", PRECS)
def test_reroute_equals_routing_over_the_faster_instances(prec):
    """Independent pin: restricted to the strictly faster instances, re-routing IS Algorithm 1
    on the transformed request (x' = prompt + generated, y' = remaining, D' = slo - elapsed),
    so it must agree with route() run on the sub-pool of eligible instances."""
    wl = W.make_workload(1, n_requests=8, n_active=3000)
    tab = oracle.instance_table(wl.types, wl.instances, 0.5, prec)
    a = wl.active
    prompt = W.make_requests(wl.cfg, wl.types, seed=99, n=a.n).prompt_len
    flag = oracle.risk(tab, *a.columns()).flag
    cand = np.nonzero(flag)[0].astype(np.int32)
    res = oracle.reroute(tab, cand, *a.columns(), prompt)
    real = np.float64 if prec == "f64" else np.float32
    seen_tiers = set()
    for j, i in enumerate(cand[:600]):
        c = a.assigned_inst[i]
        elig = np.nonzero(tab.d < tab.d[c])[0]
        if len(elig) == 0:
            assert res.new_instance[j] == -1 and res.tier[j] == 0
            seen_tiers.add(0)
            continue
        sub = oracle.InstanceTable(tab.q[elig], tab.p[elig], tab.d[elig], tab.kv[elig], 0, prec)
        x = np.array([prompt[i] + a.generated_tokens[i]], np.int32)
        y = np.array([max(a.pred_len[i] - a.generated_tokens[i], 0)], np.int32)
        D = np.array([real(a.slo_ms[i]) - real(a.elapsed_ms[i])], np.float32)
        if prec == "f32":
            assert real(D[0]) == np.float32(a.slo_ms[i]) - np.float32(a.elapsed_ms[i])
        ref = oracle.route(sub, x, y, D)
        assert res.new_instance[j] == elig[ref.instance_idx[0]]
        assert res.tier[j] == ref.tier[0]
        if prec == "f32":
            assert res.est_ms[j] == ref.est_e2e_ms[0]
        else:
            assert res.est_ms[j] == pytest.approx(ref.est_e2e_ms[0], rel=1e-6)
        seen_tiers.add(int(res.tier[j]))
    assert {1, 2} <= seen_tiers


def test_reroute_never_moves_to_a_slower_or_equal_instance():
    wl = W.make_workload(2, n_requests=8, n_active=20000)
    tab = oracle.instance_table(wl.types, wl.instances, 0.5, "f64")
    a = wl.active
    prompt = W.make_requests(wl.cfg, wl.types, seed=5, n=a.n).prompt_len
    cand = np.nonzero(oracle.risk(tab, *a.columns()).flag)[0].astype(np.int32)
    res = oracle.reroute(tab, cand, *a.columns(), prompt)
    moved = res.new_instance >= 0
    assert moved.any()
    assert (tab.d[res.new_instance[moved]] < tab.d[a.assigned_inst[cand[moved]]]).all()
    assert (res.tier[moved] > 0).all() and (res.tier[~moved] == 0).all()
    t1 = res.tier == 1
    assert (res.slack_ms[t1] >= 0).all()


# --------------------------------------------------------------------------------------
# prefix-cache term of Eq. 2 (sparse H)
# --------------------------------------------------------------------------------------

def parse_slots(text):
    if text == "-":
        return np.zeros((0, 1), np.int32), np.zeros((0, 1), np.int32)
    pairs = [tuple(int(v) for v in item.split(":")) for item in text.split(",")]
    return (np.array([[g] for g, _ in pairs], np.int32), np.array([[h] for _, h in pairs], np.int32))


@pytest.mark.parametrize("prec", PRECS)
def test_handworked_prefix(prec):
    for name, x, y, D, k0, k1, k2, slots, g, est, slack, tier in read_rows("handworked_prefix.txt"):
        types, inst = fixture_pool((int(k0), int(k1), int(k2)))
        tab = oracle.instance_table(types, inst, 0.5, prec)
        pi, ph = parse_slots(slots)
        res = oracle.route_prefix(tab, [int(x)], [int(y)], [float(D)], pi, ph)
        assert res.instance_idx[0] == int(g), name
        assert res.tier[0] == int(tier), name
        assert res.est_e2e_ms[0] == pytest.approx(float(est), rel=1e-5), name
        assert res.slack_ms[0] == pytest.approx(float(slack), rel=1e-4, abs=2e-3), name
        assert (res.status != 0) == (name in ("hit_longer_than_prompt", "empty_and_unknown_slots")), name


@pytest.mark.parametrize("prec", PRECS)
def test_prefix_without_hits_is_plain_routing(prec):
    wl = W.make_workload(1, n_requests=3000, n_active=8)
    tab = oracle.instance_table(wl.types, wl.instances, 0.5, prec)
    cols = wl.requests.columns()
    plain = oracle.route(tab, *cols)
    n = len(cols[0])
    rng = np.random.default_rng(5)
    some_inst = rng.integers(0, tab.n_instances, (2, n)).astype(np.int32)
    for pi, ph in ((np.zeros((0, n), np.int32), np.zeros((0, n), np.int32)),          # no slots at all
                   (np.full((2, n), -1, np.int32), np.full((2, n), 77, np.int32)),    # only empty slots
                   (some_inst, np.zeros((2, n), np.int32))):                          # hits of length 0
        res = oracle.route_prefix(tab, *cols, pi, ph)
        for a, b in ((res.instance_idx, plain.instance_idx), (res.tier, plain.tier),
                     (res.est_e2e_ms, plain.est_e2e_ms), (res.slack_ms, plain.slack_ms)):
            np.testing.assert_array_equal(a, b)
        assert res.status == 0


def dense_hits(pi, ph, x, M):
    """H as a dense (N, M) matrix, built with numpy scatter-max (not the oracle's slot loop)."""
    n = len(x)
    H = np.zeros((n, M), np.int64)
    for k in range(pi.shape[0]):
        ok = (pi[k] >= 0) & (pi[k] < M)
        rows = np.nonzero(ok)[0]
        np.maximum.at(H, (rows, pi[k][rows]), np.clip(ph[k][rows], 0, x[rows]))
    return H


@pytest.mark.parametrize("prec", PRECS)
@pytest.mark.parametrize("n_slots", [1, 3])
def test_prefix_matches_dense_statement(prec, n_slots):
    """Eq. 2 evaluated over a dense H matrix with numpy, then the declarative post-condition of
    Algorithm 1 on that T: nothing preferred over the answer exists."""
    rng = np.random.default_rng(31 + n_slots)
    wl = W.make_workload(1, n_requests=1500, n_active=8)
    inst = wl.instances.copy()
    inst.free_kv_tokens[rng.random(inst.n_instances) < 0.5] = 300        # all three tiers occur
    tab = oracle.instance_table(wl.types, inst, 0.5, prec)
    x, y, D = (a.copy() for a in wl.requests.columns())
    D[::3] *= 0.4
    x[::40] = 1 << 22                                                   # no instance has room for these
    M = tab.n_instances
    pi = rng.integers(-1, M + 1, (n_slots, len(x))).astype(np.int32)     # -1 = empty, M = unknown
    ph = rng.integers(-5, 20000, (n_slots, len(x))).astype(np.int32)     # some negative, some > L_in
    # a third of the deadlines sit just below the hit-free estimate of the request's first
    # cached instance, so that the hit decides whether that instance is feasible
    g0 = np.clip(pi[0], 0, M - 1)
    T_plain = tab.q[g0].astype(np.float64) + tab.p[g0] * x.astype(np.float64) + tab.d[g0] * y.astype(np.float64)
    D[1::3] = (T_plain * 0.9995).astype(np.float32)[1::3]
    res = oracle.route_prefix(tab, x, y, D, pi, ph)
    H = dense_hits(pi, ph, x, M)
    q, p, d = (np.asarray(a, np.float64) for a in (tab.q, tab.p, tab.d))
    xh = (x[:, None] - H).astype(np.float64)
    if prec == "f64":
        T = q + p * xh + d * y[:, None].astype(np.float64)
    else:
        t1 = (p * xh + q).astype(np.float32)
        T = (d * y[:, None].astype(np.float64) + t1).astype(np.float32).astype(np.float64)
    idx_all = np.arange(M)
    seen = set()
    for r in range(len(x)):
        ok = (int(x[r]) + int(y[r])) <= np.asarray(tab.kv)
        feas = ok & (T[r] <= float(D[r]))
        g = int(res.instance_idx[r])
        if feas.any():
            assert res.tier[r] == 1 and feas[g]
            assert not (feas & ((d > d[g]) | ((d == d[g]) & (idx_all < g)))).any()
        else:
            pool = ok if ok.any() else np.ones_like(ok)
            assert res.tier[r] == (2 if ok.any() else 3) and pool[g]
            assert not (pool & ((T[r] < T[r, g]) | ((T[r] == T[r, g]) & (idx_all < g)))).any()
        assert res.est_e2e_ms[r] == pytest.approx(T[r, g], rel=1e-12 if prec == "f64" else 0, abs=0)
        seen.add(int(res.tier[r]))
    assert seen == {1, 2, 3}
    assert res.status == (4 | 1)        # out-of-range hit lengths and unknown instances were seen
    plain = oracle.route(tab, x, y, D)
    assert (plain.instance_idx != res.instance_idx).mean() > 0.05       # the hits do change answers


def test_constant_hit_on_one_instance_is_a_queue_credit():
    """If every request has the same hit h on instance g, Eq. 2 reads
    (q_g - p_g h) + p_g L_in + d_g L_out on g: plain routing against a table whose q_g is
    lowered by p_g h.  Checked against route() (pinned above) in double precision."""
    wl = W.make_workload(1, n_requests=4000, n_active=8)
    tab = oracle.instance_table(wl.types, wl.instances, 0.5, "f64")
    x, y, D = wl.requests.columns()
    g, h = 5, 16                                   # every prompt has at least 16 tokens
    assert x.min() >= h
    pi = np.full((1, len(x)), g, np.int32)
    ph = np.full((1, len(x)), h, np.int32)
    res = oracle.route_prefix(tab, x, y, D, pi, ph)
    q2 = tab.q.copy()
    q2[g] -= tab.p[g] * h
    ref = oracle.route(oracle.InstanceTable(q2, tab.p, tab.d, tab.kv, 0, "f64"), x, y, D)
    same = res.instance_idx == ref.instance_idx
    assert same.mean() > 0.999                     # rounding order may flip an exact tie, nothing else
    np.testing.assert_allclose(res.est_e2e_ms[same], ref.est_e2e_ms[same], rtol=1e-12)
    np.testing.assert_array_equal(res.tier[same], ref.tier[same])


def test_prefix_single_instance_closed_form():
    types, inst = fixture_pool()
    one = W.InstanceState(*(a[1:2].copy() for a in inst.columns()))
    tab = oracle.instance_table(types, one, 0.5, "f64")
    x = np.array([1000, 1000, 50, 0], np.int32)
    y = np.array([200, 0, 7, 9], np.int32)
    hit = np.array([640, 1000, 48, 0], np.int32)
    res = oracle.route_prefix(tab, x, y, np.full(4, 1e9, np.float32), np.zeros((1, 4), np.int32), hit[None, :])
    p = float(np.float32(0.05))
    d = 14.0 + float(np.float32(0.08)) * 10
    q = 0.5 * (2000 * p) + 0.5 * float(np.float32(2000 * p))        # EMA step on the carried (float) state
    np.testing.assert_allclose(res.est_e2e_ms, q + p * (x - hit) + d * y, rtol=1e-12)


def test_prefix_threaded_split_is_identical():
    wl = W.make_workload(1, n_requests=5001, n_active=8)
    tab = oracle.instance_table(wl.types, wl.instances, 0.5, "f32")
    cols = wl.requests.columns()
    pi, ph = W.make_prefix_hits(wl.requests, tab.n_instances, seed=1, n_slots=2)
    a = oracle.route_prefix(tab, *cols, pi, ph)
    b = oracle.route_prefix(tab, *cols, pi, ph, threads=7)
    for u, v in ((a.instance_idx, b.instance_idx), (a.est_e2e_ms, b.est_e2e_ms), (a.tier, b.tier)):
        np.testing.assert_array_equal(u, v)


# --------------------------------------------------------------------------------------
# black-box coefficients: EMA step and directly given tables (Sec. 3.3)
# --------------------------------------------------------------------------------------

@pytest.mark.parametrize("prec", PRECS)
def test_ema_closed_form_and_special_cases(prec):
    """n EMA steps unroll to  (1-a)^n c0 + a * sum_k (1-a)^(n-1-k) obs_k ; alpha = 0 keeps the
    state, alpha = 1 replaces it, a constant observation is a fixed point's limit."""
    rng = np.random.default_rng(8)
    M, n, a = 50, 12, 0.3
    c0 = rng.uniform(0, 100, M).astype(np.float32)
    obs = rng.uniform(0, 100, (n, M)).astype(np.float32)
    c = c0.astype(np.float64 if prec == "f64" else np.float32)
    for k in range(n):
        c, st = oracle.ema_update(a, obs[k], c, prec)
        assert st == 0
    a32 = float(np.float32(a))
    want = (1 - a32) ** n * c0.astype(np.float64) + a32 * sum((1 - a32) ** (n - 1 - k) * obs[k].astype(np.float64) for k in range(n))
    np.testing.assert_allclose(c, want, rtol=1e-12 if prec == "f64" else 2e-6)
    same, _ = oracle.ema_update(0.0, obs[0], c0, prec)
    np.testing.assert_array_equal(same, c0)
    repl, _ = oracle.ema_update(1.0, obs[0], c0, prec)
    np.testing.assert_array_equal(repl, obs[0])
    c = c0.astype(np.float64 if prec == "f64" else np.float32)
    for _ in range(200):
        c, _ = oracle.ema_update(0.5, np.full(M, 42.0, np.float32), c, prec)
    np.testing.assert_allclose(c, 42.0, rtol=1e-6)


@pytest.mark.parametrize("prec", PRECS)
def test_ema_ignores_invalid_observations(prec):
    c0 = np.array([5.0, 6.0, 7.0, 8.0], np.float32)
    obs = np.array([1.0, -1.0, np.nan, 0.0], np.float32)
    c, st = oracle.ema_update(0.5, obs, c0, prec)
    np.testing.assert_allclose(c, [3.0, 6.0, 7.0, 4.0])
    assert st == 4


@pytest.mark.parametrize("prec", PRECS)
def test_ema_matches_the_queue_delay_step_of_the_typed_table(prec):
    """The EMA step that instance_table() applies to q (pinned above by its own closed form) is
    this same step with obs = w_g = queued * p."""
    wl = W.make_workload(1, n_requests=8, n_active=8)
    tab = oracle.instance_table(wl.types, wl.instances, 0.3, prec)
    p32 = wl.types.prefill_ms_per_tok[wl.instances.type_id]
    if prec == "f64":
        w = wl.instances.queued_prefill_tokens.astype(np.float64) * p32.astype(np.float64)
        want = float(np.float32(0.3)) * w + (1 - float(np.float32(0.3))) * wl.instances.q_ema_ms.astype(np.float64)
        np.testing.assert_allclose(tab.q, want, rtol=1e-12)
    else:
        w = (wl.instances.queued_prefill_tokens.astype(np.float32) * p32).astype(np.float32)
        got, _ = oracle.ema_update(0.3, w, wl.instances.q_ema_ms, "f32")
        np.testing.assert_array_equal(tab.q, got)


@pytest.mark.parametrize("prec", PRECS)
def test_direct_table_is_the_identity_on_valid_input_and_clamps_the_rest(prec):
    wl = W.make_workload(1, n_requests=2000, n_active=8)
    bb = W.make_blackbox_table(wl.types, wl.instances, seed=1)
    tab = oracle.direct_table(*bb.columns(), prec)
    for got, src in ((tab.q, bb.q_ms), (tab.p, bb.p_ms_per_tok), (tab.d, bb.d_ms_per_tok), (tab.kv, bb.free_kv_tokens)):
        np.testing.assert_array_equal(got, src.astype(got.dtype))
    assert tab.status == 0
    assert len(np.unique(bb.p_ms_per_tok)) > 0.9 * bb.n_instances          # no shared p: no GPU types to lean on
    # routing on it obeys the declarative post-condition of Algorithm 1
    x, y, D = wl.requests.columns()
    res = oracle.route(tab, x, y, D)
    check_postcondition(tab.q, tab.p, tab.d, tab.kv, x[:400], y[:400], D[:400], res.instance_idx, res.tier, prec)
    bad = oracle.direct_table([1, -1, np.nan, 2], [0.1, 0.1, 0.1, -0.5], [3, 3, 3, np.nan], [5, 5, -2, 5], prec)
    np.testing.assert_array_equal(bad.q, [1, 0, 0, 2])
    np.testing.assert_array_equal(bad.p, np.array([0.1, 0.1, 0.1, 0], np.float32).astype(bad.p.dtype))
    np.testing.assert_array_equal(bad.d, [3, 3, 3, 0])
    np.testing.assert_array_equal(bad.kv, [5, 5, 0, 5])
    assert bad.status == 4


def test_direct_table_of_the_typed_coefficients_routes_like_the_typed_table():
    wl = W.make_workload(1, n_requests=3000, n_active=8)
    typed = oracle.instance_table(wl.types, wl.instances, 0.5, "f32")
    direct = oracle.direct_table(typed.q, typed.p, typed.d, typed.kv.astype(np.int32), "f32")
    a = oracle.route(typed, *wl.requests.columns())
    b = oracle.route(direct, *wl.requests.columns())
    np.testing.assert_array_equal(a.instance_idx, b.instance_idx)
    np.testing.assert_array_equal(a.est_e2e_ms, b.est_e2e_ms)


# --------------------------------------------------------------------------------------
# Algorithm 1 one request at a time
# --------------------------------------------------------------------------------------

@pytest.mark.parametrize("cfg_id,alpha", [(0, 0.5), (1, 0.5), (1, 0.0), (1, 1.0)])
def test_sequential_equals_rounds_of_one_request(cfg_id, alpha):
    """The sequential reading is, by definition, rounds of a single request: table, route,
    advance -- three functions pinned above, composed here in Python."""
    wl = W.make_workload(cfg_id, n_requests=300, n_active=8)
    x, y, D = wl.requests.columns()
    D = D.copy(); D[::5] *= 0.3                       # some requests fall back
    state = wl.instances.copy()
    state.free_kv_tokens[::2] = 4000                  # KV room runs out along the way
    seq_state = state.copy()
    seq = oracle.route_sequential(wl.types, seq_state, alpha, x, y, D)
    for r in range(len(x)):
        tab = oracle.instance_table(wl.types, state, alpha, "f32")
        one = oracle.route(tab, x[r:r + 1], y[r:r + 1], D[r:r + 1])
        assert seq.instance_idx[r] == one.instance_idx[0], r
        assert seq.tier[r] == one.tier[0] and seq.est_e2e_ms[r] == one.est_e2e_ms[0], r
        assert seq.slack_ms[r] == one.slack_ms[0], r
        oracle.advance(state, tab, one.instance_idx, x[r:r + 1], y[r:r + 1])
    for a, b in zip(seq_state.columns(), state.columns()):
        np.testing.assert_array_equal(a, b)
    assert {1, 2} <= set(seq.tier.tolist())


def test_sequential_moves_on_when_the_deadline_binds():
    """Identical requests against identical idle instances.  The snapshot reading sends all of
    them to instance 0.  One at a time with a loose deadline they still all go there (the
    instance just used has the larger batch, hence the larger d, and just-enough prefers it);
    with a deadline that the growing queue breaks, later requests move to other instances."""
    types = base_types()
    M = 8
    inst = W.InstanceState(np.zeros(M, np.int32), np.zeros(M, np.int32), np.zeros(M, np.int32),
                           np.full(M, 10**6, np.int32), np.zeros(M, np.float32))
    n = 64
    x = np.full(n, 1000, np.int32); y = np.full(n, 100, np.int32)
    loose = np.full(n, 1e9, np.float32)
    snap = oracle.route(oracle.instance_table(types, inst, 0.5, "f32"), x, y, loose)
    assert (snap.instance_idx == 0).all()
    seq = oracle.route_sequential(types, inst.copy(), 0.5, x, y, loose)
    assert (seq.instance_idx == 0).all() and (seq.tier == 1).all()
    assert (np.diff(seq.est_e2e_ms) > 0).all()                       # each one waits behind the ones before
    tight = np.full(n, 8.0 * 100 + 0.025 * 1000 + 30.0, np.float32)   # unloaded T (825 ms) + 30 ms
    seq_tight = oracle.route_sequential(types, inst.copy(), 0.5, x, y, tight)
    assert seq_tight.instance_idx[0] == 0 and (seq_tight.tier[:2] == 1).all()
    assert len(set(seq_tight.instance_idx.tolist())) > 1


def test_sequential_first_request_is_the_batch_answer():
    wl = W.make_workload(1, n_requests=50, n_active=8)
    tab = oracle.instance_table(wl.types, wl.instances, 0.5, "f32")
    batch = oracle.route(tab, *wl.requests.columns())
    seq = oracle.route_sequential(wl.types, wl.instances.copy(), 0.5, *wl.requests.columns())
    assert seq.instance_idx[0] == batch.instance_idx[0] and seq.est_e2e_ms[0] == batch.est_e2e_ms[0]
