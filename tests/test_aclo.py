"""Confidence (Eq. 1), Confidence LSH tables (Sec. 3.2, Eq. 4) and the accuracy-constrained budget
choice (ACLO, Eq. 2): pins for the oracle on the CPU, then the device entry points against it."""
import math

import numpy as np
import pytest
from scipy import special

from oracle import oracle as orc
from test_oracle_method import relu_inputs
from test_oracle_pins import tiny_model

PROFILE = np.array([500, 1000, 2500, 5000, 10000], np.uint16)


def cross_entropy_scipy(z_full, z_k):
    """H(p, q) = H(p) + KL(p || q) from scipy's entropy kernels."""
    p = special.softmax(np.asarray(z_full, np.float64))
    q = special.softmax(np.asarray(z_k, np.float64))
    return float(special.entr(p).sum() + special.rel_entr(p, q).sum())


# ---------------------------------------------------------------------------
# c(k, x)
# ---------------------------------------------------------------------------

def test_confidence_hand_worked_two_classes():
    # p = (1/2, 1/2), q = softmax(ln 3, 0) = (3/4, 1/4): c = (ln 3/4 + ln 1/4) / 2
    got = orc.confidence([0.0, 0.0], [math.log(3.0), 0.0])
    assert abs(got - 0.5 * (math.log(0.75) + math.log(0.25))) < 1e-7     # ln 3 is rounded to fp32 on the way in


def test_confidence_closed_forms():
    rng = np.random.default_rng(300)
    for n in (2, 10, 1000):
        z = (rng.standard_normal(n) * 3).astype(np.float32)
        p = special.softmax(z.astype(np.float64))
        # same prediction: minus the entropy of the full network's prediction
        assert abs(orc.confidence(z, z) + special.entr(p).sum()) < 1e-12 * n
        # a constant added to every logit changes no probability
        assert abs(orc.confidence(z, z + np.float32(4.0)) - orc.confidence(z, z)) < 1e-5
        # uniform prediction of the k% network: log(1/n) whatever the full network says
        assert abs(orc.confidence(z, np.zeros(n, np.float32)) + math.log(n)) < 1e-12
        # Gibbs: no prediction is closer to p than p itself
        zk = z + rng.standard_normal(n).astype(np.float32)
        assert orc.confidence(z, zk) <= orc.confidence(z, z) + 1e-12
    # large logits do not overflow
    assert np.isfinite(orc.confidence(np.array([900.0, -900.0], np.float32), np.array([-800.0, 800.0], np.float32)))


def test_confidence_is_minus_cross_entropy():
    rng = np.random.default_rng(301)
    for n in (3, 10, 257):
        for _ in range(5):
            zf = (rng.standard_normal(n) * 2).astype(np.float32)
            zk = (rng.standard_normal(n) * 2).astype(np.float32)
            want = -cross_entropy_scipy(zf, zk)
            assert abs(orc.confidence(zf, zk) - want) <= 1e-12 * max(1.0, abs(want))


# ---------------------------------------------------------------------------
# tables
# ---------------------------------------------------------------------------

def small_net(seed=310):
    rng = np.random.default_rng(seed)
    m = tiny_model(rng, [24, 64, 48, 6], [1, 1, 0], K=3, L=2)
    calib = relu_inputs(rng, 400, 24)
    m.build(calib_dense=calib, seed=7)
    return rng, m, calib


def test_confidence_tables_brute_force():
    rng, m, calib = small_net()
    s, c = m.confidence_build(calib, PROFILE)
    full = m.run(np.full(400, 10000, np.uint16), x_dense=calib)
    want_s = np.zeros_like(s); want_c = np.zeros_like(c)
    for i, bp in enumerate(PROFILE):
        r = m.run(np.full(400, bp, np.uint16), x_dense=calib)
        for x in range(400):
            cx = -cross_entropy_scipy(full["logits"][x], r["logits"][x])
            for b in range(2):
                key = full["codes"][x, 0, b]          # first activator layer's key of table b
                want_s[b, key, i] += cx
                if i == 0:
                    want_c[b, key] += 1
    assert np.array_equal(c, want_c) and c.sum() == 2 * 400
    assert np.allclose(s, want_s, rtol=1e-10, atol=1e-12)
    # the full network agrees with itself: that column is minus the summed entropies, the largest of each bucket
    assert np.all(s[:, :, -1][:, :, None] >= s - 1e-9)


def test_confidence_tables_refuse_unsupported_networks():
    rng = np.random.default_rng(311)
    m = tiny_model(rng, [16, 32, 40], [1, 1], K=2, L=2)       # budgeted output layer: no complete logit vector
    calib = relu_inputs(rng, 50, 16)
    m.build(calib_dense=calib, seed=1)
    with pytest.raises(RuntimeError):
        m.confidence_build(calib, PROFILE)


# ---------------------------------------------------------------------------
# ACLO
# ---------------------------------------------------------------------------

def brute_force_aclo(keys, s, c, profile, thr_rows):
    out, met = [], []
    for q in range(keys.shape[0]):
        rows = sum(int(c[b, keys[q, b]]) for b in range(keys.shape[1]))
        pick, ok = 10000, 0
        if rows:
            for i, bp in enumerate(profile):
                est = sum(float(s[b, keys[q, b], i]) for b in range(keys.shape[1])) / rows
                if est >= float(thr_rows[q][i]):
                    pick, ok = int(bp), 1
                    break
        out.append(pick); met.append(ok)
    return np.array(out, np.uint16), np.array(met, np.uint8)


def test_aclo_brute_force_on_hand_made_tables():
    rng, m, calib = small_net(320)
    x = relu_inputs(rng, 60, 24)
    keys = m.run(np.full(60, 10000, np.uint16), x_dense=x)["codes"][:, 0, :]
    s = -rng.random((2, 8, PROFILE.size)) * 50.0
    c = rng.integers(0, 40, (2, 8)).astype(np.uint32)
    c[0, keys[0, 0]] = 0; c[1, keys[0, 1]] = 0                # query 0 meets no training row at all
    thr = -rng.random((3, PROFILE.size)).astype(np.float32) * 3.0
    target = rng.integers(0, 3, 60).astype(np.uint32)
    got, met, est = m.aclo_budgets(s, c, PROFILE, x, thr, target)
    want, want_met = brute_force_aclo(keys, s, c, PROFILE, thr[target])
    assert np.array_equal(got, want) and np.array_equal(met, want_met)
    assert got[0] == 10000 and met[0] == 0
    assert len(set(got.tolist())) >= 3                         # the case exercises several outcomes
    # the estimate is the pooled mean of the buckets the query falls into
    q = 5
    rows = int(c[0, keys[q, 0]]) + int(c[1, keys[q, 1]])
    assert rows > 0
    assert np.allclose(est[q], (s[0, keys[q, 0]] + s[1, keys[q, 1]]) / rows)


def test_aclo_limits_and_monotonicity():
    rng, m, calib = small_net(321)
    s, c = m.confidence_build(calib, PROFILE)
    x = relu_inputs(rng, 80, 24)
    lo = np.full((1, PROFILE.size), -np.inf, np.float32)
    hi = np.full((1, PROFILE.size), np.inf, np.float32)
    got, met, est = m.aclo_budgets(s, c, PROFILE, x, lo)
    seen = met == 1                                            # queries whose buckets hold training rows
    assert seen.sum() > 40
    assert np.all(got[seen] == PROFILE[0]) and np.all(got[~seen] == 10000)
    got, met, _ = m.aclo_budgets(s, c, PROFILE, x, hi)
    assert np.all(got == 10000) and np.all(met == 0)
    # a stricter accuracy target (higher thresholds) never lowers k
    t1 = np.quantile(est[seen], 0.4, axis=0).astype(np.float32)[None, :]
    t2 = np.quantile(est[seen], 0.8, axis=0).astype(np.float32)[None, :]
    k1, _, _ = m.aclo_budgets(s, c, PROFILE, x, t1)
    k2, _, _ = m.aclo_budgets(s, c, PROFILE, x, t2)
    assert np.all(k2 >= k1) and np.any(k2 > k1)
    # the full network's own column: a threshold at or below the estimate is always met at 100 %
    full_only = np.concatenate([hi[:, :-1], np.full((1, 1), -1e30, np.float32)], axis=1)
    got, met, _ = m.aclo_budgets(s, c, PROFILE, x, full_only)
    assert np.all(got == 10000) and np.array_equal(met, seen.astype(np.uint8))


def test_aclo_threshold_is_inclusive():
    # "confidence >= t": an estimate exactly at the threshold is accepted
    rng, m, calib = small_net(322)
    x = relu_inputs(rng, 10, 24)
    s = np.full((2, 8, PROFILE.size), -8.0)
    s[:, :, 0] = -16.0                                         # estimates: -2 at the first k, -1 afterwards
    c = np.full((2, 8), 8, np.uint32)
    thr = np.array([[-1.0, -1.0, 0.0, 0.0, 0.0]], np.float32)
    got, met, est = m.aclo_budgets(s, c, PROFILE, x, thr)
    assert np.all(est[:, 0] == -2.0) and np.all(est[:, 1] == -1.0)
    assert np.all(got == PROFILE[1]) and np.all(met == 1)


# ---------------------------------------------------------------------------
# device entry points against the oracle
# ---------------------------------------------------------------------------

def _device_case(wl, n_cal):
    import torch
    from paper_2204_08400_b200 import binding as sl, harness
    from parity_util import oracle_model
    dm = harness.DeviceModel(wl, n_cal=n_cal)
    om = oracle_model(wl, n_cal=n_cal)
    rows = wl.calib[:n_cal]
    want_s, want_c = om.confidence_build(rows, PROFILE)
    conf = sl.slonn_confidence_build(dm.model, harness._dev(rows, dm.device), PROFILE)
    got_s, got_c = sl.slonn_confidence_to_host(conf)
    assert np.array_equal(got_c, want_c), "rows per bucket"
    # same logits bit for bit, same order of additions; exp and log come from two math libraries
    assert np.allclose(got_s, want_s, rtol=1e-11, atol=1e-11), "bucket sums"
    return torch, sl, harness, dm, om, conf, want_s, want_c


@pytest.mark.gpu
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_device_confidence_tables_and_aclo_budgets(dtype):
    from test_gpu_parity import custom_workload
    wl = custom_workload(330, [136, 200, 96, 24], [1, 1, 0], dtype, n=500, n_cal=700, K=4, L=2)
    torch, sl, harness, dm, om, conf, s, c = _device_case(wl, 700)
    # thresholds between observed estimates (no query sits on a threshold), three accuracy targets
    _, seen, est = om.aclo_budgets(s, c, PROFILE, wl.x, np.full((1, PROFILE.size), -np.inf, np.float32))
    qs = [0.25, 0.5, 0.8]
    thr = np.stack([np.quantile(est[seen == 1], q, axis=0) for q in qs]).astype(np.float32)
    target = np.random.default_rng(331).integers(0, 3, wl.n_queries).astype(np.uint32)
    want_bp, want_met, want_est = om.aclo_budgets(s, c, PROFILE, wl.x, thr, target)
    margin = np.min(np.abs(want_est - thr[target].astype(np.float64)), axis=1)
    dev = dm.device
    x = harness._dev(wl.x, dev)
    bp = torch.zeros(wl.n_queries, dtype=torch.int16, device=dev)
    met = torch.zeros(wl.n_queries, dtype=torch.uint8, device=dev)
    estd = torch.zeros((wl.n_queries, PROFILE.size), dtype=torch.float64, device=dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    sl.slonn_aclo_budgets(dm.model, conf, x, harness._dev(thr, dev), bp, target=harness._dev(target, dev), met=met,
                          estimate=estd, status=status)
    torch.cuda.synchronize()
    assert status.cpu().numpy()[0] == 0
    got_bp = bp.cpu().numpy().view(np.uint16)
    assert np.allclose(estd.cpu().numpy(), want_est, rtol=1e-11, atol=1e-11)
    clear = margin > 1e-9                                     # decisions away from a threshold are unique
    assert clear.mean() > 0.99
    assert np.array_equal(got_bp[clear], want_bp[clear]) and np.array_equal(met.cpu().numpy()[clear], want_met[clear])
    assert len(set(got_bp.tolist())) >= 3
    # the budgets feed the forward pass as they are
    g = harness.run_once(dm, wl.x, got_bp, max_budget_bp=10000)
    o = om.run(got_bp, x_dense=wl.x)
    assert g["status"][0] == 0 and np.array_equal(g["pred"], o["pred"]) and np.array_equal(g["logits"], o["logits"])
    # a target index outside the threshold table is reported, not followed
    bad = torch.full((wl.n_queries,), 7, dtype=torch.int32, device=dev)
    sl.slonn_aclo_budgets(dm.model, conf, x, harness._dev(thr, dev), bp, target=bad, status=status)
    torch.cuda.synchronize()
    assert status.cpu().numpy().view(np.uint32)[0] == 1       # -SLONN_ERR_ARG
    sl.slonn_confidence_free(conf)
    dm.free()


@pytest.mark.gpu
def test_device_aclo_input_width_just_below_the_shared_memory_opt_in_limit():
    """11,900 fp32 inputs are 47.6 KB of staged query: with the kernel's static shared memory that is more than a
    launch gets without opting in."""
    from test_gpu_parity import custom_workload
    wl = custom_workload(340, [11900, 64, 10], [1, 0], "f32", n=64, n_cal=200, K=3, L=2)
    torch, sl, harness, dm, om, conf, s, c = _device_case(wl, 200)
    thr = np.full((1, PROFILE.size), -1.0, np.float32)
    want_bp, want_met, want_est = om.aclo_budgets(s, c, PROFILE, wl.x, thr)
    dev = dm.device
    bp = torch.zeros(wl.n_queries, dtype=torch.int16, device=dev)
    estd = torch.zeros((wl.n_queries, PROFILE.size), dtype=torch.float64, device=dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    sl.slonn_aclo_budgets(dm.model, conf, harness._dev(wl.x, dev), harness._dev(thr, dev), bp, estimate=estd, status=status)
    torch.cuda.synchronize()
    assert status.cpu().numpy()[0] == 0
    assert np.allclose(estd.cpu().numpy(), want_est, rtol=1e-11, atol=1e-11)
    clear = np.min(np.abs(want_est - thr[0].astype(np.float64)), axis=1) > 1e-9
    assert np.array_equal(bp.cpu().numpy().view(np.uint16)[clear], want_bp[clear])
    sl.slonn_confidence_free(conf)
    dm.free()


@pytest.mark.gpu
def test_device_confidence_tables_c2_reduced():
    from paper_2204_08400_b200 import workloads as wl_mod
    wl = wl_mod.load("c2", n_queries=256, n_cal=2048, budget_bp=1000)
    torch, sl, harness, dm, om, conf, s, c = _device_case(wl, 2048)
    sl.slonn_confidence_free(conf)
    dm.free()


@pytest.mark.gpu
def test_device_confidence_refuses_unsupported_models_and_profiles():
    from paper_2204_08400_b200 import binding as sl, harness
    from test_gpu_parity import custom_workload
    wl = custom_workload(332, [72, 160, 328], [1, 1], "f32", n=16, n_cal=200, K=3, L=2)   # budgeted output layer
    dm = harness.DeviceModel(wl)
    rows = harness._dev(wl.calib, dm.device)
    with pytest.raises(sl.SlonnError) as e:
        sl.slonn_confidence_build(dm.model, rows, PROFILE)
    assert e.value.code == sl.ERR["ARG"]
    dm.free()
    wl = custom_workload(333, [72, 160, 24], [1, 0], "f32", n=16, n_cal=200, K=3, L=2)
    dm = harness.DeviceModel(wl)
    rows = harness._dev(wl.calib, dm.device)
    for prof, code in (([1000, 500], "ARG"), ([0, 500], "BUDGET"), (list(range(1, 70)), "DIM")):
        with pytest.raises(sl.SlonnError) as e:
            sl.slonn_confidence_build(dm.model, rows, prof)
        assert e.value.code == sl.ERR[code]
    dm.free()
