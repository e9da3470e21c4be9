"""Pins for the oracle's rolling z-score gate and backward-pass budget:
hand-built norm streams, a worked example, a library mean/std, and the
(shutoff step, total backward passes) pairs the paper prints."""
import math
import os

import numpy as np
import pytest

from oracle import gxpo_oracle as ora

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def run_stream(norms, **kw):
    gate = ora.Gate(ora.GxpoCfg(**kw))
    recs = []
    for x in norms:
        if not gate.active:
            break
        recs.append(gate.update(x))
    return gate, recs


def test_constant_stream_never_trips():
    gate, recs = run_stream([0.0175] * 200, tau=0.5)
    assert gate.active and gate.s_star == -1 and gate.t == 200
    assert all(not r[0] for r in recs)
    assert all(abs(r[1]) < 1e-6 for r in recs[2:])      # sigma ~ 0, numerator ~ 0 (rounding only)
    gate, recs = run_stream([0.5] * 50, tau=0.5)        # 0.5 sums exactly
    assert all(r[1] == 0.0 for r in recs[2:])


def test_worked_example():
    # past norms 1, 2, 3 then 4:  mu = 2, sigma = sqrt(2/3), Z = 2 / (sigma + eps)
    gate, recs = run_stream([1.0, 2.0, 3.0, 4.0], tau=100.0, gate_eps=1e-8)
    tripped, z, mu, sigma = recs[3]
    assert mu == 2.0
    assert sigma == pytest.approx(math.sqrt(2.0 / 3.0), rel=1e-15)
    assert z == pytest.approx(2.0 / (math.sqrt(2.0 / 3.0) + 1e-8), rel=1e-15)
    assert not tripped
    # sample standard deviation when asked for: sigma = 1
    gate, recs = run_stream([1.0, 2.0, 3.0, 4.0], tau=100.0, std_ddof=1)
    assert recs[3][3] == pytest.approx(1.0, rel=1e-15)


def test_warm_up_and_earliest_trip():
    # Algorithm 1 checks only when the buffer holds more than one norm
    gate, recs = run_stream([1.0, 50.0, 1.0, 2.0], tau=0.5)
    assert math.isnan(recs[0][1]) and math.isnan(recs[1][1])   # steps 0, 1: fill only
    assert not recs[0][0] and not recs[1][0]
    gate, recs = run_stream([1.0, 1.0, 2.0, 2.0, 2.0], tau=0.5)
    assert [r[0] for r in recs] == [False, False, True]
    assert gate.s_star == 3 and not gate.active                 # s* = t + 1 with t = 2
    assert gate.t == 3


def test_step_up_by_eight_at_step_40():
    norms = [0.0175] * 40 + [0.14] + [0.0175] * 23
    gate, recs = run_stream(norms, tau=0.5, window=20)
    assert len(recs) == 41 and recs[40][0]
    assert gate.s_star == 41
    # with a little jitter in the baseline too
    rng = np.random.default_rng(0)
    base = 0.0175 * (1 + 1e-3 * rng.standard_normal(64))
    base[40] *= 8
    z_max_before = max(r[1] for r in run_stream(base[:40], tau=1e9)[1][2:])
    gate, recs = run_stream(base, tau=z_max_before + 1.0, window=20)
    assert gate.s_star == 41


def test_check_happens_before_insert():
    # past [1, 3]: mu 2, sigma 1 -> Z(2.9) = 0.9.  Had 2.9 been inserted first:
    # mu 2.3, sigma 0.92 -> Z 0.65.  tau = 0.8 separates the two readings.
    gate, recs = run_stream([1.0, 3.0, 2.9], tau=0.8, gate_eps=0.0)
    assert recs[2][1] == pytest.approx(0.9, rel=1e-12) and recs[2][0]


def test_threshold_is_inclusive_and_one_sided():
    gate, recs = run_stream([1.0, 3.0, 3.0], tau=1.0, gate_eps=0.0)
    assert recs[2][1] == 1.0 and recs[2][0]                     # Z == tau trips
    gate, recs = run_stream([1.0, 3.0, 2.999], tau=1.0, gate_eps=0.0)
    assert not recs[2][0]
    gate, recs = run_stream([3.0, 3.1, 0.001, 3.0, 3.1], tau=3.0)
    assert recs[2][1] < -3.0 and not recs[2][0]                 # a sharp DROP does not trip


def test_window_drops_oldest():
    # w = 3: at step 4 the past is [1, 1, 1] (0 dropped) -> sigma 0 -> Z huge
    gate, recs = run_stream([0.0, 1.0, 1.0, 1.0, 1.2], tau=2.0, window=3)
    assert recs[4][0] and recs[4][2] == 1.0 and recs[4][3] == 0.0
    # w = 4: past [0, 1, 1, 1] -> mu .75, sigma .433 -> Z = 1.04 < 2
    gate, recs = run_stream([0.0, 1.0, 1.0, 1.0, 1.2], tau=2.0, window=4)
    assert not recs[4][0]
    assert recs[4][1] == pytest.approx((1.2 - 0.75) / (math.sqrt(0.1875) + 1e-8), rel=1e-12)


def test_against_library_mean_std_on_random_stream():
    rng = np.random.default_rng(123)
    norms = np.abs(1.0 + 0.2 * rng.standard_normal(300))
    w, eps = 7, 1e-8
    gate, recs = run_stream(norms, tau=1e9, window=w, gate_eps=eps)
    for t in range(2, 300):
        past = norms[max(0, t - w):t]
        z = (norms[t] - np.mean(past)) / (np.std(past) + eps)
        assert recs[t][1] == pytest.approx(float(z), rel=1e-9, abs=1e-12)
    zs = np.array([r[1] for r in recs[2:]])
    tau = 1.5
    first = 2 + int(np.argmax(zs >= tau))
    gate, recs = run_stream(norms, tau=tau, window=w, gate_eps=eps)
    assert gate.s_star == first + 1 and len(recs) == first + 1


def test_trip_is_permanent_and_tripping_norm_is_pushed():
    gate = ora.Gate(ora.GxpoCfg(tau=0.5, window=4))
    for x in [1.0, 1.0, 1.0, 9.0]:
        gate.update(x)
    assert gate.s_star == 4 and not gate.active
    for _ in range(10):
        gate.fallback_tick()
    assert gate.s_star == 4 and gate.t == 14 and not gate.active
    # the 9.0 went into the buffer: a further (hypothetical) update sees it in mu
    _, _, mu, _ = gate.update(1.0)
    assert mu == pytest.approx((1.0 + 1.0 + 1.0 + 9.0) / 4)


def test_nonfinite_norm_trips():
    gate, recs = run_stream([1.0, 1.0, float("nan")], tau=0.5)
    assert recs[2][0] and gate.s_star == 3
    gate, recs = run_stream([float("inf")], tau=0.5)
    assert recs[0][0] and gate.s_star == 1


def _budget_rows():
    rows = []
    with open(os.path.join(GOLDEN, "backward_budget_rows.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                rows.append(tuple(int(x) for x in line.split()))
    return rows


def test_budget_identity_reproduces_printed_rows():
    rows = _budget_rows()
    assert len(rows) == 6
    for T, s_star, total in rows:
        assert ora.backward_budget(s_star, T) == total
    assert ora.backward_budget(-1, 300) == 900            # never trips: 3 T


@pytest.mark.parametrize("row", [0, 3])
def test_outer_loop_counts_backward_passes(row):
    """Run Algorithm 1's outer loop for T steps on a tiny problem whose g_slow
    norm jumps at step s*-1 and count the gradient evaluations it really makes."""
    T, s_star, total = _budget_rows()[row]
    calls = {"n": 0}
    step = {"t": 0}
    n = 8
    base = np.full(n, 1e-2)

    def grad_fn(which, theta):
        calls["n"] += 1
        scale = 8.0 if (which == 2 and step["t"] == s_star - 1) else 1.0
        return base * scale

    st = ora.State(np.zeros(n), ora.OptCfg(kind="adamw", lr=1e-7))
    gate = ora.Gate(ora.GxpoCfg(tau=0.5, window=20))
    cfg = ora.GxpoCfg(K=3, alpha=0.5)
    passes = 0
    for t in range(T):
        step["t"] = t
        rec = ora.train_step(st, gate, cfg, grad_fn, round_f32=True)
        passes += rec["backward_passes"]
        assert (rec["phase"] == "active") == (t < s_star)
    assert gate.s_star == s_star
    assert calls["n"] == passes == total
    assert st.t_opt == total                              # one optimizer step per backward pass


def test_z_score_is_invariant_to_shift_and_positive_scale_of_the_norm_stream():
    """Z = (x - mu) / (sigma + eps) (Eq. (z_score)): adding a constant to every norm changes
    nothing, and with eps = 0 neither does multiplying them by c > 0 -- so the gate flips at the
    same step.  A mean taken over the wrong window, a variance without the mean removed or a
    sigma that is a variance all break one of the two."""
    t = np.arange(60)
    norms = 1.0 + 0.05 * (-1.0) ** t + 0.01 * np.sin(t)       # |Z| stays near 1 from the second entry on
    norms[37] += 0.5                                          # a clear upward jump: Z ~ 10
    ref_gate, ref = run_stream(norms, tau=2.5, gate_eps=0.0, window=10)
    assert ref_gate.s_star == 38
    for shift, scale in ((100.0, 1.0), (0.0, 1e-3), (5.0, 40.0)):
        gate, recs = run_stream(shift + scale * norms, tau=2.5, gate_eps=0.0, window=10)
        assert gate.s_star == ref_gate.s_star and len(recs) == len(ref)
        for (t0, z0, mu0, s0), (t1, z1, mu1, s1) in zip(ref, recs):
            assert t0 == t1
            if not math.isnan(z0):
                assert z1 == pytest.approx(z0, rel=1e-7, abs=1e-9)
                assert mu1 == pytest.approx(shift + scale * mu0, rel=1e-12)
                assert s1 == pytest.approx(scale * s0, rel=1e-7, abs=1e-12)
