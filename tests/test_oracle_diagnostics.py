"""Pins of the oracle's active-step diagnostics (the quantities of the paper's
"Active-phase GXPO diagnostics" table) to things other than itself: a hand-computed
example, closed forms on the diagonal quadratic, library routines, degenerate cases."""
import math

import numpy as np
import pytest

from oracle import gxpo_oracle as ora


def f64(*x):
    return np.array(x, dtype=np.float64)


def test_hand_computed_example():
    # three active coordinates with r = 1/2, 2, -1/2 and one inactive (|g0| <= delta); K = 3:
    # scale = (1 + r + r^2) / (1 + r) = 7/6, 7/3, 3/2; inactive: 1
    g0 = f64(2.0, 1.0, -4.0, 1e-9)
    g1 = f64(1.0, 2.0, 2.0, 5.0)
    gs = f64(1.0, 0.0, 0.0, 0.0)
    th0 = f64(0.0, 0.0, 0.0, 0.0)
    th2 = f64(6.0, 3.0, 2.0, 1.0)                      # Delta_2
    d = ora.active_diagnostics(th0, th2, g0, g1, gs, K=3, delta=1e-8)
    assert d["g0_norm"] == pytest.approx(math.sqrt(4 + 1 + 16 + 1e-18), rel=1e-15)
    assert d["g1_norm"] == pytest.approx(math.sqrt(1 + 4 + 4 + 25), rel=1e-15)
    assert d["gslow_norm"] == 1.0
    assert d["cos_g0_gslow"] == pytest.approx(2.0 / math.sqrt(21 + 1e-18), rel=1e-15)
    assert d["ratio_mean"] == pytest.approx((0.5 + 2.0 - 0.5) / 3, rel=1e-15)
    assert d["ratio_std"] == pytest.approx(math.sqrt(((0.5 - 2 / 3) ** 2 + (2 - 2 / 3) ** 2 + (-0.5 - 2 / 3) ** 2) / 3), rel=1e-14)
    assert d["scale_mean"] == pytest.approx((7 / 6 + 7 / 3 + 3 / 2 + 1) / 4, rel=1e-15)
    dk = math.sqrt((6 * 7 / 6) ** 2 + (3 * 7 / 3) ** 2 + (2 * 3 / 2) ** 2 + 1)
    assert d["disp_ratio"] == pytest.approx(dk / math.sqrt(36 + 9 + 4 + 1), rel=1e-15)
    assert d["inactive_frac"] == 0.25 and d["n_active"] == 3 and d["n_irregular"] == 0


@pytest.mark.parametrize("K", [3, 5, 10])
def test_closed_forms_on_the_diagonal_quadratic(K):
    """Plain GD on f = sum a x^2/2 - b x: r_i = 1 - eta a_i exactly, and the extrapolated
    displacement is (r^K - 1)(theta0 - theta*) against (r^2 - 1)(theta0 - theta*)."""
    rng = np.random.default_rng(K)
    n, eta = 500, 0.1
    a = rng.uniform(0.1, 1.0, n)
    b = rng.standard_normal(n)
    th0 = rng.standard_normal(n)
    g0 = a * th0 - b
    th1 = th0 - eta * g0
    g1 = a * th1 - b
    th2 = th1 - eta * g1
    d = ora.active_diagnostics(th0, th2, g0, g1, g1, K=K, delta=1e-12)
    r = 1.0 - eta * a
    star = b / a
    assert d["ratio_mean"] == pytest.approx(np.mean(r), rel=1e-10)
    assert d["ratio_std"] == pytest.approx(np.std(r), rel=1e-8)
    assert d["scale_mean"] == pytest.approx(np.mean((1 - r ** K) / (1 - r ** 2)), rel=1e-10)
    want = np.linalg.norm((r ** K - 1) * (th0 - star)) / np.linalg.norm((r ** 2 - 1) * (th0 - star))
    assert d["disp_ratio"] == pytest.approx(want, rel=1e-9)
    assert d["inactive_frac"] == 0.0


def test_library_routines_on_random_data():
    rng = np.random.default_rng(3)
    n = 2000
    g0 = rng.standard_normal(n)
    g1 = g0 * rng.uniform(0.2, 1.2, n)
    gs = g0 + 0.3 * rng.standard_normal(n)
    g0[::50] = 0.0                                     # 2 % inactive
    th0 = rng.standard_normal(n)
    th2 = th0 + 1e-2 * rng.standard_normal(n)
    d = ora.active_diagnostics(th0, th2, g0, g1, gs, K=5, delta=1e-8)
    act = np.abs(g0) > 1e-8
    r = g1[act] / g0[act]
    assert d["g0_norm"] == pytest.approx(np.linalg.norm(g0), rel=1e-13)
    assert d["g1_norm"] == pytest.approx(np.linalg.norm(g1), rel=1e-13)
    assert d["cos_g0_gslow"] == pytest.approx(np.dot(g0, gs) / np.linalg.norm(g0) / np.linalg.norm(gs), rel=1e-12)
    assert d["ratio_mean"] == pytest.approx(np.mean(r), rel=1e-12)
    assert d["ratio_std"] == pytest.approx(np.std(r), rel=1e-11)
    scale = np.ones(n)
    scale[act] = sum(r ** k for k in range(5)) / (1 + r)
    assert d["scale_mean"] == pytest.approx(np.mean(scale), rel=1e-12)
    assert d["disp_ratio"] == pytest.approx(np.linalg.norm((th2 - th0) * scale) / np.linalg.norm(th2 - th0), rel=1e-12)
    assert d["inactive_frac"] == pytest.approx(1 - act.mean(), abs=1e-15) and d["n_active"] == act.sum()


def test_degenerate_cases():
    th0, th2 = f64(0.0, 0.0, 0.0), f64(1.0, 2.0, 3.0)
    # K = 2: every scale is 1, the extrapolated displacement is the observed one
    d = ora.active_diagnostics(th0, th2, f64(1.0, 2.0, 3.0), f64(0.5, -0.7, 9.0), f64(1.0, 2.0, 3.0), K=2, delta=0.0)
    assert d["scale_mean"] == 1.0 and d["disp_ratio"] == 1.0 and d["cos_g0_gslow"] == pytest.approx(1.0, rel=1e-15)
    # nothing active: no ratio, scale 1
    d = ora.active_diagnostics(th0, th2, f64(0.0, 0.0, 0.0), f64(1.0, 1.0, 1.0), f64(1.0, 0.0, 0.0), K=5, delta=1e-8)
    assert d["inactive_frac"] == 1.0 and d["scale_mean"] == 1.0 and math.isnan(d["ratio_mean"]) and math.isnan(d["cos_g0_gslow"])
    # orthogonal gradients; the pole r = -1 is irregular (its scale is not finite) and left out
    d = ora.active_diagnostics(th0, th2, f64(1.0, 1.0, 0.0), f64(-1.0, 0.5, 0.0), f64(0.0, 0.0, 2.0), K=5, delta=1e-8)
    assert d["cos_g0_gslow"] == 0.0 and d["n_irregular"] == 1 and d["n_active"] == 2
    assert d["ratio_mean"] == 0.5 and d["ratio_std"] == 0.0
    s = (1 + 0.5 + 0.25 + 0.125 + 0.0625) / 1.5
    assert d["scale_mean"] == pytest.approx((s + 1.0) / 2, rel=1e-15)      # coordinates 1 and 2
    assert d["disp_ratio"] == pytest.approx(math.sqrt((2 * s) ** 2 + 9) / math.sqrt(4 + 9), rel=1e-15)
    # a ratio too large for float32 is irregular as well
    d = ora.active_diagnostics(th0, th2, f64(1e-30, 1.0, 1.0), f64(1e30, 0.5, 0.5), f64(1.0, 1.0, 1.0), K=3, delta=0.0)
    assert d["n_irregular"] == 1 and d["ratio_mean"] == 0.5
