"""Pins for the CPU oracle: it is checked against what the paper and the
mathematics fix, never against itself and never against the CUDA path.

  * Corollary 1 / Appendix A.6: diagonal quadratic + plain GD + alpha = 1 makes
    the extrapolated point the K-th GD iterate and the new point the (K+1)-th.
  * brute force: K explicit GD steps written as Python loops.
  * identities of the scale factor (Eq. (scale_factor), Eq. (geom_sum_def)).
  * AdamW: a library AdamW in float64, and the closed form of its first step.
  * norm: closed forms and a library norm.
"""
import math

import numpy as np
import pytest

from oracle import gxpo_oracle as ora
from paper_2605_06755_b200 import workloads


def quad_grad_fn(a, b):
    a64, b64 = a.astype(np.float64), b.astype(np.float64)
    return lambda which, theta: a64 * theta - b64


# ---------------------------------------------------------------------------
# Corollary 1: closed form on the diagonal-quadratic surrogate (BASELINE config 0)
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("K", [2, 3, 5, 10])
@pytest.mark.parametrize("alpha", [1.0, 0.5, 0.1, 0.0])
def test_closed_form_diagonal_quadratic(K, alpha):
    n, eta = 4096, 0.1
    a, b, theta0 = workloads.quadratic_surrogate(n, seed=0)
    a64, b64, t64 = (x.astype(np.float64) for x in (a, b, theta0))
    star = b64 / a64
    r = 1.0 - eta * a64
    st = ora.State(theta0, ora.OptCfg(kind="gd", lr=eta))
    cfg = ora.GxpoCfg(K=K, alpha=alpha, delta=1e-8)
    trace = {}
    nrm = ora.active_step(st, cfg, quad_grad_fn(a, b), round_f32=False, trace=trace)
    assert np.all(np.abs(a64 * t64 - b64) > 1e-8)          # every coordinate active
    # the two probes are GD iterates 1 and 2
    np.testing.assert_allclose(trace["theta1"], star + r * (t64 - star), rtol=0, atol=1e-12)
    np.testing.assert_allclose(trace["theta2"], star + r**2 * (t64 - star), rtol=0, atol=1e-12)
    # extrapolated point = K-th GD iterate (Appendix A.6)
    np.testing.assert_allclose(trace["theta_K"], star + r**K * (t64 - star), rtol=0, atol=1e-10)
    # repositioned point for general alpha (Eq. (blend_step) applied to the above)
    blend = 1.0 - alpha + alpha * r**K
    np.testing.assert_allclose(trace["theta_tilde"], star + blend * (t64 - star), rtol=0, atol=1e-10)
    # slow correction: one more GD step from theta-tilde
    np.testing.assert_allclose(st.theta, star + r * blend * (t64 - star), rtol=0, atol=1e-10)
    if alpha == 1.0:
        np.testing.assert_allclose(st.theta, star + r**(K + 1) * (t64 - star), rtol=0, atol=1e-10)
    # ||g_slow|| where g_slow = a (theta_tilde - theta*)
    want = math.sqrt(float(np.sum((a64 * blend * (t64 - star))**2)))
    assert nrm == pytest.approx(want, rel=1e-12)


def test_m_active_steps_equal_m_times_K_plus_1_gd_steps():
    n, eta, K, m_steps = 512, 0.1, 5, 20
    a, b, theta0 = workloads.quadratic_surrogate(n, seed=3)
    a64, b64, t64 = (x.astype(np.float64) for x in (a, b, theta0))
    star, r = b64 / a64, 1.0 - eta * a64
    st = ora.State(theta0, ora.OptCfg(kind="gd", lr=eta))
    cfg = ora.GxpoCfg(K=K, alpha=1.0, delta=0.0)
    for s in range(1, m_steps + 1):
        ora.active_step(st, cfg, quad_grad_fn(a, b))
        np.testing.assert_allclose(st.theta, star + r**((K + 1) * s) * (t64 - star), rtol=0,
                                   atol=1e-9)


@pytest.mark.parametrize("K", [2, 3, 5, 10])
def test_brute_force_K_explicit_gd_steps(K):
    n, eta = 16, 0.1
    a, b, theta0 = workloads.quadratic_surrogate(n, seed=11)
    st = ora.State(theta0, ora.OptCfg(kind="gd", lr=eta))
    trace = {}
    ora.active_step(st, ora.GxpoCfg(K=K, alpha=1.0, delta=1e-8), quad_grad_fn(a, b), trace=trace)
    for i in range(n):                      # plain Python loops, coordinate by coordinate
        x = float(theta0[i])
        for _ in range(K):
            x = x - eta * (float(a[i]) * x - float(b[i]))
        assert trace["theta_K"][i] == pytest.approx(x, abs=1e-12)
        x = x - eta * (float(a[i]) * x - float(b[i]))
        assert st.theta[i] == pytest.approx(x, abs=1e-12)


# ---------------------------------------------------------------------------
# scale factor identities
# ---------------------------------------------------------------------------
def _scale(r, K, delta=1e-8, den_eps=0.0):
    r = np.atleast_1d(np.asarray(r, dtype=np.float64))
    g0 = np.ones_like(r)
    g1 = r.copy()
    z = np.zeros_like(r)
    one = np.ones_like(r)
    # theta0 = 0, theta2 = 1, alpha = 1  ->  theta_tilde = scale
    _, _, sc = ora.extrapolate(z, one, g0, g1, K, 1.0, delta, den_eps, want_aux=True)
    return sc


def test_scale_identities():
    r = np.array([-3.0, -0.5, 0.0, 0.3, 0.9, 1.0, 1.7, 4.0])
    for K in (2, 3, 4, 5, 10):
        np.testing.assert_allclose(_scale(1.0, K), K / 2.0, rtol=1e-15)     # S_K(1) = K
        np.testing.assert_allclose(_scale(0.0, K), 1.0, rtol=1e-15)
    np.testing.assert_allclose(_scale(r, 2), np.ones_like(r), rtol=1e-15)    # K = 2: observed
    np.testing.assert_allclose(_scale(r, 3), 1.0 + r**2 / (1.0 + r), rtol=1e-14)
    np.testing.assert_allclose(_scale(r, 4), 1.0 + r**2, rtol=1e-14)
    rr = r[r != 1.0]
    for K in (3, 5, 10):                    # the simplified form printed under Eq. (scale_factor)
        np.testing.assert_allclose(_scale(rr, K), (1.0 - rr**K) / (1.0 - rr**2), rtol=1e-12)


def test_literal_pole_at_minus_one_and_guard():
    assert np.isposinf(_scale(-1.0, 3)[0])          # S_3(-1) / 0 = 1 / 0
    assert np.isnan(_scale(-1.0, 4)[0])             # 0 / 0
    assert _scale(-1.0, 3, den_eps=1e-6)[0] == 1.0  # guarded: treated as inactive
    assert _scale(-1.0 + 1e-7, 3, den_eps=1e-6)[0] == 1.0
    assert _scale(-1.0 + 1e-3, 3, den_eps=1e-6)[0] != 1.0


def test_active_set_is_strict_and_inactive_keeps_two_probe_displacement():
    delta = 1e-3
    g0 = np.array([1e-3, -1e-3, 1.0000001e-3, 0.0, 5e-4, -2.0])
    g1 = np.array([7.0, 7.0, 2e-3, 3.0, 1.0, -1.0])
    theta0 = np.linspace(-1, 1, 6)
    theta2 = theta0 + np.array([0.1, -0.2, 0.3, 0.4, -0.5, 0.6])
    K, alpha = 5, 0.5
    tilde, tk, sc = ora.extrapolate(theta0, theta2, g0, g1, K, alpha, delta, want_aux=True)
    assert list(sc[[0, 1, 3, 4]]) == [1.0] * 4        # |g0| == delta is NOT active
    assert sc[2] != 1.0 and sc[5] != 1.0
    np.testing.assert_allclose(tk[[0, 1, 3, 4]], theta2[[0, 1, 3, 4]], rtol=1e-14)
    np.testing.assert_allclose(tilde, theta0 + alpha * (tk - theta0), rtol=1e-15)
    # inactive coordinates under GD keep -eta (g0 + g1): run the whole step
    eta = 0.25
    st = ora.State(theta0, ora.OptCfg(kind="gd", lr=eta))
    grads = [g0, g1, np.zeros(6)]
    trace = {}
    ora.active_step(st, ora.GxpoCfg(K=K, alpha=1.0, delta=delta), lambda w, th: grads[w],
                    trace=trace)
    np.testing.assert_allclose(trace["theta_K"][[0, 1, 3, 4]],
                               (theta0 - eta * (g0 + g1))[[0, 1, 3, 4]], rtol=1e-15)


def test_alpha_endpoints():
    rng = np.random.default_rng(5)
    theta0, theta2 = rng.standard_normal(64), rng.standard_normal(64)
    g0, g1 = rng.standard_normal(64), rng.standard_normal(64)
    t0, tk, _ = ora.extrapolate(theta0, theta2, g0, g1, 5, 0.0, 1e-8, want_aux=True)
    np.testing.assert_array_equal(t0, theta0)                     # alpha = 0 ignores it
    t1, tk, _ = ora.extrapolate(theta0, theta2, g0, g1, 5, 1.0, 1e-8, want_aux=True)
    np.testing.assert_allclose(t1, tk, rtol=1e-14)                # alpha = 1 adopts it


def test_round_f32_rounds_once_at_the_boundary():
    rng = np.random.default_rng(6)
    theta0, theta2 = rng.standard_normal(256), rng.standard_normal(256)
    g0, g1 = rng.standard_normal(256), rng.standard_normal(256)
    exact = ora.extrapolate(theta0, theta2, g0, g1, 5, 0.5, 1e-8)
    rounded = ora.extrapolate(theta0, theta2, g0, g1, 5, 0.5, 1e-8, round_f32=True)
    np.testing.assert_array_equal(rounded, exact.astype(np.float32).astype(np.float64))


# ---------------------------------------------------------------------------
# AdamW against a library routine and a closed form
# ---------------------------------------------------------------------------
def test_adamw_matches_library_float64():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(7)
    n = 1000
    theta = rng.standard_normal(n)
    opt = ora.OptCfg(kind="adamw", lr=3e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    p = torch.nn.Parameter(torch.tensor(theta, dtype=torch.float64))
    lib_opt = torch.optim.AdamW([p], lr=opt.lr, betas=(opt.beta1, opt.beta2), eps=opt.eps,
                                weight_decay=opt.weight_decay)
    st = ora.State(theta, opt)
    for step in range(5):
        g = rng.standard_normal(n) * 10.0 ** rng.integers(-6, 1, size=n)
        p.grad = torch.tensor(g, dtype=torch.float64)
        lib_opt.step()
        st.optim_step(ora.as_f64(g), round_f32=False)
        assert st.t_opt == step + 1
        s = lib_opt.state[p]
        np.testing.assert_allclose(st.theta, p.detach().numpy(), rtol=1e-12, atol=1e-15)
        np.testing.assert_allclose(st.m, s["exp_avg"].numpy(), rtol=1e-12, atol=1e-300)
        np.testing.assert_allclose(st.v, s["exp_avg_sq"].numpy(), rtol=1e-12, atol=1e-300)


def test_adamw_first_step_is_sign_step():
    # from m = v = 0 with no decay: m_hat = g, v_hat = g^2, update = lr g / (|g| + eps)
    g = np.array([3.0, -0.5, 1e-3, -20.0])
    theta = np.array([1.0, 2.0, -3.0, 0.25])
    opt = ora.OptCfg(kind="adamw", lr=0.1, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0)
    st = ora.State(theta, opt)
    st.optim_step(g, round_f32=False)
    np.testing.assert_allclose(st.theta, theta - 0.1 * g / (np.abs(g) + 1e-8), rtol=1e-12)
    np.testing.assert_allclose(st.m, 0.1 * g, rtol=1e-12)
    np.testing.assert_allclose(st.v, 0.001 * g * g, rtol=1e-12)


def test_adamw_weight_decay_is_decoupled():
    # zero gradient from zero state: only the decay acts, theta <- theta (1 - lr wd)
    theta = np.array([2.0, -4.0])
    opt = ora.OptCfg(kind="adamw", lr=0.5, weight_decay=0.1)
    st = ora.State(theta, opt)
    st.optim_step(np.zeros(2), round_f32=False)
    np.testing.assert_allclose(st.theta, theta * 0.95, rtol=1e-15)


def test_active_step_advances_optimizer_state_three_times():
    rng = np.random.default_rng(8)
    n = 64
    opt = ora.OptCfg(kind="adamw", lr=1e-3)
    st = ora.State(rng.standard_normal(n), opt)
    gs = [rng.standard_normal(n) for _ in range(3)]
    ora.active_step(st, ora.GxpoCfg(K=5, alpha=0.5), lambda w, th: gs[w])
    assert st.t_opt == 3
    # moments are those of three plain AdamW updates with g0, g1, g_slow (never rewound)
    m = np.zeros(n)
    v = np.zeros(n)
    for g in gs:
        m = 0.9 * m + (1 - 0.9) * g
        v = 0.999 * v + (1 - 0.999) * g * g
    np.testing.assert_allclose(st.m, m, rtol=1e-13)
    np.testing.assert_allclose(st.v, v, rtol=1e-13)


def test_adamw_active_steps_against_library_optimizer_with_manual_reposition():
    """Algorithm 1's active branch with the library's AdamW as OptimStep: two fast steps,
    the parameters repositioned by hand with the closed form (1 - r^K) / (1 - r^2) of
    Eq. (scale_factor), the third step with g_slow; optimizer state never rewound.  Two
    consecutive active steps, float64."""
    import torch
    rng = np.random.default_rng(21)
    n, K, alpha, delta = 200, 5, 0.5, 1e-8
    theta0 = rng.standard_normal(n)
    opt = ora.OptCfg(kind="adamw", lr=1e-2, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    st = ora.State(theta0, opt)
    p = torch.nn.Parameter(torch.from_numpy(theta0.copy()))
    lib = torch.optim.AdamW([p], lr=1e-2, betas=(0.9, 0.999), eps=1e-8, weight_decay=0.01)
    for step in range(2):
        g0 = rng.standard_normal(n)
        g0[::17] = 0.0                                  # some inactive coordinates
        g1 = g0 * rng.uniform(0.3, 1.3, n) + (g0 == 0) * 0.5
        gs = rng.standard_normal(n)
        grads = [g0, g1, gs]
        nrm = ora.active_step(st, ora.GxpoCfg(K=K, alpha=alpha, delta=delta), lambda w, th: grads[w])
        start = p.detach().numpy().copy()
        for g in (g0, g1):
            p.grad = torch.from_numpy(g.copy())
            lib.step()
        th2 = p.detach().numpy().copy()
        act = np.abs(g0) > delta
        r = np.where(act, g1 / np.where(act, g0, 1.0), 0.0)
        scale = np.where(act, (1 - r ** K) / (1 - r ** 2), 1.0)
        with torch.no_grad():
            p.copy_(torch.from_numpy(start + alpha * (th2 - start) * scale))
        p.grad = torch.from_numpy(gs.copy())
        lib.step()
        np.testing.assert_allclose(st.theta, p.detach().numpy(), rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(st.m, lib.state[p]["exp_avg"].numpy(), rtol=1e-12, atol=1e-15)
        np.testing.assert_allclose(st.v, lib.state[p]["exp_avg_sq"].numpy(), rtol=1e-12, atol=1e-18)
        assert nrm == pytest.approx(np.linalg.norm(gs), rel=1e-14)
    assert st.t_opt == 6 and int(lib.state[p]["step"]) == 6


# ---------------------------------------------------------------------------
# norm
# ---------------------------------------------------------------------------
def test_norm_closed_forms_and_library():
    assert ora.l2norm(np.array([3.0, 4.0])) == 5.0
    n, c = 10000, -0.37
    assert ora.l2norm(np.full(n, c)) == pytest.approx(abs(c) * math.sqrt(n), rel=1e-13)
    x = np.random.default_rng(9).standard_normal(100003)
    assert ora.l2norm(x) == pytest.approx(float(np.linalg.norm(x)), rel=1e-13)
    assert ora.l2norm(8.0 * x) == pytest.approx(8.0 * ora.l2norm(x), rel=1e-15)
    assert ora.l2norm(np.zeros(0)) == 0.0


def test_bf16_conversion_helpers_are_exact():
    x = np.array([1.0, -2.5, 3.140625, 1e-3, 0.0, -0.0, 65504.0], dtype=np.float32)
    bits = workloads.f32_to_bf16_bits(x)
    back = workloads.bf16_bits_to_f32(bits)
    # bf16 keeps 8 significand bits: relative error <= 2^-9, and the round trip is idempotent
    assert np.all(np.abs(back - x) <= np.abs(x) * 2.0**-8)
    np.testing.assert_array_equal(workloads.f32_to_bf16_bits(back), bits)
    np.testing.assert_array_equal(ora.bf16_bits_to_f64(bits), back.astype(np.float64))
    # ties go to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    tie = np.array([1.0 + 2.0**-8, 1.0 + 3 * 2.0**-8], dtype=np.float32)
    np.testing.assert_array_equal(workloads.bf16_bits_to_f32(workloads.f32_to_bf16_bits(tie)),
                                  np.array([1.0, 1.0 + 2.0**-6], dtype=np.float32))


def test_clip_coefficient_matches_the_library_routine():
    """Global-norm clipping against torch.nn.utils.clip_grad_norm_ (float64, CPU)."""
    import torch
    rng = np.random.default_rng(11)
    for scale, max_norm in [(1.0, 1.0), (1e-3, 1.0), (5.0, 0.3), (1.0, 100.0)]:
        gs = [scale * rng.standard_normal(n) for n in (7, 100, 1)]
        ps = [torch.nn.Parameter(torch.zeros(g.size, dtype=torch.float64)) for g in gs]
        for p, g in zip(ps, gs):
            p.grad = torch.from_numpy(g.copy())
        total = float(torch.nn.utils.clip_grad_norm_(ps, max_norm))
        norm = math.sqrt(sum(ora.sum_squares(np.ascontiguousarray(g)) for g in gs))
        assert norm == pytest.approx(total, rel=1e-14)
        c = ora.clip_coef(norm, max_norm)
        for p, g in zip(ps, gs):
            np.testing.assert_allclose(p.grad.numpy(), g * c, rtol=1e-14, atol=0)
        assert (c == 1.0) == (max_norm / (norm + 1e-6) >= 1.0)
    assert ora.clip_coef(0.0, 1.0) == 1.0 and ora.clip_coef(2.0, 1.0) == pytest.approx(1 / (2 + 1e-6), rel=1e-15)


def test_bf16_rounding_matches_the_library_conversion():
    """Round-to-nearest-even float32 -> bfloat16 against torch's conversion, on random
    values, exact ties, the largest finite values, subnormals, zeros and infinities."""
    import torch
    rng = np.random.default_rng(12)
    x = np.concatenate([
        rng.standard_normal(20000).astype(np.float32) * np.float32(0.02),
        (rng.standard_normal(2000) * 1e30).astype(np.float32),
        np.array([0.0, -0.0, np.inf, -np.inf, 3.4028235e38, -3.4028235e38, 1e-40, -1e-45, 1.0, -1.0], dtype=np.float32),
        # exact ties: patterns ending in 0x8000 after an even and after an odd upper half
        np.array([0x3F808000, 0x3F818000, 0xBF808000, 0x7F7F8000, 0x00008000, 0x00018000], dtype=np.uint32).view(np.float32),
    ])
    got = ora.round_to_bf16(x.astype(np.float64))
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(got, want)
    # ties go to even; the largest float32 rounds up to infinity
    assert got[-6] == 0x3F80 and got[-5] == 0x3F82 and got[-3] == 0x7F80
    nan = ora.round_to_bf16(np.array([np.nan]))
    assert (nan[0] & 0x7F80) == 0x7F80 and (nan[0] & 0x007F) != 0


# ---------------------------------------------------------------------------
# invariances the mathematics fixes (no value is taken from any implementation)
# ---------------------------------------------------------------------------
def test_geometric_sum_recurrence_links_consecutive_depths():
    """S_{K+1}(r) = 1 + r S_K(r) (Eq. (geom_sum_def)), and scale_K (1 + r) = S_K(r): the oracle's
    scale factors for consecutive K must satisfy scale_{K+1} (1+r) = 1 + r scale_K (1+r).  A wrong
    loop bound, a dropped term or a swapped numerator/denominator breaks it for some K."""
    rng = np.random.default_rng(5)
    r = np.concatenate([rng.uniform(-0.95, 2.5, 200), [-3.0, 0.0, 1.0, 7.5]])
    for K in range(2, 12):
        sk, sk1 = _scale(r, K), _scale(r, K + 1)
        np.testing.assert_allclose(sk1 * (1.0 + r), 1.0 + r * sk * (1.0 + r), rtol=1e-11, atol=1e-12)


def test_extrapolation_depends_on_the_gradients_only_through_their_ratio_and_is_linear_in_the_displacement():
    rng = np.random.default_rng(6)
    n = 300
    th0 = rng.standard_normal(n)
    d = 1e-2 * rng.standard_normal(n)
    g0 = rng.standard_normal(n)
    g1 = g0 * rng.uniform(-0.8, 1.6, n)
    for K in (3, 5, 10):
        base = ora.extrapolate(th0, th0 + d, g0, g1, K, 0.5, 1e-8)
        for c in (1e-3, 7.0):                    # (g0, g1) -> (c g0, c g1): same ratio, same active set
            same = ora.extrapolate(th0, th0 + d, c * g0, c * g1, K, 0.5, 1e-8 * min(c, 1.0))
            np.testing.assert_allclose(same, base, rtol=1e-12, atol=1e-15)
        dbl = ora.extrapolate(th0, th0 + 2.0 * d, g0, g1, K, 0.5, 1e-8)      # Eq. (blend_step): linear in theta2 - theta0
        np.testing.assert_allclose(dbl - th0, 2.0 * (base - th0), rtol=1e-11, atol=1e-15)
        neg = ora.extrapolate(th0, th0 + d, -g0, -g1, K, 0.5, 1e-8)          # a common sign drops out of g1 / g0
        np.testing.assert_allclose(neg, base, rtol=1e-13, atol=0)


def test_adam_update_is_invariant_to_the_scale_of_the_gradients_when_eps_is_zero():
    """m / sqrt(v) is homogeneous of degree zero in the gradient history: with eps = 0 and no weight
    decay, multiplying every gradient by c > 0 leaves every parameter where it was (the textbook
    scale invariance of Adam).  It pins the pairing of m with sqrt(v), both bias corrections and
    the place of eps."""
    rng = np.random.default_rng(7)
    n, steps = 64, 6
    grads = [rng.standard_normal(n) for _ in range(steps)]
    outs = []
    for c in (1.0, 1e-4, 3e3):
        opt = ora.OptCfg(kind="adamw", lr=1e-2, eps=0.0, weight_decay=0.0)
        st = ora.State(np.linspace(-1.0, 1.0, n), opt)
        for g in grads:
            st.optim_step(c * g, False)
        outs.append(st.theta.copy())
    np.testing.assert_allclose(outs[1], outs[0], rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(outs[2], outs[0], rtol=1e-11, atol=1e-13)
    # and with eps > 0 the invariance must break in the expected direction: tiny gradients move less
    opt = ora.OptCfg(kind="adamw", lr=1e-2, eps=1e-3, weight_decay=0.0)
    small, big = ora.State(np.zeros(n), opt), ora.State(np.zeros(n), opt)
    small.optim_step(1e-4 * grads[0], False)
    big.optim_step(grads[0], False)
    assert np.all(np.abs(small.theta) < np.abs(big.theta))
