"""Parity of the CUDA library (through its C ABI) against the CPU oracle,
element by element on the same seeded inputs.  Sizes span several 2048-element
tiles, several 32768-element chunks and ragged tails."""
import math

import numpy as np
import pytest

from oracle import gxpo_oracle as ora
from paper_2605_06755_b200 import workloads
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

SIZES = [1, 7, 8, 2048, 2049, 40003, 3 * 32768 + 5]


def _binding():
    from paper_2605_06755_b200 import binding
    return binding


def _problem(n, seed, grad_dtype, warm=True, zero_frac=0.0, offset=0):
    th, m, v, g0, g1, gs = workloads.llm_inputs_numpy(n, seed, grad_dtype, zero_frac, warm)
    return gu.Problem(th, m, v, g0, g1, gs, offset_elems=offset)


def _ctx(b, grad_dtype, **kw):
    cfg, opt = b.make_cfg(**kw)
    return b.Context(cfg, opt, b.BF16 if grad_dtype == "bf16" else b.F32), cfg, opt


@pytest.mark.parametrize("n", SIZES)
@pytest.mark.parametrize("grad_dtype", ["bf16", "f32"])
@pytest.mark.parametrize("kind", ["adamw", "gd"])
@pytest.mark.parametrize("placement", [0, 1])
def test_active_step_matches_oracle(n, grad_dtype, kind, placement):
    b = _binding()
    import torch
    pr = _problem(n, seed=100 + n, grad_dtype=grad_dtype)
    ctx, cfg, opt = _ctx(b, grad_dtype, kind=b.OPT_ADAMW if kind == "adamw" else b.OPT_GD,
                         lr=1e-3, K=5, alpha=0.5, placement=placement)
    gcfg, ocfg = gu.ora_cfgs(cfg, opt)
    ctx.bind([pr.ptrs()])
    st = pr.oracle_state(ocfg, t_opt=0)
    grads = pr.oracle_grads()

    # the oracle, step by step
    theta0 = st.theta.copy()
    st.optim_step(grads[0], True)
    o_theta1, o_m1, o_v1 = st.theta.copy(), None if st.m is None else st.m.copy(), None if st.v is None else st.v.copy()
    st.optim_step(grads[1], True)
    o_theta2 = st.theta.copy()
    o_tilde, _, o_scale = ora.extrapolate(theta0, o_theta2, grads[0], grads[1], gcfg.K, gcfg.alpha,
                                          gcfg.delta, gcfg.den_eps, True, want_aux=True)
    sat = ~np.isfinite(o_scale) | (np.abs(o_scale) > 1e30)
    st.theta = o_tilde.copy()
    st.optim_step(grads[2], True)
    o_norm = ora.l2norm(grads[2])

    # the library, call by call
    ctx.probe_step(0)
    live1 = pr.work if placement == 0 else pr.theta
    gu.assert_close(gu.to_host_f64(live1), o_theta1, "theta1")
    if placement == 1:
        np.testing.assert_array_equal(gu.to_host_f64(pr.work), theta0)      # snapshot of theta^t
    else:
        np.testing.assert_array_equal(gu.to_host_f64(pr.theta), theta0)     # theta^t untouched
    if kind == "adamw":
        gu.assert_close(gu.to_host_f64(pr.m), o_m1, "m after probe 0")
        gu.assert_close(gu.to_host_f64(pr.v), o_v1, "v after probe 0")
    ctx.probe_step(1)
    # theta2 starts from the library's own theta1 (within an ulp of the oracle's)
    gu.assert_close(gu.to_host_f64(live1), o_theta2, "theta2", rtol=2e-6)
    ctx.extrapolate()
    # chained: (theta2 - theta0) cancels, the scale factor amplifies theta2's last-ulp
    # differences; the strict per-call check is test_extrapolate_call_alone
    slack = gu.displacement_slack(theta0, o_theta2, o_scale, gcfg.alpha)
    gu.assert_close(gu.to_host_f64(pr.theta), o_tilde, "theta-tilde", saturated=sat, extra_abs=slack)
    ctx.slow_step()
    res = ctx.gate_update(allow_nonfinite=True)
    torch.cuda.synchronize()
    gu.assert_close(gu.to_host_f64(pr.theta), st.theta, "theta after slow step", saturated=sat,
                    rtol=2e-6, extra_abs=slack)
    if kind == "adamw":
        gu.assert_close(gu.to_host_f64(pr.m), st.m, "m after slow step")
        gu.assert_close(gu.to_host_f64(pr.v), st.v, "v after slow step")
    assert res.norm == pytest.approx(o_norm, rel=gu.RTOL_NORM)
    assert ctx.optimizer_steps() == 3 and res.t == 1 and res.active == 1
    assert math.isnan(res.z)
    ctx.close()


def _run_extrapolate_alone(b, theta0, theta2, g0d, g1d, grad_dtype, kind, placement, **kw):
    """gxpo_extrapolate on given theta^t and theta^{t,2}: the library's own probe
    steps with lr = 0 are identities and put the context in the right state; the
    two points are then written where the placement expects them."""
    n = theta0.size
    dummy = np.zeros(n, dtype=np.float32)
    pr = gu.Problem(theta0, dummy if kind == "adamw" else None, dummy if kind == "adamw" else None,
                    g0d, g1d, g0d)
    ctx, cfg, opt = _ctx(b, grad_dtype, kind=b.OPT_ADAMW if kind == "adamw" else b.OPT_GD, lr=0.0,
                         weight_decay=0.0, placement=placement, **kw)
    ctx.bind([pr.ptrs()])
    ctx.probe_step(0)
    ctx.probe_step(1)
    if placement == 0:
        pr.theta.copy_(gu.to_dev(theta0)); pr.work.copy_(gu.to_dev(theta2))
    else:
        pr.theta.copy_(gu.to_dev(theta2)); pr.work.copy_(gu.to_dev(theta0))
    ctx.extrapolate()
    got = gu.to_host_f64(pr.theta)
    ctx.close()
    return got


@pytest.mark.parametrize("K", [3, 5, 10])
@pytest.mark.parametrize("grad_dtype", ["bf16", "f32"])
@pytest.mark.parametrize("placement", [0, 1])
def test_extrapolate_call_alone(K, grad_dtype, placement):
    """Strict 1e-6 check of the extrapolation call on seeded theta^t, theta^{t,2}, g0, g1
    with the heavy-tailed ratios of the LLM-shaped recipe, 3 % inactive coordinates."""
    b = _binding()
    n = 2 * 32768 + 1234
    th, _, _, g0, g1, _ = workloads.llm_inputs_numpy(n, seed=900 + K, grad_dtype=grad_dtype, zero_frac=0.03)
    rng = np.random.default_rng(K)
    theta2 = (th + 2e-3 * rng.standard_normal(n)).astype(np.float32)
    got = _run_extrapolate_alone(b, th, theta2, g0, g1, grad_dtype, "adamw", placement, K=K, alpha=0.5)
    want, _, scale = ora.extrapolate(th.astype(np.float64), theta2.astype(np.float64), gu.grad_to_f64(g0),
                                     gu.grad_to_f64(g1), K, 0.5, 1e-8, 0.0, True, want_aux=True)
    sat = ~np.isfinite(scale) | (np.abs(scale) > 1e30)
    gu.assert_close(got, want, f"theta-tilde K={K}", saturated=sat)
    assert 0.02 < (scale == 1.0).mean() < 0.05


@pytest.mark.parametrize("K", [2, 3, 4, 5, 10])
@pytest.mark.parametrize("grad_dtype", ["bf16", "f32"])
def test_extrapolate_edge_values(K, grad_dtype):
    """r = +-1, |g0| = delta exactly, zeros, huge and tiny ratios, negative ratios."""
    b = _binding()
    delta = np.float32(2.0 ** -20)                      # exact in bfloat16 too
    g0 = np.array([1.0, 1.0, delta, -delta, 0.0, 2.0 ** -19, 1.0, -1.0, 2.0 ** -19, 0.5, 3.0, -0.25,
                   1.0, 1.0, 2.0, 1.0], dtype=np.float32)
    g1 = np.array([1.0, -1.0, 5.0, 5.0, 1.0, 2.0 ** 10, 0.0, -0.99609375, -2.0 ** 12, 0.4375, -3.0, 0.75,
                   -0.9921875, -1.0078125, -1.0, 1.5], dtype=np.float32)
    rng = np.random.default_rng(K)
    reps = 700                                          # 11200 elements: several tiles
    g0 = np.tile(g0, reps)
    g1 = np.tile(g1, reps)
    n = g0.size
    theta0 = rng.standard_normal(n).astype(np.float32)
    theta2 = (theta0 + 1e-2 * rng.standard_normal(n)).astype(np.float32)
    if grad_dtype == "bf16":
        g0d, g1d = workloads.f32_to_bf16_bits(g0), workloads.f32_to_bf16_bits(g1)
        np.testing.assert_array_equal(workloads.bf16_bits_to_f32(g0d), g0)   # all exact in bf16
        np.testing.assert_array_equal(workloads.bf16_bits_to_f32(g1d), g1)
    else:
        g0d, g1d = g0, g1
    for den_eps in (0.0, 2.0 ** -6):
        # place theta^t in `theta` and theta^{t,2} in `work` (PINGPONG layout) by hand:
        # run the library's own probe steps with lr = 0 so that they are identities
        pr = gu.Problem(theta0, None, None, g0d, g1d, g0d)
        ctx, cfg, opt = _ctx(b, grad_dtype, kind=b.OPT_GD, lr=0.0, K=K, alpha=0.5, delta=float(delta),
                             den_eps=den_eps)
        ctx.bind([pr.ptrs()])
        ctx.probe_step(0)
        ctx.probe_step(1)
        pr.work.copy_(gu.to_dev(theta2))
        ctx.extrapolate()
        want, _, scale = ora.extrapolate(theta0.astype(np.float64), theta2.astype(np.float64),
                                         g0.astype(np.float64), g1.astype(np.float64), K, 0.5,
                                         float(delta), den_eps, True, want_aux=True)
        sat = ~np.isfinite(scale) | (np.abs(scale) > 1e30)
        got = gu.to_host_f64(pr.theta)
        gu.assert_close(got, want, f"K={K} den_eps={den_eps}", saturated=sat)
        # r = -1 with the literal formula: both sides non-finite
        if den_eps == 0.0:
            assert not np.isfinite(want[1]) and not np.isfinite(got[1])
            assert np.all(np.isfinite(got[2:5]))       # |g0| <= delta: scale 1, finite
        else:
            assert np.isfinite(got[1]) and np.isfinite(got[12])   # guarded: scale 1
        ctx.close()


def test_multi_tensor_list_with_odd_sizes_and_misaligned_tensors():
    b = _binding()
    sizes = [512, 3584, 1, 70001, 2 * 32768, 33, 32768 + 2047, 5]
    offsets = [0, 0, 0, 1, 0, 3, 2, 0]                  # element offsets -> misaligned pointers
    probs = [_problem(n, seed=7 + i, grad_dtype="bf16", zero_frac=0.03, offset=off)
             for i, (n, off) in enumerate(zip(sizes, offsets))]
    ctx, cfg, opt = _ctx(b, "bf16", lr=1e-3, K=10, alpha=0.5)
    gcfg, ocfg = gu.ora_cfgs(cfg, opt)
    ctx.bind([p.ptrs() for p in probs])
    res = ctx.active_step(allow_nonfinite=True)
    sumsq = 0.0
    for i, p in enumerate(probs):
        st = p.oracle_state(ocfg)
        grads = p.oracle_grads()
        trace = {}
        ora.active_step(st, gcfg, lambda w, th: grads[w], round_f32=True, trace=trace)
        sat = ~np.isfinite(trace["scale"]) | (np.abs(trace["scale"]) > 1e30)
        slack = gu.displacement_slack(p.np_in["theta"].astype(np.float64), trace["theta2"],
                                      trace["scale"], gcfg.alpha)
        gu.assert_close(gu.to_host_f64(p.theta), st.theta, f"tensor {i} theta", saturated=sat,
                        rtol=2e-6, extra_abs=slack)
        gu.assert_close(gu.to_host_f64(p.m), st.m, f"tensor {i} m")
        gu.assert_close(gu.to_host_f64(p.v), st.v, f"tensor {i} v")
        sumsq += ora.sum_squares(grads[2])
        if p.n >= 3584:
            assert (trace["scale"] == 1.0).mean() > 0.01    # the inactive branch was exercised
    assert res.norm == pytest.approx(math.sqrt(sumsq), rel=gu.RTOL_NORM)
    ctx.close()


def test_empty_list_and_empty_tensor():
    b = _binding()
    ctx, cfg, opt = _ctx(b, "bf16")
    ctx.bind([])
    res = ctx.active_step()
    assert res.norm == 0.0 and res.t == 1
    pr = _problem(100, 1, "bf16")
    empty = b.TensorPtrs(0, 0, 0, 0, 0, 0, 0, 0)
    before = gu.to_host_f64(pr.theta)
    ctx.bind([empty, pr.ptrs(), empty])
    res = ctx.active_step()
    assert res.norm == pytest.approx(ora.l2norm(pr.oracle_grads()[2]), rel=gu.RTOL_NORM)
    assert not np.array_equal(gu.to_host_f64(pr.theta), before)
    ctx.close()


def test_access_variants_and_launch_shapes_agree_bitwise():
    b = _binding()
    n = 5 * 32768 + 77
    outs = []
    for variant, ctas, unit in [(1, 0, 0), (2, 0, 0), (2, 1, 1), (1, 7, 4), (2, 3, 16), (2, 2, 2), (3, 0, 0)]:
        pr = _problem(n, seed=42, grad_dtype="bf16")
        ctx, cfg, opt = _ctx(b, "bf16", lr=1e-3, K=5)
        ctx.tune(ctas, variant, unit)
        ctx.bind([pr.ptrs()])
        res = ctx.active_step(allow_nonfinite=True)
        outs.append((gu.to_host_f64(pr.theta), gu.to_host_f64(pr.m), gu.to_host_f64(pr.v), res.norm))
        ctx.close()
    for o in outs[1:]:
        for a, c in zip(o[:3], outs[0][:3]):
            np.testing.assert_array_equal(a, c)
        # the norm's float32 partial sums group 4 or 8 squares depending on the access width
        assert o[3] == pytest.approx(outs[0][3], rel=1e-7)


def test_run_to_run_determinism_with_bf16_only_probe_points():
    """The recomputing slow sweep sums sum(g_slow^2) in a fixed order as well."""
    import torch
    b = _binding()
    n = 5 * 32768 + 4096 + 11
    got = []
    for _ in range(2):
        pr = _problem(n, seed=5, grad_dtype="bf16")
        ctx, cfg, opt = _ctx(b, "bf16", lr=1e-3)
        ctx.bind([pr.ptrs()])
        wb = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
        ctx.bind_model_weights([wb.data_ptr()], bf16_only=b.BF16_ONLY_PROBE_POINTS)
        ctx.set_gradients_persist(True)
        res = [ctx.active_step(allow_nonfinite=True, deferred=True).norm for _ in range(2)]
        got.append((gu.to_host_f64(pr.theta), gu.to_host_f64(pr.m), gu.to_host_f64(wb), res))
        ctx.close()
    for x, y in zip(got[0][:3], got[1][:3]):
        np.testing.assert_array_equal(x, y)
    assert got[0][3] == got[1][3]


@pytest.mark.parametrize("staged", [False, True])
def test_run_to_run_determinism(staged):
    """Two runs on the same bits give the same bits, the norm included: the reductions have a
    fixed order for a fixed launch shape (register-staged sweeps; and the shared-memory
    staged ones under the gradients-persist promise, diagnostics included in a second step)."""
    b = _binding()
    n = 5 * 32768 + 4096 + 11
    got = []
    for _ in range(2):
        pr = _problem(n, seed=5, grad_dtype="bf16")
        ctx, cfg, opt = _ctx(b, "bf16", lr=1e-3)
        ctx.bind([pr.ptrs()])
        if staged:
            ctx.tune(0, 3, 0)
            ctx.set_gradients_persist(True)
        res = ctx.active_step(allow_nonfinite=True, deferred=staged)
        ctx.enable_diagnostics(True)
        res2 = ctx.active_step(allow_nonfinite=True, deferred=staged)
        d = ctx.get_diagnostics()
        got.append((gu.to_host_f64(pr.theta), gu.to_host_f64(pr.m), res.norm, res2.norm,
                    (d.g0_norm, d.g1_norm, d.cos_g0_gslow, d.ratio_mean, d.ratio_std, d.scale_mean, d.disp_ratio)))
        ctx.close()
    np.testing.assert_array_equal(got[0][0], got[1][0])
    np.testing.assert_array_equal(got[0][1], got[1][1])
    assert got[0][2:] == got[1][2:]                     # bitwise: fixed summation order


def test_probe_step_against_library_adamw_on_device():
    """The fallback step is one AdamW step: cross-check with torch.optim.AdamW (fp32)."""
    b = _binding()
    import torch
    n = 100003
    pr = _problem(n, seed=9, grad_dtype="f32", warm=False)
    ctx, cfg, opt = _ctx(b, "f32", lr=1e-3)
    ctx.bind([pr.ptrs()])
    p = torch.nn.Parameter(pr.theta.clone())
    lib = torch.optim.AdamW([p], lr=1e-3, betas=(0.9, 0.999), eps=1e-8, weight_decay=0.01)
    for g in (pr.g0, pr.g1):
        p.grad = g.clone()
        lib.step()
        pr.g0.copy_(g)
        ctx.probe_step(-1)
    torch.cuda.synchronize()
    got, want = pr.theta.double().cpu().numpy(), p.detach().double().cpu().numpy()
    gu.assert_close(got, want, "theta vs torch AdamW", rtol=2e-6)
    gu.assert_close(pr.m.double().cpu().numpy(), lib.state[p]["exp_avg"].double().cpu().numpy(), "m", rtol=2e-6)
    gu.assert_close(pr.v.double().cpu().numpy(), lib.state[p]["exp_avg_sq"].double().cpu().numpy(), "v", rtol=2e-6)
    assert ctx.gate_peek()[2] == 2 and ctx.optimizer_steps() == 2
    ctx.close()


@pytest.mark.parametrize("kind,grad_dtype", [("adamw", "bf16"), ("adamw", "f32"), ("gd", "f32"), ("gd", "bf16")])
@pytest.mark.parametrize("placement", [0, 1])
def test_fused_probe_extrapolate_is_bit_identical_to_the_two_calls(kind, grad_dtype, placement):
    """theta^{t,2} kept in registers: same theta-tilde, m, v, final theta and norm as
    gxpo_probe_step(1) followed by gxpo_extrapolate -- which the other tests compare
    with the oracle."""
    b = _binding()
    sizes = [3 * 32768 + 5, 2047, 1, 40003]
    offsets = [0, 0, 0, 1]
    outs = []
    for fused in (False, True):
        probs = [_problem(n, seed=60 + i, grad_dtype=grad_dtype, zero_frac=0.03, offset=off)
                 for i, (n, off) in enumerate(zip(sizes, offsets))]
        ctx, cfg, opt = _ctx(b, grad_dtype, kind=b.OPT_ADAMW if kind == "adamw" else b.OPT_GD, lr=1e-3,
                             K=5, alpha=0.5, placement=placement)
        ctx.bind([p.ptrs() for p in probs])
        ctx.probe_step(0)
        if fused:
            ctx.probe_extrapolate()
        else:
            ctx.probe_step(1)
            ctx.extrapolate()
        tilde = [gu.to_host_f64(p.theta) for p in probs]
        ctx.slow_step()
        res = ctx.gate_update(allow_nonfinite=True)
        outs.append((tilde, [gu.to_host_f64(p.theta) for p in probs], [gu.to_host_f64(p.m) for p in probs],
                     [gu.to_host_f64(p.v) for p in probs], res.norm, ctx.optimizer_steps(), ctx.launch_count()))
        ctx.close()
    for a, c in zip(outs[0][:4], outs[1][:4]):
        for x, y in zip(a, c):
            np.testing.assert_array_equal(x, y)
    assert outs[0][4] == outs[1][4] and outs[0][5] == outs[1][5] == 3
    assert (outs[0][6], outs[1][6]) == (5, 4)


@pytest.mark.parametrize("kind,grad_dtype", [("adamw", "bf16"), ("adamw", "f32"), ("gd", "f32"), ("gd", "bf16")])
@pytest.mark.parametrize("placement", [0, 1])
def test_deferred_state_flow_is_bit_identical_to_the_four_calls(kind, grad_dtype, placement):
    """gxpo_probe_step_deferred leaves m, v alone and gxpo_probe_extrapolate replays the
    first probe step in registers: theta^{t,1}, theta-tilde, the final theta, m, v and the
    norm must equal, bit for bit, what probe 0, probe 1, extrapolate give -- the sequence
    the other tests compare with the oracle -- over two consecutive steps."""
    b = _binding()
    sizes = [3 * 32768 + 5, 2047, 1, 40003, 4096]
    offsets = [0, 0, 0, 1, 0]
    outs = []
    for deferred in (False, True):
        probs = [_problem(n, seed=80 + i, grad_dtype=grad_dtype, zero_frac=0.03, offset=off)
                 for i, (n, off) in enumerate(zip(sizes, offsets))]
        ctx, cfg, opt = _ctx(b, grad_dtype, kind=b.OPT_ADAMW if kind == "adamw" else b.OPT_GD, lr=1e-3,
                             K=5, alpha=0.5, placement=placement)
        ctx.bind([p.ptrs() for p in probs])
        rec = []
        for step in range(2):
            m_before = [gu.to_host_f64(p.m) for p in probs]
            if deferred:
                ctx.probe_step_deferred()
                for p, mb in zip(probs, m_before):          # optimizer state not written yet
                    np.testing.assert_array_equal(gu.to_host_f64(p.m), mb)
                rec.append([gu.to_host_f64(p.work if placement == 0 else p.theta) for p in probs])
                ctx.probe_extrapolate()
            else:
                ctx.probe_step(0)
                rec.append([gu.to_host_f64(p.work if placement == 0 else p.theta) for p in probs])
                ctx.probe_step(1)
                ctx.extrapolate()
            rec.append([gu.to_host_f64(p.theta) for p in probs])
            ctx.slow_step()
            res = ctx.gate_update(allow_nonfinite=True)
            rec.append([gu.to_host_f64(p.theta) for p in probs])
            rec.append([gu.to_host_f64(p.m) for p in probs])
            rec.append([gu.to_host_f64(p.v) for p in probs])
            rec.append([np.array(res.norm)])
        outs.append((rec, ctx.optimizer_steps(), ctx.launch_count()))
        ctx.close()
    for a, c in zip(outs[0][0], outs[1][0]):
        for x, y in zip(a, c):
            np.testing.assert_array_equal(x, y)
    assert outs[0][1] == outs[1][1] == 6
    assert (outs[0][2], outs[1][2]) == (10, 8)


def test_deferred_call_order():
    b = _binding()
    pr = _problem(1000, 1, "bf16")
    ctx, cfg, opt = _ctx(b, "bf16")
    ctx.bind([pr.ptrs()])
    ctx.probe_step_deferred()
    for call in (lambda: ctx.probe_step(1), ctx.extrapolate, ctx.slow_step, ctx.gate_update,
                 ctx.probe_step_deferred, lambda: ctx.probe_step(0), lambda: ctx.probe_step(-1)):
        with pytest.raises(b.GxpoError) as e:
            call()
        assert e.value.status == b.ERR_STATE
    ctx.probe_extrapolate()
    ctx.slow_step()
    assert ctx.gate_update().t == 1 and ctx.optimizer_steps() == 3
    ctx.close()


def test_fused_call_order():
    b = _binding()
    pr = _problem(1000, 1, "bf16")
    ctx, cfg, opt = _ctx(b, "bf16")
    ctx.bind([pr.ptrs()])
    with pytest.raises(b.GxpoError) as e:
        ctx.probe_extrapolate()
    assert e.value.status == b.ERR_STATE
    ctx.probe_step(0)
    ctx.probe_extrapolate()
    for call in (ctx.probe_extrapolate, ctx.extrapolate, lambda: ctx.probe_step(1)):
        with pytest.raises(b.GxpoError) as e:
            call()
        assert e.value.status == b.ERR_STATE
    ctx.slow_step()
    assert ctx.gate_update().t == 1
    ctx.close()


@pytest.mark.parametrize("flow,staging", [(f, s) for f in ("deferred", "fused", "unfused", "fallback")
                                          for s in ("registers", "staged")] + [("deferred", "staged+promise"),
                                                                               ("deferred", "bf16-only points")])
@pytest.mark.parametrize("placement", [0, 1])
def test_no_sweep_writes_outside_its_tensors(flow, placement, staging):
    """Every output buffer (theta, work, m, v and the bfloat16 copies) sits between two
    guard bands filled with a sentinel; after a step the bands must be untouched and the
    read-only gradient buffers bit-identical.  Sizes end mid-vector, mid-tile, mid-stage and
    mid-chunk, aligned and misaligned; the shared-memory staged sweeps (with and without the
    gradients-persist promise, which needs diagnostics off) are held to the same, and so is
    the step with bfloat16-only probe points, which must not touch `work` at all."""
    import torch
    b = _binding()
    only16 = staging == "bf16-only points"
    if only16 and placement == 1:
        pytest.skip("bfloat16-only points need PINGPONG placement")
    sizes = [1, 7, 2049, 32768 + 3, 2 * 32768 - 1, 70001, 3 * 4096 + 2048 + 5]
    offsets = [0, 3, 0, 0, 1, 0, 0]
    GUARD = 4096
    sentinel = 1234.5

    def guarded(x):
        big = torch.full((x.numel() + 2 * GUARD,), sentinel, dtype=x.dtype, device="cuda")
        big[GUARD:GUARD + x.numel()] = x
        return big, big[GUARD:GUARD + x.numel()]

    bigs, ptrs, grads, wptrs = [], [], [], []
    for i, (n, off) in enumerate(zip(sizes, offsets)):
        pr = _problem(n, seed=500 + i, grad_dtype="bf16", zero_frac=0.03, offset=off)
        views = []
        for t in (pr.theta, pr.work, pr.m, pr.v):
            big, view = guarded(t if off == 0 else torch.cat([t.new_zeros(off), t]))
            bigs.append(big)
            views.append(view[off:] if off else view)
        wbig, wview = guarded(torch.zeros(n + off, dtype=torch.bfloat16, device="cuda"))
        bigs.append(wbig)
        wptrs.append((wview[off:] if off else wview).data_ptr())
        ptrs.append(b.tensor_ptrs(views[0], views[1], views[2], views[3], pr.g0, pr.g1, pr.gs))
        grads.append((pr, [pr.g0.clone(), pr.g1.clone(), pr.gs.clone()]))
    ctx, cfg, opt = _ctx(b, "bf16", lr=1e-3, K=5, alpha=0.5, placement=placement)
    ctx.bind(ptrs)
    ctx.bind_model_weights(wptrs, bf16_only=b.BF16_ONLY_PROBE_POINTS if only16 else b.BF16_BESIDE)
    ctx.tune(0, 2 if staging == "registers" else 3, 0)
    ctx.enable_diagnostics(staging not in ("staged+promise", "bf16-only points"))
    ctx.set_gradients_persist(staging in ("staged+promise", "bf16-only points"))
    work_before = [bigs[5 * i + 1].clone() for i in range(len(sizes))] if only16 else None
    for _ in range(2):
        if flow == "fallback":
            ctx.probe_step(-1)
        else:
            ctx.active_step(allow_nonfinite=True, fused=(flow == "fused"), deferred=(flow == "deferred"))
    torch.cuda.synchronize()
    for big in bigs:
        s = torch.tensor(sentinel, dtype=big.dtype, device="cuda")
        assert torch.all(big[:GUARD] == s) and torch.all(big[-GUARD:] == s)
    if only16:
        for i, w in enumerate(work_before):
            assert torch.equal(bigs[5 * i + 1].view(torch.int32), w.view(torch.int32)), f"tensor {i}: `work` was written"
    for pr, (g0, g1, gs) in grads:
        assert torch.equal(pr.g0.view(torch.int16), g0.view(torch.int16))
        assert torch.equal(pr.g1.view(torch.int16), g1.view(torch.int16))
        assert torch.equal(pr.gs.view(torch.int16), gs.view(torch.int16))
    ctx.close()


@pytest.mark.parametrize("kind,grad_dtype", [("adamw", "bf16"), ("adamw", "f32"), ("gd", "f32"), ("gd", "bf16")])
@pytest.mark.parametrize("deferred", [False, True])
def test_bulk_copy_staged_fused_sweep_is_bit_identical(kind, grad_dtype, deferred):
    """Variant 3 (tiles staged in shared memory by bulk asynchronous copies) against the
    register-staged sweep: full tiles, ragged chunk ends, a misaligned tensor, tensors
    smaller than a tile, many chunks per CTA, gradient scales and bfloat16 copies on."""
    import torch
    b = _binding()
    sizes = [40 * 32768 + 5, 2047, 1, 40003, 2048, 3 * 2048 + 17, 300 * 32768]
    offsets = [0, 0, 0, 1, 0, 0, 0]
    outs, norms = [], []
    for variant in (2, 3):
        probs = [_problem(n, seed=90 + i, grad_dtype=grad_dtype, zero_frac=0.03, offset=off)
                 for i, (n, off) in enumerate(zip(sizes, offsets))]
        ctx, cfg, opt = _ctx(b, grad_dtype, kind=b.OPT_ADAMW if kind == "adamw" else b.OPT_GD, lr=1e-3, K=5, alpha=0.5)
        ctx.tune(0, variant, 0)
        ctx.bind([p.ptrs() for p in probs])
        wbs = [torch.zeros(p.n, dtype=torch.bfloat16, device="cuda") for p in probs]
        ctx.bind_model_weights([w.data_ptr() for w in wbs])
        scales = torch.tensor([0.5, 0.75, 1.0], dtype=torch.float32, device="cuda")
        for k in range(3):
            ctx.set_grad_scale(k, scales.data_ptr() + 4 * k)
        rec = []
        for _ in range(2):
            res = ctx.active_step(allow_nonfinite=True, fused=not deferred, deferred=deferred)
            rec += [gu.to_host_f64(p.theta) for p in probs] + [gu.to_host_f64(p.m) for p in probs]
            rec += [gu.to_host_f64(p.v) for p in probs] + [gu.to_host_f64(w) for w in wbs]
            norms.append(res.norm)
        outs.append(rec)
        ctx.close()
    for x, y in zip(outs[0], outs[1]):
        np.testing.assert_array_equal(x, y)
    # the norm's partial sums are grouped by CTA, and the two variants use different grids
    assert norms[0] == pytest.approx(norms[2], rel=1e-12) and norms[1] == pytest.approx(norms[3], rel=1e-12)


def test_bounded_wait_gives_up_and_reports_timeout():
    """A wait on a barrier that nothing completes must end by itself, raise the device
    error word and leave the context usable."""
    b = _binding()
    pr = _problem(5000, 3, "bf16")
    ctx, cfg, opt = _ctx(b, "bf16", lr=1e-3)
    ctx.bind([pr.ptrs()])
    assert ctx.selftest_bounded_wait() == b.ERR_TIMEOUT
    assert "gave up" in b._lib.gxpo_last_error(ctx._h).decode()
    res = ctx.active_step(allow_nonfinite=True, deferred=True)     # still works, and the word was cleared
    assert res.t == 1
    ctx.tune(0, 3, 0)
    assert ctx.active_step(allow_nonfinite=True, deferred=True).t == 2
    ctx.close()


def test_injected_timeout_is_reported_by_active_and_by_fallback_steps():
    """The device error word, raised from the host exactly as a wait that gave up would
    raise it (no waiting kernel runs): an active step reports it from its gate update; a
    fallback step, which has no gate update, from the next call that looks at the context.
    Either way it is reported once and the context stays usable."""
    b = _binding()
    pr = _problem(3 * 32768 + 100, 5, "bf16")
    ctx, cfg, opt = _ctx(b, "bf16", lr=1e-3)
    ctx.bind([pr.ptrs()])
    ctx.tune(0, 3, 0)                                        # the staged sweeps: the ones that wait
    # active step
    ctx.probe_step_deferred()
    ctx.selftest_inject_timeout()
    ctx.probe_extrapolate()
    ctx.slow_step()
    with pytest.raises(b.GxpoError) as e:
        ctx.gate_update()
    assert e.value.status == b.ERR_TIMEOUT and "step 0" in str(e.value)
    assert ctx.active_step(deferred=True).t == 2             # reported once; the word was cleared
    # fallback step
    ctx.selftest_inject_timeout()
    ctx.probe_step(-1)                                       # the sweep itself returns OK (asynchronous)
    with pytest.raises(b.GxpoError) as e:
        ctx.gate_peek()
    assert e.value.status == b.ERR_TIMEOUT and "fallback step 2" in str(e.value)
    assert ctx.gate_peek()[2] == 3                           # once
    ctx.probe_step(-1)
    ctx.selftest_inject_timeout()
    ctx.probe_step(-1)
    with pytest.raises(b.GxpoError) as e:
        ctx.probe_step(-1)                                   # the next step refuses to build on an incomplete one
    assert e.value.status == b.ERR_TIMEOUT and "fallback step 4" in str(e.value)
    ctx.probe_step(-1)
    assert ctx.gate_peek()[2] == 6 and ctx.optimizer_steps() == 6 + 4
    ctx.close()


@pytest.mark.parametrize("n", [40003, 3 * 32768 + 5])
@pytest.mark.parametrize("kind,grad_dtype", [("adamw", "bf16"), ("adamw", "f32"), ("gd", "f32")])
@pytest.mark.parametrize("mode", ["plain", "staged", "replay"])
def test_slow_step_call_alone(n, kind, grad_dtype, mode):
    """Strict 1e-6 check of gxpo_slow_step by itself: the oracle's OptimStep starts from the
    very bits the library holds before the call (theta-tilde, m, v copied back), so no
    earlier call's rounding enters and no slack is needed.  `replay`: under the
    gradients-persist promise m and v in memory still predate the two probe steps and the
    slow sweep advances them with g0 and g1 first; the oracle is given the same inputs."""
    if kind == "gd" and mode == "replay":
        pytest.skip("plain gradient descent has no state to replay")
    b = _binding()
    pr = _problem(n, seed=700 + n, grad_dtype=grad_dtype, zero_frac=0.03)
    ctx, cfg, opt = _ctx(b, grad_dtype, kind=b.OPT_ADAMW if kind == "adamw" else b.OPT_GD, lr=1e-3, K=5, alpha=0.5)
    gcfg, ocfg = gu.ora_cfgs(cfg, opt)
    ctx.bind([pr.ptrs()])
    ctx.tune(0, 0 if mode == "plain" else 3, 0)
    ctx.set_gradients_persist(mode == "replay")
    ctx.probe_step_deferred()
    ctx.probe_extrapolate()
    grads = pr.oracle_grads()
    st = ora.State(gu.to_host_f64(pr.theta), ocfg, None if kind == "gd" else gu.to_host_f64(pr.m),
                   None if kind == "gd" else gu.to_host_f64(pr.v), t_opt=0 if mode == "replay" else 2)
    if mode == "replay":
        assert ctx.last_sweep().bytes_written_per_param == 4         # m, v really were left unwritten
        tilde = st.theta.copy()
        st.optim_step(grads[0], True)                                # only m, v matter here
        st.optim_step(grads[1], True)
        st.theta = tilde
    with np.errstate(all="ignore"):
        st.optim_step(grads[2], True)
    ctx.slow_step()
    res = ctx.gate_update(allow_nonfinite=True)
    gu.assert_close(gu.to_host_f64(pr.theta), st.theta, "theta after the slow step alone")
    if kind == "adamw":
        gu.assert_close(gu.to_host_f64(pr.m), st.m, "m")
        gu.assert_close(gu.to_host_f64(pr.v), st.v, "v")
    assert res.norm == pytest.approx(ora.l2norm(grads[2]), rel=gu.RTOL_NORM)
    ctx.close()


def test_last_sweep_reports_what_the_dispatch_chose():
    """gxpo_last_sweep is where a benchmark gets kernel names and byte counts from; check it
    against the documented dispatch on a short list (register-staged), with the staged
    kernels forced, with bfloat16 copies, and for plain gradient descent."""
    import torch
    b = _binding()
    pr = _problem(3 * 32768 + 5, 9, "bf16")
    ctx, cfg, opt = _ctx(b, "bf16", lr=1e-3)
    with pytest.raises(b.GxpoError) as e:
        ctx.last_sweep()
    assert e.value.status == b.ERR_STATE
    ctx.bind([pr.ptrs()])

    def sweep():
        k = ctx.last_sweep()
        return k.kernel.decode(), k.staged, k.bytes_read_per_param, k.bytes_written_per_param

    ctx.probe_step(0); assert sweep() == ("step_kernel", 0, 14, 12)
    ctx.probe_step(1); assert sweep() == ("step_kernel", 0, 14, 12)
    ctx.extrapolate(); assert sweep() == ("extrap_kernel", 0, 12, 4)
    ctx.slow_step(); assert sweep() == ("step_kernel", 0, 14, 12)
    ctx.gate_update(allow_nonfinite=True)
    ctx.probe_step_deferred(); assert sweep() == ("step_kernel", 0, 14, 4)
    ctx.probe_extrapolate(); assert sweep() == ("fused_kernel", 0, 16, 12)
    ctx.slow_step(); ctx.gate_update(allow_nonfinite=True)
    ctx.probe_step(0); ctx.probe_extrapolate(); assert sweep() == ("fused_kernel", 0, 20, 12)
    ctx.slow_step(); ctx.gate_update(allow_nonfinite=True)
    ctx.tune(0, 3, 0)
    ctx.set_gradients_persist(True)
    ctx.probe_step_deferred(); assert sweep() == ("step_kernel", 0, 14, 4)
    ctx.probe_extrapolate(); assert sweep() == ("fused_bulk_light_kernel", 1, 16, 4)
    ctx.slow_step(); assert sweep() == ("step_bulk_kernel", 1, 18, 12)
    ctx.gate_update(allow_nonfinite=True)
    ctx.set_gradients_persist(False)
    wb = torch.zeros(pr.n, dtype=torch.bfloat16, device="cuda")
    ctx.bind_model_weights([wb.data_ptr()], only_bf16_theta1=True)
    ctx.probe_step_deferred(); assert sweep() == ("step_kernel", 0, 14, 2)
    ctx.probe_extrapolate(); assert sweep() == ("fused_bulk_kernel", 1, 16, 14)
    ctx.slow_step(); assert sweep() == ("step_bulk_kernel", 1, 14, 14)
    ctx.gate_update(allow_nonfinite=True)
    ctx.probe_step(-1); assert sweep() == ("step_bulk_kernel", 1, 14, 14)
    ctx.clip_grad_norm(0, 1.0); assert sweep() == ("dot_kernel", 0, 2, 0)
    ctx.close()
    th, m, v, g0, g1, gs = workloads.llm_inputs_numpy(50000, 3, "f32")
    pg = gu.Problem(th, None, None, g0, g1, gs)
    cfg, opt = b.make_cfg(kind=b.OPT_GD, lr=1e-2)
    gd = b.Context(cfg, opt, b.F32)
    gd.bind([pg.ptrs()])
    gd.probe_step(0)
    k = gd.last_sweep()
    assert (k.kernel, k.bytes_read_per_param, k.bytes_written_per_param) == (b"step_kernel", 8, 4)
    gd.probe_extrapolate()
    k = gd.last_sweep()
    assert (k.kernel, k.bytes_read_per_param, k.bytes_written_per_param) == (b"fused_kernel", 16, 4)
    gd.close()
