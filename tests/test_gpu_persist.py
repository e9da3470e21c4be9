"""gxpo_set_gradients_persist: with the caller's promise that g0 and g1 outlive the slow
step's sweep, the fused sweep may leave m and v unwritten and the slow step replays both
moment updates.  Nothing observable may change: theta, m, v, the norm, the bfloat16
copies and the diagnostics are compared bit for bit with the same steps taken without
the promise (a call sequence the oracle checks elsewhere), and once directly with the
oracle."""
import numpy as np
import pytest

from oracle import gxpo_oracle as ora
from paper_2605_06755_b200 import workloads
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

# whole staged tiles, a ragged rest, a short tensor, one element, a misaligned tensor
SIZES = [3 * 32768 + 4096 + 5, 2047, 1, 40003, 8192]
OFFSETS = [0, 0, 0, 1, 0]


def _binding():
    from paper_2605_06755_b200 import binding
    return binding


def _problems(grad_dtype, seed=500):
    probs = []
    for i, (n, off) in enumerate(zip(SIZES, OFFSETS)):
        arrs = workloads.llm_inputs_numpy(n, seed + i, grad_dtype, zero_frac=0.03, warm_state=True)
        probs.append(gu.Problem(*arrs, offset_elems=off))
    return probs


def _ctx(b, probs, grad_dtype, placement, variant, persist, lr=1e-3):
    cfg, opt = b.make_cfg(lr=lr, K=5, alpha=0.5, placement=placement)
    ctx = b.Context(cfg, opt, b.BF16 if grad_dtype == "bf16" else b.F32)
    ctx.bind([p.ptrs() for p in probs])
    ctx.tune(0, variant, 0)
    ctx.set_gradients_persist(persist)
    return ctx, cfg, opt


def _state(probs):
    return [tuple(gu.to_host_f64(t) for t in (p.theta, p.m, p.v)) for p in probs]


def _assert_same(a, b, what):
    for i, (x, y) in enumerate(zip(a, b)):
        for nm, u, w in zip(("theta", "m", "v"), x, y):
            np.testing.assert_array_equal(u, w, err_msg=f"{what}: tensor {i} {nm}")


@pytest.mark.parametrize("grad_dtype", ["bf16", "f32"])
@pytest.mark.parametrize("placement", [0, 1])
def test_promise_changes_no_bit_over_three_steps(grad_dtype, placement):
    b = _binding()
    pa, pb = _problems(grad_dtype), _problems(grad_dtype)
    ca, _, _ = _ctx(b, pa, grad_dtype, placement, 3, False)
    cb, _, _ = _ctx(b, pb, grad_dtype, placement, 3, True)
    for step in range(3):
        start = _state(pb)
        for c in (ca, cb):
            c.probe_step_deferred()
            c.probe_extrapolate()
        mid_a, mid_b = _state(pa), _state(pb)
        for i, (x, y, z) in enumerate(zip(mid_a, mid_b, start)):
            np.testing.assert_array_equal(x[0], y[0], err_msg=f"theta-tilde, tensor {i}")
            # the path under test really ran: m and v are still the start-of-step values
            np.testing.assert_array_equal(y[1], z[1])
            np.testing.assert_array_equal(y[2], z[2])
            assert not np.array_equal(x[1], z[1]) or x[1].size < 2
        for c in (ca, cb):
            c.slow_step()
        ra, rb = ca.gate_update(allow_nonfinite=True), cb.gate_update(allow_nonfinite=True)
        _assert_same(_state(pa), _state(pb), f"step {step}")
        assert ra.norm == rb.norm
        assert ra.z == rb.z or (np.isnan(ra.z) and np.isnan(rb.z))
    assert ca.launch_count() == cb.launch_count()
    ca.close(); cb.close()


def test_against_the_oracle():
    b = _binding()
    probs = _problems("bf16", seed=520)
    ctx, cfg, opt = _ctx(b, probs, "bf16", 0, 3, True)
    gcfg, ocfg = gu.ora_cfgs(cfg, opt)
    res = ctx.active_step(allow_nonfinite=True, deferred=True)
    sumsq = 0.0
    for i, p in enumerate(probs):
        st = p.oracle_state(ocfg)
        grads = p.oracle_grads()
        trace = {}
        ora.active_step(st, gcfg, lambda w, th: grads[w], round_f32=True, trace=trace)
        sat = ~np.isfinite(trace["scale"]) | (np.abs(trace["scale"]) > 1e30)
        slack = gu.displacement_slack(p.np_in["theta"].astype(np.float64), trace["theta2"], trace["scale"], gcfg.alpha)
        gu.assert_close(gu.to_host_f64(p.theta), st.theta, f"tensor {i} theta", rtol=2e-6, saturated=sat, extra_abs=slack)
        gu.assert_close(gu.to_host_f64(p.m), st.m, f"tensor {i} m")
        gu.assert_close(gu.to_host_f64(p.v), st.v, f"tensor {i} v")
        sumsq += ora.sum_squares(grads[2])
    assert res.norm == pytest.approx(np.sqrt(sumsq), rel=gu.RTOL_NORM)
    ctx.close()


@pytest.mark.parametrize("diag", [False, True])
def test_with_gradient_scales_clipping_copies_and_diagnostics(diag):
    """With diagnostics on the library does not use the promise (their arithmetic bounds the
    fused sweep, not its state writes): same results again, by the ordinary path."""
    import torch
    b = _binding()
    outs = []
    for persist in (False, True):
        probs = _problems("bf16", seed=540)
        ctx, cfg, opt = _ctx(b, probs, "bf16", 0, 3, persist)
        wbs = [torch.zeros(p.n, dtype=torch.bfloat16, device="cuda") for p in probs]
        ctx.bind_model_weights([w.data_ptr() for w in wbs])
        ctx.enable_diagnostics(diag)
        scale = torch.tensor([0.7], dtype=torch.float32, device="cuda")
        ctx.set_grad_scale(1, scale.data_ptr())
        ctx.clip_grad_norm(0, 0.05)
        m_before = gu.to_host_f64(probs[0].m)
        ctx.probe_step_deferred()
        ctx.probe_extrapolate()
        lagging = np.array_equal(m_before, gu.to_host_f64(probs[0].m))
        assert lagging == (persist and not diag)
        ctx.clip_grad_norm(2, 0.05)
        ctx.slow_step()
        res = ctx.gate_update(allow_nonfinite=True)
        if diag:
            d = ctx.get_diagnostics()
            figures = (d.g0_norm, d.g1_norm, d.gslow_norm, d.ratio_mean, d.scale_mean, d.n_active, d.n_irregular,
                       d.cos_g0_gslow)
        else:
            figures = ()
        outs.append((_state(probs), [w.view(torch.int16).cpu().numpy() for w in wbs], res.norm, figures))
        ctx.close()
    _assert_same(outs[0][0], outs[1][0], "scaled and clipped")
    for x, y in zip(outs[0][1], outs[1][1]):
        np.testing.assert_array_equal(x, y)
    assert outs[0][2] == outs[1][2] and outs[0][3] == outs[1][3]


def test_promise_is_ignored_where_it_cannot_hold_or_does_not_pay():
    b = _binding()
    # g_slow in g1's buffer: the fused sweep must write m and v as usual
    probs = _problems("bf16", seed=560)
    cfg, opt = b.make_cfg(lr=1e-3)
    ctx = b.Context(cfg, opt, b.BF16)
    ctx.bind([b.tensor_ptrs(p.theta, p.work, p.m, p.v, p.g0, p.g1, p.g1) for p in probs])
    ctx.tune(0, 3, 0)
    ctx.set_gradients_persist(True)
    before = _state(probs)
    ctx.probe_step_deferred()
    with pytest.raises(b.GxpoError) as e:
        ctx.set_gradients_persist(False)                       # mid-step
    assert e.value.status == b.ERR_STATE
    ctx.probe_extrapolate()
    after = _state(probs)
    assert not np.array_equal(before[0][1], after[0][1])       # m advanced in memory
    ctx.slow_step(); ctx.gate_update(allow_nonfinite=True)
    ctx.close()
    # short list, default variant: register-staged sweeps, state written by the fused sweep
    probs = _problems("bf16", seed=560)
    ctx, _, _ = _ctx(b, probs, "bf16", 0, 0, True)
    before = _state(probs)
    ctx.probe_step_deferred(); ctx.probe_extrapolate()
    assert not np.array_equal(before[0][1], _state(probs)[0][1])
    ctx.slow_step(); ctx.gate_update(allow_nonfinite=True)
    # plain gradient descent has no state to defer
    th, m, v, g0, g1, gs = workloads.llm_inputs_numpy(50000, 3, "f32")
    pr = gu.Problem(th, m, v, g0, g1, gs)
    cfg, opt = b.make_cfg(kind=b.OPT_GD, lr=1e-2)
    gd = b.Context(cfg, opt, b.F32)
    gd.bind([pr.ptrs()])
    gd.tune(0, 3, 0)
    gd.set_gradients_persist(True)
    gd.active_step(allow_nonfinite=True, deferred=True)
    gd.close(); ctx.close()
