"""Gradient scaling and global-norm clipping inside the sweeps, against the oracle fed
with explicitly scaled gradients: g' = float32(g * s) is what the optimizer steps and
the retention ratio must see, while the gate's norm stays that of the gradient as given."""
import math

import numpy as np
import pytest

from oracle import gxpo_oracle as ora
from paper_2605_06755_b200 import workloads
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

SIZES = [3 * 32768 + 5, 2047, 1, 40003]
OFFSETS = [0, 0, 0, 1]


def _binding():
    from paper_2605_06755_b200 import binding
    return binding


def _problems(grad_dtype, gain=1.0):
    probs = []
    for i, (n, off) in enumerate(zip(SIZES, OFFSETS)):
        th, m, v, g0, g1, gs = workloads.llm_inputs_numpy(n, 700 + i, "f32", zero_frac=0.03, warm_state=True)
        g0, g1, gs = (np.float32(gain) * x for x in (g0, g1, gs))
        if grad_dtype == "bf16":
            g0, g1, gs = (workloads.f32_to_bf16_bits(x) for x in (g0, g1, gs))
        probs.append(gu.Problem(th, m, v, g0, g1, gs, offset_elems=off))
    return probs


def _scaled(g64, s):
    """float32(g * s) as float64: one rounding, like the kernels' multiply on load."""
    return (g64.astype(np.float32) * np.float32(s)).astype(np.float32).astype(np.float64)


def _check(probs, scales, ctx, res, gcfg, ocfg, steps_done=1):
    sumsq = 0.0
    for i, p in enumerate(probs):
        raw = p.oracle_grads()
        grads = [_scaled(g, s) for g, s in zip(raw, scales)]
        st = p.oracle_state(ocfg)
        trace = {}
        ora.active_step(st, gcfg, lambda w, th: grads[w], round_f32=True, trace=trace)
        sat = ~np.isfinite(trace["scale"]) | (np.abs(trace["scale"]) > 1e30)
        slack = gu.displacement_slack(p.np_in["theta"].astype(np.float64), trace["theta2"], trace["scale"], gcfg.alpha)
        gu.assert_close(gu.to_host_f64(p.theta), st.theta, f"tensor {i} theta", rtol=2e-6, saturated=sat, extra_abs=slack)
        if st.m is not None:
            gu.assert_close(gu.to_host_f64(p.m), st.m, f"tensor {i} m")
            gu.assert_close(gu.to_host_f64(p.v), st.v, f"tensor {i} v")
        sumsq += ora.sum_squares(raw[2])
    assert res.norm == pytest.approx(math.sqrt(sumsq), rel=gu.RTOL_NORM)     # the gate sees the raw gradient


@pytest.mark.parametrize("flow", ["deferred", "fused", "unfused"])
@pytest.mark.parametrize("grad_dtype,kind", [("bf16", "adamw"), ("f32", "gd")])
def test_caller_supplied_scales(flow, grad_dtype, kind):
    import torch
    b = _binding()
    probs = _problems(grad_dtype)
    cfg, opt = b.make_cfg(kind=b.OPT_ADAMW if kind == "adamw" else b.OPT_GD, lr=1e-3, K=5, alpha=0.5)
    ctx = b.Context(cfg, opt, b.BF16 if grad_dtype == "bf16" else b.F32)
    ctx.bind([p.ptrs() for p in probs])
    scales = [0.3, 0.7, 0.45]
    dev = torch.tensor(scales, dtype=torch.float32, device="cuda")
    for k in range(3):
        ctx.set_grad_scale(k, dev.data_ptr() + 4 * k)
    res = ctx.active_step(allow_nonfinite=True, fused=(flow == "fused"), deferred=(flow == "deferred"))
    gcfg, ocfg = gu.ora_cfgs(cfg, opt)
    _check(probs, [float(np.float32(s)) for s in scales], ctx, res, gcfg, ocfg)
    ctx.probe_step_deferred()
    with pytest.raises(b.GxpoError) as e:
        ctx.set_grad_scale(0, 0)                          # mid-step
    assert e.value.status == b.ERR_STATE
    ctx.close()


@pytest.mark.parametrize("flow", ["deferred", "unfused"])
def test_clip_grad_norm_matches_oracle_and_expires(flow):
    """Gradients 40x the recipe's size have norms of about 13, so clipping at 1.0 bites."""
    import torch
    b = _binding()
    probs = _problems("bf16", gain=40.0)
    cfg, opt = b.make_cfg(lr=1e-3, K=5, alpha=0.5)
    ctx = b.Context(cfg, opt, b.BF16)
    ctx.bind([p.ptrs() for p in probs])
    norms = [math.sqrt(sum(ora.sum_squares(p.oracle_grads()[k]) for p in probs)) for k in range(3)]
    coefs = [float(np.float32(ora.clip_coef(x, 1.0))) for x in norms]
    assert all(c < 0.2 for c in coefs)
    for bad in (1, 2):
        with pytest.raises(b.GxpoError) as e:
            ctx.clip_grad_norm(bad, 1.0)                  # not the gradient the next sweep consumes
        assert e.value.status == b.ERR_STATE
    ctx.clip_grad_norm(0, 1.0)
    if flow == "deferred":
        ctx.probe_step_deferred()
        ctx.clip_grad_norm(1, 1.0)
        ctx.probe_extrapolate()
    else:
        ctx.probe_step(0)
        ctx.clip_grad_norm(1, 1.0)
        ctx.probe_step(1)
        ctx.extrapolate()
    ctx.clip_grad_norm(2, 1.0)
    ctx.slow_step()
    res = ctx.gate_update(allow_nonfinite=True)
    gcfg, ocfg = gu.ora_cfgs(cfg, opt)
    _check(probs, coefs, ctx, res, gcfg, ocfg)
    # the coefficients belonged to that step: an unclipped step must match an unclipped twin
    twin = _problems("bf16", gain=40.0)
    for p, q in zip(probs, twin):
        q.theta.copy_(p.theta); q.m.copy_(p.m); q.v.copy_(p.v)
    ctx2 = b.Context(cfg, opt, b.BF16)
    ctx2.bind([q.ptrs() for q in twin])
    ctx2.state_import(ctx.state_export())
    ctx.active_step(allow_nonfinite=True, deferred=True)
    ctx2.active_step(allow_nonfinite=True, deferred=True)
    torch.cuda.synchronize()
    for p, q in zip(probs, twin):
        np.testing.assert_array_equal(gu.to_host_f64(p.theta), gu.to_host_f64(q.theta))
    with pytest.raises(b.GxpoError) as e:
        ctx.clip_grad_norm(0, -1.0)
    assert e.value.status == b.ERR_INVALID_ARG
    ctx.close()
    ctx2.close()
