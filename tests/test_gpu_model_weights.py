"""bfloat16 model-weight copies emitted by the sweeps: each copy must be the
round-to-nearest-even bfloat16 of the float32 point the same sweep stored (exactly, by
the oracle's rounding function), lie within one bfloat16 step of the oracle's own
chain, and binding the copies must change no float32 output."""
import numpy as np
import pytest

from oracle import gxpo_oracle as ora
from paper_2605_06755_b200 import workloads
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

SIZES = [3 * 32768 + 5, 2047, 1, 40003, 4096]
OFFSETS = [0, 0, 0, 1, 0]          # tensor 3 is misaligned: scalar path


def _binding():
    from paper_2605_06755_b200 import binding
    return binding


def _setup(b, kind, placement, with_weights, only_bf16=False):
    import torch
    probs = []
    for i, (n, off) in enumerate(zip(SIZES, OFFSETS)):
        th, m, v, g0, g1, gs = workloads.llm_inputs_numpy(n, 300 + i, "bf16", zero_frac=0.03, warm_state=True)
        th = (th * np.float32(50.0)).astype(np.float32)        # theta ~ N(0, 1): lr 1e-3 moves bf16 digits
        probs.append(gu.Problem(th, m, v, g0, g1, gs, offset_elems=off))
    cfg, opt = b.make_cfg(kind=b.OPT_ADAMW if kind == "adamw" else b.OPT_GD, lr=1e-2, K=5, alpha=0.5,
                          placement=placement)
    ctx = b.Context(cfg, opt, b.BF16)
    ctx.bind([p.ptrs() for p in probs])
    wbs = None
    if with_weights:
        wbs = []
        for p, off in zip(probs, OFFSETS):
            big = torch.full((p.n + off + 16,), float("nan"), dtype=torch.bfloat16, device="cuda")
            wbs.append(big[off:off + p.n])
        ctx.bind_model_weights([w.data_ptr() for w in wbs], only_bf16_theta1=only_bf16)
    return probs, ctx, cfg, opt, wbs


def _bits(t):
    import torch
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def _assert_copy_of(wb, theta_f32_tensor, what):
    want = ora.round_to_bf16(gu.to_host_f64(theta_f32_tensor))
    got = _bits(wb)
    nan = (want & 0x7FFF) > 0x7F80
    np.testing.assert_array_equal(got[~nan], want[~nan], err_msg=what)
    assert np.all((got[nan] & 0x7FFF) > 0x7F80), what          # a NaN stays a NaN


def _assert_within_one_step(wb, oracle_theta, what):
    """|copy - bf16(oracle)| <= one bfloat16 spacing (the two float32 values agree to
    1e-6, so their roundings can differ by a step only when they straddle a tie)."""
    got = workloads.bf16_bits_to_f32(_bits(wb)).astype(np.float64)
    want = workloads.bf16_bits_to_f32(ora.round_to_bf16(oracle_theta)).astype(np.float64)
    fin = np.isfinite(want) & (np.abs(oracle_theta) < 1e30)
    step = np.abs(want) * 2.0 ** -7 + 1e-38
    assert np.all(np.abs(got[fin] - want[fin]) <= step[fin]), what
    assert np.mean(got[fin] == want[fin]) > 0.99, what


@pytest.mark.parametrize("flow", ["deferred", "fused", "unfused"])
@pytest.mark.parametrize("kind", ["adamw", "gd"])
@pytest.mark.parametrize("placement", [0, 1])
def test_copies_follow_every_backward_point(flow, kind, placement):
    b = _binding()
    probs, ctx, cfg, opt, wbs = _setup(b, kind, placement, True)
    ref, ctx_ref, _, _, _ = _setup(b, kind, placement, False)
    gcfg, ocfg = gu.ora_cfgs(cfg, opt)
    traces, states = [], []
    for p in probs:
        st = p.oracle_state(ocfg)
        grads = p.oracle_grads()
        tr = {}
        ora.active_step(st, gcfg, lambda w, th: grads[w], round_f32=True, trace=tr)
        traces.append(tr); states.append(st)
    live1 = (lambda p: p.work) if placement == 0 else (lambda p: p.theta)
    for c, deferred in ((ctx, flow == "deferred"), (ctx_ref, flow == "deferred")):
        c.probe_step_deferred() if deferred else c.probe_step(0)
    for p, w, tr in zip(probs, wbs, traces):
        _assert_copy_of(w, live1(p), "theta1 copy")
        _assert_within_one_step(w, tr["theta1"], "theta1 vs oracle")
    for c in (ctx, ctx_ref):
        if flow == "unfused":
            c.probe_step(1)
    if flow == "unfused":
        # the second probe step's point is not a backward point: the copy still holds theta1
        for w, tr in zip(wbs, traces):
            _assert_within_one_step(w, tr["theta1"], "copy untouched by probe 1")
    for c in (ctx, ctx_ref):
        c.extrapolate() if flow == "unfused" else c.probe_extrapolate()
    for p, w in zip(probs, wbs):
        _assert_copy_of(w, p.theta, "theta-tilde copy")
    for c in (ctx, ctx_ref):
        c.slow_step()
        c.gate_update(allow_nonfinite=True)
    for p, q, w, st, tr in zip(probs, ref, wbs, states, traces):
        _assert_copy_of(w, p.theta, "theta after slow step copy")
        sat = ~np.isfinite(tr["scale"]) | (np.abs(tr["scale"]) > 1e30)
        ok = ~sat & (np.abs(tr["scale"]) < 1e3)               # where the chained float32 values agree to 1e-6
        _assert_within_one_step(w, np.where(ok, st.theta, np.nan), "final vs oracle")
        for a, c2 in ((p.theta, q.theta), (p.m, q.m), (p.v, q.v)):       # binding copies changes nothing else
            np.testing.assert_array_equal(gu.to_host_f64(a), gu.to_host_f64(c2))
    # fallback step emits too
    ctx.probe_step(-1)
    for p, w in zip(probs, wbs):
        _assert_copy_of(w, p.theta, "fallback copy")
    ctx.close(); ctx_ref.close()


def test_only_bf16_theta1_leaves_work_alone_and_gives_the_same_step():
    import torch
    b = _binding()
    a_p, a_ctx, cfg, opt, a_w = _setup(b, "adamw", 0, True, only_bf16=False)
    b_p, b_ctx, _, _, b_w = _setup(b, "adamw", 0, True, only_bf16=True)
    for p in b_p:
        p.work.fill_(123.0)
    a_ctx.probe_step_deferred(); b_ctx.probe_step_deferred()
    for p, q, wa, wb in zip(a_p, b_p, a_w, b_w):
        np.testing.assert_array_equal(_bits(wa), _bits(wb))            # same bfloat16 theta1
        assert torch.all(q.work == 123.0)                              # float32 theta1 never written
    a_ctx.probe_extrapolate(); b_ctx.probe_extrapolate()
    a_ctx.slow_step(); b_ctx.slow_step()
    ra, rb = a_ctx.gate_update(allow_nonfinite=True), b_ctx.gate_update(allow_nonfinite=True)
    for p, q, wa, wb in zip(a_p, b_p, a_w, b_w):
        np.testing.assert_array_equal(gu.to_host_f64(p.theta), gu.to_host_f64(q.theta))
        np.testing.assert_array_equal(_bits(wa), _bits(wb))
    assert ra.norm == rb.norm
    a_ctx.close(); b_ctx.close()


def test_binding_rules():
    b = _binding()
    probs, ctx, cfg, opt, wbs = _setup(b, "adamw", 1, True)
    ptrs = [w.data_ptr() for w in wbs]
    for bad, status in [(lambda: ctx.bind_model_weights(ptrs[:-1]), b.ERR_INVALID_ARG),
                        (lambda: ctx.bind_model_weights([ptrs[0] + 1] + ptrs[1:]), b.ERR_ALIGNMENT),
                        (lambda: ctx.bind_model_weights(ptrs, only_bf16_theta1=True), b.ERR_INVALID_ARG)]:  # SNAPSHOT
        with pytest.raises(b.GxpoError) as e:
            bad()
        assert e.value.status == status
    ctx.probe_step(0)
    with pytest.raises(b.GxpoError) as e:
        ctx.bind_model_weights(ptrs)
    assert e.value.status == b.ERR_STATE
    ctx.probe_extrapolate(); ctx.slow_step(); ctx.gate_update(allow_nonfinite=True)
    ctx.bind_model_weights(None)                                       # unbind: copies stay as they are
    before = [_bits(w).copy() for w in wbs]
    ctx.active_step(allow_nonfinite=True, deferred=True)
    for w, x in zip(wbs, before):
        np.testing.assert_array_equal(_bits(w), x)
    ctx.close()


@pytest.mark.parametrize("variant", [0, 3])
@pytest.mark.parametrize("bind_work", [True, False])
def test_bf16_only_probe_points_is_bit_identical_and_never_touches_work(variant, bind_work):
    """GXPO_BF16_ONLY_PROBE_POINTS: theta^{t,1} and theta-tilde exist as bfloat16 copies only,
    theta^t stays in `theta` and m, v stay put until the slow step, which recomputes
    theta-tilde.  Over three steps every copy and every float32 result must equal, bit for
    bit, what the same steps give with all float32 points stored (a flow the oracle checks
    above); `work` may be bound as NULL."""
    import torch
    b = _binding()
    a_p, a_ctx, cfg, opt, a_w = _setup(b, "adamw", 0, True)                     # float32 points beside the copies
    b_p, b_ctx, _, _, b_w = _setup(b, "adamw", 0, False)
    if not bind_work:
        b_ctx.bind([b.tensor_ptrs(p.theta, None, p.m, p.v, p.g0, p.g1, p.gs) for p in b_p])
    b_w = []
    for p, off in zip(b_p, OFFSETS):
        big = torch.full((p.n + off + 16,), float("nan"), dtype=torch.bfloat16, device="cuda")
        b_w.append(big[off:off + p.n])
        p.work.fill_(123.0)
    b_ctx.bind_model_weights([w.data_ptr() for w in b_w], bf16_only=b.BF16_ONLY_PROBE_POINTS)
    for c in (a_ctx, b_ctx):
        c.tune(0, variant, 0)
        c.set_gradients_persist(True)
    for step in range(3):
        start = [(gu.to_host_f64(p.theta), gu.to_host_f64(p.m), gu.to_host_f64(p.v)) for p in b_p]
        a_ctx.probe_step_deferred(); b_ctx.probe_step_deferred()
        for wa, wb in zip(a_w, b_w):
            np.testing.assert_array_equal(_bits(wa), _bits(wb), err_msg=f"step {step}: theta1 copy")
        a_ctx.probe_extrapolate(); b_ctx.probe_extrapolate()
        k = b_ctx.last_sweep()
        assert (k.kernel, k.bytes_read_per_param, k.bytes_written_per_param) == (b"fused_bulk_light_kernel", 16, 2)
        for p, wa, wb, s0 in zip(b_p, a_w, b_w, start):
            np.testing.assert_array_equal(_bits(wa), _bits(wb), err_msg=f"step {step}: theta-tilde copy")
            np.testing.assert_array_equal(gu.to_host_f64(p.theta), s0[0])      # theta^t still in place
            np.testing.assert_array_equal(gu.to_host_f64(p.m), s0[1])          # m, v still unwritten
            np.testing.assert_array_equal(gu.to_host_f64(p.v), s0[2])
        a_ctx.slow_step(); b_ctx.slow_step()
        k = b_ctx.last_sweep()
        assert (k.kernel, k.bytes_read_per_param, k.bytes_written_per_param) == (b"slow_recompute_bulk_kernel", 18, 14)
        ra, rb = a_ctx.gate_update(allow_nonfinite=True), b_ctx.gate_update(allow_nonfinite=True)
        for i, (p, q, wa, wb) in enumerate(zip(a_p, b_p, a_w, b_w)):
            for nm in ("theta", "m", "v"):
                np.testing.assert_array_equal(gu.to_host_f64(getattr(p, nm)), gu.to_host_f64(getattr(q, nm)),
                                              err_msg=f"step {step}, tensor {i}: {nm}")
            np.testing.assert_array_equal(_bits(wa), _bits(wb), err_msg=f"step {step}: theta^{{t+1}} copy")
            assert torch.all(q.work == 123.0)                                  # never written
        # the norm's float32 partial sums are grouped by the sweep's shape (tiles of 8 here, single
        # coordinates in the ragged ends there): equal to float32 rounding of the groups, not to the bit
        assert rb.norm == pytest.approx(ra.norm, rel=1e-7)
    assert a_ctx.launch_count() == b_ctx.launch_count() == 12
    # the fallback step needs no `work` either and emits its copy
    b_ctx.probe_step(-1)
    for p, w in zip(b_p, b_w):
        _assert_copy_of(w, p.theta, "fallback copy")
    a_ctx.close(); b_ctx.close()


def test_bf16_only_probe_points_against_the_oracle():
    b = _binding()
    probs, ctx, cfg, opt, wbs = _setup(b, "adamw", 0, True)
    ctx.bind_model_weights([w.data_ptr() for w in wbs], bf16_only=b.BF16_ONLY_PROBE_POINTS)
    ctx.set_gradients_persist(True)
    gcfg, ocfg = gu.ora_cfgs(cfg, opt)
    res = ctx.active_step(allow_nonfinite=True, deferred=True)
    sumsq = 0.0
    for i, (p, w) in enumerate(zip(probs, wbs)):
        st = p.oracle_state(ocfg)
        grads = p.oracle_grads()
        tr = {}
        ora.active_step(st, gcfg, lambda k, th: grads[k], round_f32=True, trace=tr)
        sat = ~np.isfinite(tr["scale"]) | (np.abs(tr["scale"]) > 1e30)
        slack = gu.displacement_slack(p.np_in["theta"].astype(np.float64), tr["theta2"], tr["scale"], gcfg.alpha,
                                      theta1=tr["theta1"])
        gu.assert_close(gu.to_host_f64(p.theta), st.theta, f"tensor {i} theta", rtol=2e-6, saturated=sat, extra_abs=slack)
        gu.assert_close(gu.to_host_f64(p.m), st.m, f"tensor {i} m")
        gu.assert_close(gu.to_host_f64(p.v), st.v, f"tensor {i} v")
        _assert_copy_of(w, p.theta, "theta^{t+1} copy")
        sumsq += ora.sum_squares(grads[2])
    assert res.norm == pytest.approx(np.sqrt(sumsq), rel=gu.RTOL_NORM)
    ctx.close()


def test_bf16_only_probe_points_rules():
    b = _binding()
    probs, ctx, cfg, opt, wbs = _setup(b, "adamw", 0, True)
    ptrs = [w.data_ptr() for w in wbs]
    ctx.bind_model_weights(ptrs, bf16_only=b.BF16_ONLY_PROBE_POINTS)
    with pytest.raises(b.GxpoError) as e:                     # no promise: refused before the step starts
        ctx.probe_step_deferred()
    assert e.value.status == b.ERR_STATE and "gradients_persist" in str(e.value)
    ctx.set_gradients_persist(True)
    ctx.probe_step(0)                                         # the non-deferred first step is legal ...
    with pytest.raises(b.GxpoError) as e:
        ctx.probe_extrapolate()                               # ... but this mode cannot follow it
    assert e.value.status == b.ERR_STATE
    ctx.probe_step(1); ctx.extrapolate(); ctx.slow_step(); ctx.gate_update(allow_nonfinite=True)
    ctx.enable_diagnostics(True)
    with pytest.raises(b.GxpoError) as e:
        ctx.probe_step_deferred()
    assert e.value.status == b.ERR_STATE and "diagnostics" in str(e.value)
    ctx.enable_diagnostics(False)
    ctx.tune(0, 2, 0)
    with pytest.raises(b.GxpoError) as e:
        ctx.probe_step_deferred()
    assert e.value.status == b.ERR_STATE
    ctx.tune(0, 0, 0)
    assert ctx.active_step(allow_nonfinite=True, deferred=True).t == 2
    with pytest.raises(b.GxpoError) as e:
        ctx.bind_model_weights(ptrs, bf16_only=3)
    assert e.value.status == b.ERR_INVALID_ARG
    ctx.close()
    # work == NULL: only the calls that keep no point there
    ctx = b.Context(cfg, opt, b.BF16)
    ctx.bind([b.tensor_ptrs(p.theta, None, p.m, p.v, p.g0, p.g1, p.gs) for p in probs])
    for call in (lambda: ctx.probe_step(0), lambda: ctx.probe_step_deferred()):
        with pytest.raises(b.GxpoError) as e:
            call()
        assert e.value.status == b.ERR_STATE and "work" in str(e.value)
    ctx.probe_step(-1)                                        # the fallback step works in place
    ctx.close()
    # plain gradient descent: not built
    gp, gctx, _, _, gw = _setup(b, "gd", 0, True)
    with pytest.raises(b.GxpoError) as e:
        gctx.bind_model_weights([w.data_ptr() for w in gw], bf16_only=b.BF16_ONLY_PROBE_POINTS)
    assert e.value.status == b.ERR_INVALID_ARG
    gctx.close()


def test_bf16_only_probe_points_with_gradient_scales_and_clipping():
    """The recomputing slow sweep scales g0, g1 and g_slow as the sweeps before it did: a caller's
    scale on g1 and clipping coefficients on g0 and g_slow give the same bits as with every
    float32 point stored."""
    import torch
    b = _binding()
    outs = []
    for mode in (b.BF16_BESIDE, b.BF16_ONLY_PROBE_POINTS):
        probs, ctx, cfg, opt, wbs = _setup(b, "adamw", 0, True)
        ctx.bind_model_weights([w.data_ptr() for w in wbs], bf16_only=mode)
        ctx.tune(0, 3, 0)
        ctx.set_gradients_persist(True)
        scale = torch.tensor([0.7], dtype=torch.float32, device="cuda")
        ctx.set_grad_scale(1, scale.data_ptr())
        for _ in range(2):
            ctx.clip_grad_norm(0, 0.05)
            ctx.probe_step_deferred()
            ctx.probe_extrapolate()
            ctx.clip_grad_norm(2, 0.05)
            ctx.slow_step()
            res = ctx.gate_update(allow_nonfinite=True)
        outs.append(([(gu.to_host_f64(p.theta), gu.to_host_f64(p.m), gu.to_host_f64(p.v)) for p in probs],
                     [_bits(w) for w in wbs], res.norm))
        ctx.close()
    for x, y in zip(outs[0][0], outs[1][0]):
        for u, w in zip(x, y):
            np.testing.assert_array_equal(u, w)
    for x, y in zip(outs[0][1], outs[1][1]):
        np.testing.assert_array_equal(x, y)
    assert outs[1][2] == pytest.approx(outs[0][2], rel=1e-7)
