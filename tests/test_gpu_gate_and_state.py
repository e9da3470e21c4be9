"""Gate timing, call-order state machine, argument checks and the small-state
checkpoint of the CUDA library, against the CPU oracle."""
import math

import numpy as np
import pytest

from oracle import gxpo_oracle as ora
from paper_2605_06755_b200 import workloads
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def _binding():
    from paper_2605_06755_b200 import binding
    return binding


def _small_list(b, sizes, seed):
    """LLM-shaped tensors whose retention ratios g1/g0 stay in [0.2, 1.2] (the range the
    paper reports, 0.5-0.6 +- 0.7, without the synthetic recipe's heavy tail): over many
    chained steps a huge scale factor would amplify last-ulp differences into visible
    ones, which is a property of the formula, not of either implementation."""
    probs = []
    for i, n in enumerate(sizes):
        rng = np.random.default_rng(seed + i)
        th = (0.02 * rng.standard_normal(n)).astype(np.float32)
        g0f = (1e-3 * rng.standard_normal(n)).astype(np.float32)
        g1f = (g0f * rng.uniform(0.2, 1.2, n)).astype(np.float32)
        gsf = (g0f * rng.uniform(0.5, 1.0, n)).astype(np.float32)
        z = np.zeros(n, dtype=np.float32)
        probs.append(gu.Problem(th, z, z.copy(), workloads.f32_to_bf16_bits(g0f),
                                workloads.f32_to_bf16_bits(g1f), workloads.f32_to_bf16_bits(gsf)))
    return probs


def test_gate_trips_at_the_oracle_step_on_a_64_step_stream():
    """g_slow scaled x1 for steps 0..39 and x8 at step 40 (exact in bfloat16): the
    library must fall back at exactly the oracle's step, and keep matching it
    through the fallback phase."""
    import torch
    b = _binding()
    sizes = [4096, 70000, 512, 33000]
    probs = _small_list(b, sizes, seed=50)
    cfg, opt = b.make_cfg(lr=1e-3, K=5, alpha=0.5, tau=0.5, window=20)
    ctx = b.Context(cfg, opt, b.BF16)
    ctx.bind([p.ptrs() for p in probs])
    gcfg, ocfg = gu.ora_cfgs(cfg, opt)
    states = [p.oracle_state(ocfg) for p in probs]
    gate = ora.Gate(gcfg)
    base_gs = [p.gs.clone() for p in probs]
    phases = []
    for t in range(64):
        scale = 8.0 if t == 40 else 1.0
        for p, g in zip(probs, base_gs):
            p.gs.copy_(g * scale)
        grads = [[gu.to_host_f64(p.g0), gu.to_host_f64(p.g1), gu.to_host_f64(p.gs)] for p in probs]
        active_lib, s_star_lib, t_lib = ctx.gate_peek()
        assert t_lib == t and active_lib == gate.active
        if gate.active:
            sumsq = 0.0
            for st, g in zip(states, grads):
                ora.active_step(st, gcfg, lambda w, th, g=g: g[w], round_f32=True)
                sumsq += ora.sum_squares(g[2])
            tripped, z, mu, sg = gate.update(math.sqrt(sumsq))
            res = ctx.active_step()
            assert bool(res.tripped) == tripped
            assert res.norm == pytest.approx(math.sqrt(sumsq), rel=gu.RTOL_NORM)
            if not math.isnan(z):
                assert res.z == pytest.approx(z, rel=1e-3, abs=1e-3) or abs(z) > 1e3
            phases.append("active")
        else:
            for st, g in zip(states, grads):
                ora.fallback_step(st, lambda w, th, g=g: g[w], round_f32=True)
            gate.fallback_tick()
            ctx.probe_step(-1)
            phases.append("fallback")
        assert ctx.gate_peek()[1] == gate.s_star
    torch.cuda.synchronize()
    assert gate.s_star == 41 and ctx.gate_peek()[1] == 41
    assert phases == ["active"] * 41 + ["fallback"] * 23
    assert ctx.backward_passes() == ora.backward_budget(41, 64) == 3 * 41 + 23
    assert ctx.optimizer_steps() == 3 * 41 + 23
    for i, (p, st) in enumerate(zip(probs, states)):
        gu.assert_close(gu.to_host_f64(p.theta), st.theta, f"tensor {i} theta after 64 steps", rtol=2e-5)
        gu.assert_close(gu.to_host_f64(p.m), st.m, f"tensor {i} m", rtol=5e-6)
        gu.assert_close(gu.to_host_f64(p.v), st.v, f"tensor {i} v", rtol=5e-6)
    with pytest.raises(b.GxpoError) as e:
        ctx.probe_step(0)                                   # active phase is over for good
    assert e.value.status == b.ERR_STATE
    ctx.close()


def test_gate_matches_oracle_on_random_norm_streams():
    """Drive only the norm: one-element tensors whose g_slow is the norm itself."""
    import torch
    b = _binding()
    rng = np.random.default_rng(77)
    for trial, (tau, window, ddof) in enumerate([(1.5, 7, 0), (0.5, 20, 0), (2.0, 5, 1), (0.8, 3, 0)]):
        norms = np.abs(1.0 + 0.2 * rng.standard_normal(120)).astype(np.float32)
        cfg, opt = b.make_cfg(kind=b.OPT_GD, lr=0.0, tau=tau, window=window, std_ddof=ddof)
        ctx = b.Context(cfg, opt, b.F32)
        th = torch.zeros(1, device="cuda")
        wk = torch.zeros(1, device="cuda")
        g = torch.ones(1, device="cuda")
        gs = torch.zeros(1, device="cuda")
        ctx.bind([b.tensor_ptrs(th, wk, None, None, g, g, gs)])
        gcfg, _ = gu.ora_cfgs(cfg, opt)
        gate = ora.Gate(gcfg)
        for t, x in enumerate(norms):
            if not gate.active:
                break
            gs.fill_(float(x))
            res = ctx.active_step()
            tripped, z, mu, sg = gate.update(float(x))
            # float32 gradients are squared in float32: one rounding, 6e-8 relative
            assert res.norm == pytest.approx(float(x), rel=2e-7)
            assert bool(res.tripped) == tripped and res.s_star == gate.s_star
            if not math.isnan(z):
                assert abs(z - tau) > 1e-3, "stream has a step too close to the threshold"
                assert res.z == pytest.approx(z, rel=1e-4, abs=1e-5)
                assert res.mu == pytest.approx(mu, rel=1e-6) and res.sigma == pytest.approx(sg, rel=1e-4, abs=1e-9)
            else:
                assert math.isnan(res.z)
        assert ctx.gate_peek()[1] == gate.s_star
        assert gate.s_star > 0, "stream was meant to trip"
        ctx.close()


def test_nonfinite_norm_trips_and_reports():
    import torch
    b = _binding()
    cfg, opt = b.make_cfg(kind=b.OPT_GD, lr=0.0)
    ctx = b.Context(cfg, opt, b.F32)
    th = torch.zeros(4, device="cuda"); wk = torch.zeros(4, device="cuda")
    g = torch.ones(4, device="cuda"); gs = torch.tensor([1.0, float("inf"), 0.0, 0.0], device="cuda")
    ctx.bind([b.tensor_ptrs(th, wk, None, None, g, g, gs)])
    ctx.probe_step(0); ctx.probe_step(1); ctx.extrapolate(); ctx.slow_step()
    with pytest.raises(b.GxpoError) as e:
        ctx.gate_update()
    assert e.value.status == b.ERR_NONFINITE
    active, s_star, t = ctx.gate_peek()
    assert not active and s_star == 1 and t == 1
    ctx.close()


def test_call_order_and_argument_checks():
    import torch
    b = _binding()
    cfg, opt = b.make_cfg()
    for bad in [dict(K=1), dict(alpha=1.5), dict(alpha=-0.1), dict(delta=-1.0), dict(window=0),
                dict(min_history=0), dict(std_ddof=2), dict(placement=7), dict(kind=5),
                dict(beta1=1.0), dict(lr=float("nan")), dict(den_eps=-1.0)]:
        c2, o2 = b.make_cfg(**bad)
        with pytest.raises(b.GxpoError) as e:
            b.Context(c2, o2, b.BF16)
        assert e.value.status == b.ERR_INVALID_ARG, bad
    with pytest.raises(b.GxpoError):
        b.Context(cfg, opt, 9)
    ctx = b.Context(cfg, opt, b.BF16)
    with pytest.raises(b.GxpoError) as e:
        ctx.probe_step(0)                                   # nothing bound
    assert e.value.status == b.ERR_STATE
    n = 1000
    th, m, v, g0, g1, gs = workloads.llm_inputs_numpy(n, 1, "bf16")
    pr = gu.Problem(th, m, v, g0, g1, gs)
    good = pr.ptrs()
    for field, val, status in [("n", -1, b.ERR_INVALID_ARG), ("theta", 0, b.ERR_INVALID_ARG),
                               ("m", 0, b.ERR_INVALID_ARG), ("g_slow", 0, b.ERR_INVALID_ARG),
                               ("theta", good.theta + 2, b.ERR_ALIGNMENT),
                               ("g1", good.g1 + 1, b.ERR_ALIGNMENT)]:
        t = b.TensorPtrs(**{**good.__dict__, field: val})
        with pytest.raises(b.GxpoError) as e:
            ctx.bind([t])
        assert e.value.status == status, field
    # `work` may be left out at bind time; the calls that keep a point there then refuse
    ctx.bind([b.TensorPtrs(**{**good.__dict__, "work": 0})])
    for call in (lambda: ctx.probe_step(0), ctx.probe_step_deferred):
        with pytest.raises(b.GxpoError) as e:
            call()
        assert e.value.status == b.ERR_STATE and "work" in str(e.value)
    ctx.bind([good])
    for call in (lambda: ctx.probe_step(1), ctx.extrapolate, ctx.slow_step, ctx.gate_update):
        with pytest.raises(b.GxpoError) as e:
            call()
        assert e.value.status == b.ERR_STATE
    with pytest.raises(b.GxpoError) as e:
        ctx.probe_step(2)
    assert e.value.status == b.ERR_INVALID_ARG
    ctx.probe_step(0)
    for call in (lambda: ctx.probe_step(0), lambda: ctx.probe_step(-1), ctx.extrapolate,
                 ctx.slow_step, ctx.gate_update, lambda: ctx.bind([good]), ctx.state_export):
        with pytest.raises(b.GxpoError) as e:
            call()
        assert e.value.status == b.ERR_STATE
    ctx.probe_step(1)
    with pytest.raises(b.GxpoError):
        ctx.slow_step()
    ctx.extrapolate()
    with pytest.raises(b.GxpoError):
        ctx.gate_update()
    ctx.slow_step()
    res = ctx.gate_update()
    assert res.t == 1 and ctx.optimizer_steps() == 3
    with pytest.raises(b.GxpoError) as e:
        ctx.tune(99, 0, 0)
    assert e.value.status == b.ERR_INVALID_ARG
    assert "ctas_per_sm" in str(e.value)
    torch.cuda.synchronize()
    ctx.close()


def test_state_export_import_round_trip():
    import torch
    b = _binding()
    rng = np.random.default_rng(6)            # max Z over the first 25 steps is 2.4: far below tau
    norms = np.abs(1.0 + 0.05 * rng.standard_normal(30)).astype(np.float32)
    norms[25] = 3.0

    def make():
        cfg, opt = b.make_cfg(kind=b.OPT_GD, lr=0.0, tau=6.0, window=6)
        ctx = b.Context(cfg, opt, b.F32)
        th = torch.zeros(1, device="cuda"); wk = torch.zeros(1, device="cuda")
        g = torch.ones(1, device="cuda"); gs = torch.zeros(1, device="cuda")
        ctx.bind([b.tensor_ptrs(th, wk, None, None, g, g, gs)])
        return ctx, gs, (th, wk, g)

    def drive(ctx, gs, xs):
        out = []
        for x in xs:
            if not ctx.gate_peek()[0]:
                ctx.probe_step(-1)
                out.append(None)
                continue
            gs.fill_(float(x))
            r = ctx.active_step()
            out.append((r.tripped, r.z, r.mu, r.sigma, r.s_star, r.t))
        return out

    ref, gs_ref, keep1 = make()
    want = drive(ref, gs_ref, norms)
    a, gs_a, keep2 = make()
    drive(a, gs_a, norms[:13])
    blob = a.state_export()
    bctx, gs_b, keep3 = make()
    bctx.state_import(blob)
    assert bctx.gate_peek() == a.gate_peek() and bctx.optimizer_steps() == a.optimizer_steps() == 39
    got = drive(bctx, gs_b, norms[13:])
    for w, g in zip(want[13:], got):
        assert (w is None) == (g is None)
        if w is not None:
            assert w[0] == g[0] and w[4] == g[4] and w[5] == g[5]
            assert (math.isnan(w[1]) and math.isnan(g[1])) or w[1] == g[1]   # bitwise equal Z
    assert ref.gate_peek() == bctx.gate_peek() and ref.gate_peek()[1] == 26
    with pytest.raises(b.GxpoError):
        bctx.state_import(blob[:10])
    with pytest.raises(b.GxpoError):
        bctx.state_import(b"\0" * len(blob))
    for c in (ref, a, bctx):
        c.close()


def test_async_gate_update_gives_the_same_decisions():
    """gxpo_gate_update_async + whoever collects the outcome (the next probe step, gate_peek,
    gate_last) against the synchronous call, on a stream that trips at step 9."""
    import torch
    b = _binding()
    rng = np.random.default_rng(3)
    norms = np.abs(1.0 + 0.01 * rng.standard_normal(14)).astype(np.float32)
    norms[9] = 2.0

    def make():
        cfg, opt = b.make_cfg(kind=b.OPT_GD, lr=0.0, tau=3.0, window=8)
        ctx = b.Context(cfg, opt, b.F32)
        th = torch.zeros(1, device="cuda"); wk = torch.zeros(1, device="cuda")
        g = torch.ones(1, device="cuda"); gs = torch.zeros(1, device="cuda")
        ctx.bind([b.tensor_ptrs(th, wk, None, None, g, g, gs)])
        return ctx, gs, (th, wk, g)

    sync, gs_s, k1 = make()
    asyn, gs_a, k2 = make()
    with pytest.raises(b.GxpoError) as e:
        asyn.gate_last()
    assert e.value.status == b.ERR_STATE
    for t, x in enumerate(norms):
        assert sync.gate_peek() == asyn.gate_peek()
        if not sync.gate_peek()[0]:
            sync.probe_step(-1); asyn.probe_step(-1)
            continue
        gs_s.fill_(float(x)); gs_a.fill_(float(x))
        want = sync.active_step()
        asyn.probe_step_deferred(); asyn.probe_extrapolate(); asyn.slow_step()
        asyn.gate_update_async()
        if t % 3 == 0:
            got = asyn.gate_last()                       # collected explicitly
        elif t % 3 == 1:
            asyn.gate_peek(); got = asyn.gate_last()     # collected by gate_peek
        else:
            got = None                                   # collected by the next probe step
        if got is not None:
            assert (got.tripped, got.s_star, got.t, got.active) == (want.tripped, want.s_star, want.t, want.active)
            assert got.norm == want.norm and (got.z == want.z or (math.isnan(got.z) and math.isnan(want.z)))
    assert sync.gate_peek() == asyn.gate_peek() and sync.gate_peek()[1] == 10
    assert sync.backward_passes() == asyn.backward_passes() == 3 * 10 + 4
    assert asyn.state_export() == sync.state_export()
    with pytest.raises(b.GxpoError) as e:
        asyn.probe_step_deferred()                       # tripped: the active phase is over
    assert e.value.status == b.ERR_STATE
    sync.close(); asyn.close()


def test_two_contexts_on_two_streams_and_rebinding():
    """Contexts own their scratch, so two of them may run at the same time on different
    streams; and a context may be re-bound to another list between steps.  Results must be
    those of the same steps run one after the other."""
    import torch
    b = _binding()
    sizes = [5 * 32768 + 77, 70001]

    def fresh(seed):
        probs = _small_list(b, sizes, seed=seed)
        cfg, opt = b.make_cfg(lr=1e-3, K=5, alpha=0.5)
        ctx = b.Context(cfg, opt, b.BF16)
        ctx.bind([p.ptrs() for p in probs])
        return probs, ctx

    # serial reference
    ref = []
    for seed in (11, 12):
        probs, ctx = fresh(seed)
        for _ in range(3):
            r = ctx.active_step(deferred=True)
        ref.append(([gu.to_host_f64(p.theta) for p in probs], r.norm))
        ctx.close()
    # the same two runs interleaved on two streams
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    (p1, c1), (p2, c2) = fresh(11), fresh(12)
    torch.cuda.synchronize()
    for _ in range(3):
        c1.probe_step_deferred(s1); c2.probe_step_deferred(s2)
        c1.probe_extrapolate(s1); c2.probe_extrapolate(s2)
        c1.slow_step(s1); c2.slow_step(s2)
        c1.gate_update_async(s1); c2.gate_update_async(s2)
    r1, r2 = c1.gate_last(), c2.gate_last()
    torch.cuda.synchronize()
    for probs, r, (want, norm) in ((p1, r1, ref[0]), (p2, r2, ref[1])):
        for p, w in zip(probs, want):
            np.testing.assert_array_equal(gu.to_host_f64(p.theta), w)
        assert r.norm == norm
    # re-bind c1 to the second list's tensors (state carries over, data is the caller's)
    c1.bind([p.ptrs() for p in p2])
    before = [gu.to_host_f64(p.theta) for p in p2]
    c1.active_step(deferred=True)
    assert c1.optimizer_steps() == 12 and c1.gate_peek()[2] == 4
    assert any(not np.array_equal(gu.to_host_f64(p.theta), x) for p, x in zip(p2, before))
    c1.close(); c2.close()
