"""gxpo_slow_step_noalloc, the slow correction for callers that cannot allocate device
memory (all of it handed to a pool, a GPU filled to the brim by the model, a callback
in which allocation is forbidden).  It keeps its reduction scratch in an array built
into the library instead of in a context.

The check: through the C ABI, on the same theta-tilde, m, v and g_slow, it must give
what gxpo_slow_step + gxpo_gate_update give -- parameters and optimizer state within
the element tolerance of the parity tests, the norm within the norm tolerance -- on two
calls in a row (the second call reuses the scratch the first one left behind).
Further cases hold it against the CPU oracle directly: a buffer with more chunks than the
grid has CTAs, a short buffer right after it, a single parameter, and two calls on two
streams ordered by an event.

This file is named so that pytest collects it last; it depends on nothing the other
tests do and passes in a fresh process as well."""
import math

import numpy as np
import pytest

from paper_2605_06755_b200 import workloads
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def _binding():
    from paper_2605_06755_b200 import binding
    return binding


@pytest.mark.parametrize("kind,grad_dtype,offset", [("adamw", "bf16", 0), ("gd", "f32", 0), ("adamw", "bf16", 3)])
def test_noalloc_slow_step_matches_context_slow_step_twice_in_a_row(kind, grad_dtype, offset):
    import torch
    b = _binding()
    n = 5 * 32768 + 77                                   # several chunks and a ragged tail
    th, m, v, g0, g1, gs = workloads.llm_inputs_numpy(n, 2024, grad_dtype, zero_frac=0.03, warm_state=True)
    pr = gu.Problem(th, m, v, g0, g1, gs, offset_elems=offset)      # offset 3: misaligned, scalar path
    cfg, opt = b.make_cfg(kind=b.OPT_ADAMW if kind == "adamw" else b.OPT_GD, lr=1e-3, K=5, alpha=0.5)
    dt = b.BF16 if grad_dtype == "bf16" else b.F32
    ctx = b.Context(cfg, opt, dt)
    ctx.bind([pr.ptrs()])
    sumsq = torch.full((1,), float("nan"), dtype=torch.float64, device="cuda")
    for call in range(2):
        ctx.probe_step(0)
        ctx.probe_extrapolate()
        torch.cuda.synchronize()
        # same starting point for both entry points: copies of theta-tilde, m, v
        th2, m2, v2 = pr.theta.clone(), pr.m.clone(), pr.v.clone()
        if offset:                                        # keep the copy misaligned too
            big = [torch.empty(n + offset + 64, dtype=torch.float32, device="cuda") for _ in range(3)]
            for dst, src in zip(big, (th2, m2, v2)):
                dst[offset:offset + n] = src
            th2, m2, v2 = (x[offset:offset + n] for x in big)
        ctx.slow_step()
        res = ctx.gate_update(allow_nonfinite=True)
        b.slow_step_noalloc(th2.data_ptr(), m2.data_ptr() if kind == "adamw" else 0,
                            v2.data_ptr() if kind == "adamw" else 0, pr.gs.data_ptr(), n, dt, opt,
                            ctx.optimizer_steps(), sumsq.data_ptr())
        torch.cuda.synchronize()
        sat = ~np.isfinite(gu.to_host_f64(pr.theta))      # a saturated scale factor is non-finite in both
        gu.assert_close(gu.to_host_f64(th2), gu.to_host_f64(pr.theta), f"theta, call {call}", saturated=sat)
        if kind == "adamw":
            gu.assert_close(gu.to_host_f64(m2), gu.to_host_f64(pr.m), f"m, call {call}")
            gu.assert_close(gu.to_host_f64(v2), gu.to_host_f64(pr.v), f"v, call {call}")
        assert math.sqrt(float(sumsq.item())) == pytest.approx(res.norm, rel=gu.RTOL_NORM)
        assert ctx.optimizer_steps() == 3 * (call + 1)
    ctx.close()


def test_noalloc_rejects_oversize_and_handles_empty():
    import torch
    b = _binding()
    _, opt = b.make_cfg()
    sumsq = torch.full((1,), 7.0, dtype=torch.float64, device="cuda")
    x = torch.zeros(8, device="cuda")
    with pytest.raises(b.GxpoError) as e:                 # rejected before anything is touched
        b.slow_step_noalloc(x.data_ptr(), x.data_ptr(), x.data_ptr(), x.data_ptr(),
                            b.NOALLOC_MAX_PARAMS + 1, b.F32, opt, 1, sumsq.data_ptr())
    assert e.value.status == b.ERR_INVALID_ARG and "GXPO_NOALLOC_MAX_PARAMS" in str(e.value)
    with pytest.raises(b.GxpoError) as e:
        b.slow_step_noalloc(x.data_ptr(), 0, 0, x.data_ptr(), 8, b.F32, opt, 1, sumsq.data_ptr())
    assert e.value.status == b.ERR_INVALID_ARG            # AdamW without m, v
    b.slow_step_noalloc(0, 0, 0, 0, 0, b.F32, opt, 1, sumsq.data_ptr())
    torch.cuda.synchronize()
    assert float(sumsq.item()) == 0.0


def _oracle_slow_step(th, m, v, gs, ocfg, t_opt):
    """OptimStep(theta, g_slow) and sum(g_slow^2) by the CPU oracle, on the same bits."""
    from oracle import gxpo_oracle as ora
    g = gu.grad_to_f64(gs)
    st = ora.State(th, ocfg, m, v, t_opt=t_opt - 1)          # optim_step counts this step itself
    st.optim_step(g, True)
    return st, ora.sum_squares(g)


def _prepare(b, n, seed, grad_dtype, t_opt, what=""):
    """Seeded inputs on the device; returns (launch(stream), check())."""
    import torch
    th, m, v, _, _, gs = workloads.llm_inputs_numpy(n, seed, grad_dtype, warm_state=True)
    cfg, opt = b.make_cfg(lr=1e-3)
    _, ocfg = gu.ora_cfgs(cfg, opt)
    d_th, d_m, d_v = gu.to_dev(th), gu.to_dev(m), gu.to_dev(v)
    d_gs = gu.to_dev(gs, grad_dtype == "bf16")
    sumsq = torch.full((1,), float("nan"), dtype=torch.float64, device="cuda")

    def launch(stream=None):
        b.slow_step_noalloc(d_th.data_ptr(), d_m.data_ptr(), d_v.data_ptr(), d_gs.data_ptr(), n,
                            b.BF16 if grad_dtype == "bf16" else b.F32, opt, t_opt, sumsq.data_ptr(), stream)

    def check():
        _compare(d_th, d_m, d_v, sumsq, _oracle_slow_step(th, m, v, gs, ocfg, t_opt), what)

    return launch, check


def _compare(d_th, d_m, d_v, sumsq, want, what):
    st, want_sumsq = want
    gu.assert_close(gu.to_host_f64(d_th), st.theta, what + " theta")      # one call, the oracle on the same bits: 1e-6
    gu.assert_close(gu.to_host_f64(d_m), st.m, what + " m")
    gu.assert_close(gu.to_host_f64(d_v), st.v, what + " v")
    assert float(sumsq.item()) == pytest.approx(want_sumsq, rel=gu.RTOL_NORM)


def test_noalloc_against_the_oracle_with_more_chunks_than_ctas_then_fewer():
    """700 chunks and a ragged tail: every CTA of the grid takes several chunks in turn, so the
    per-chunk reduction inside the loop and the reuse of its shared scratch are exercised.
    Then a much shorter buffer, whose call finds the long call's partial sums still sitting
    in the slots beyond its own chunks and must not pick them up; then a single parameter.
    All three against the CPU oracle directly."""
    import torch
    b = _binding()
    for n, seed in ((700 * 32768 + 5, 31), (3 * 32768 + 11, 32), (1, 33)):
        launch, check = _prepare(b, n, seed, "bf16", t_opt=7, what=f"n={n}")
        launch()
        torch.cuda.synchronize()
        check()


def test_noalloc_calls_on_two_streams_ordered_by_an_event():
    """All calls share the one built-in scratch array, so calls on different streams have to
    be ordered by the caller.  With an event between them the second call, on another
    stream, must give the oracle's result just like the first."""
    import torch
    b = _binding()
    launch1, check1 = _prepare(b, 600 * 32768 + 123, 41, "f32", t_opt=3, what="stream 1")
    launch2, check2 = _prepare(b, 9 * 32768 + 1, 42, "f32", t_opt=4, what="stream 2")
    torch.cuda.synchronize()                                  # inputs in place; from here on only the event orders
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    launch1(s1)
    done = torch.cuda.Event()
    done.record(s1)
    s2.wait_event(done)                                       # the second call starts after the first has finished
    launch2(s2)
    s1.synchronize()
    s2.synchronize()
    check1()
    check2()
