"""Parity on the LoRA-shaped list (rank-128 adapters on the q, k, v, o projections of a
Qwen2.5-7B-shaped decoder: the paper's 7B training setting): 224 tensors of 65,536 or
458,752 parameters, 80,740,352 in all, 2464 chunks.  The list is bound with the library's
DEFAULT launch configuration -- on this length that means the shared-memory staged pair
(fused sweep with m, v unwritten, slow sweep replaying them) with every CTA walking some
17 chunks of many different tensors, and half-chunk work units for the register-staged
sweeps -- a dispatch the short lists of the other parity tests only reach when it is forced.

Two consecutive active steps, the benchmark's call sequence and the four literal calls;
every element of all 224 tensors is compared with the CPU oracle.  Each step is compared
as one step: the oracle starts from the bits the library itself holds at the start of that
step (copied back to the host), so nothing but the step under test enters the comparison."""
import math

import numpy as np
import pytest

from oracle import gxpo_oracle as ora
from paper_2605_06755_b200 import workloads
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def _device_list(torch, b, shapes, seed):
    d = sum(k for _, k in shapes)
    theta, work, m, v = (torch.empty(d, dtype=torch.float32, device="cuda") for _ in range(4))
    g0, g1, gs = (torch.empty(d, dtype=torch.bfloat16, device="cuda") for _ in range(3))
    workloads.fill_llm_inputs_torch(theta, m, v, g0, g1, gs, seed, zero_frac=0.03)
    work.fill_(float("nan"))
    ptrs, off = [], 0
    for _, k in shapes:
        ptrs.append(b.TensorPtrs(theta.data_ptr() + 4 * off, work.data_ptr() + 4 * off, m.data_ptr() + 4 * off,
                                 v.data_ptr() + 4 * off, g0.data_ptr() + 2 * off, g1.data_ptr() + 2 * off,
                                 gs.data_ptr() + 2 * off, k))
        off += k
    return d, ptrs, (theta, work, m, v, g0, g1, gs)


@pytest.mark.parametrize("flow", ["deferred_persist", "unfused"])
def test_lora_list_in_the_default_dispatch_matches_the_oracle_on_every_element(flow):
    import torch
    from paper_2605_06755_b200 import binding as b
    shapes = workloads.lora_qwen25_7b_shapes()
    assert len(shapes) == 224 and sum(k for _, k in shapes) == 80_740_352
    d, ptrs, keep = _device_list(torch, b, shapes, 77)
    theta, work, m, v, g0, g1, gs = keep
    cfg, opt = b.make_cfg(lr=1e-3, K=5, alpha=0.5)
    gcfg, ocfg = gu.ora_cfgs(cfg, opt)
    ctx = b.Context(cfg, opt, b.BF16)                       # no gxpo_tune: the default dispatch
    ctx.bind(ptrs)
    ctx.set_gradients_persist(flow == "deferred_persist")
    h_g = [gu.to_host_f64(g) for g in (g0, g1, gs)]         # the gradients stay the same over both steps
    want_norm = math.sqrt(ora.sum_squares(h_g[2]))
    nsat = 0
    for step in range(2):
        h_th, h_m, h_v = (gu.to_host_f64(x) for x in (theta, m, v))   # the library's own bits
        if flow == "deferred_persist":
            ctx.probe_step_deferred()
            k0 = ctx.last_sweep()
            ctx.probe_extrapolate()
            k1 = ctx.last_sweep()
            ctx.slow_step()
            k2 = ctx.last_sweep()
            # what the library chose for this list: the staged pair, state written once
            assert (k0.kernel, k0.bytes_read_per_param, k0.bytes_written_per_param) == (b"step_kernel", 14, 4)
            assert (k1.kernel, k1.bytes_read_per_param, k1.bytes_written_per_param) == (b"fused_bulk_light_kernel", 16, 4)
            assert (k2.kernel, k2.bytes_read_per_param, k2.bytes_written_per_param) == (b"step_bulk_kernel", 18, 12)
        else:
            ctx.probe_step(0)
            ctx.probe_step(1)
            ctx.extrapolate()
            ctx.slow_step()
            assert ctx.last_sweep().kernel == b"step_kernel"            # under 32 chunks per SM: register-staged
        res = ctx.gate_update(allow_nonfinite=True)
        torch.cuda.synchronize()
        assert res.norm == pytest.approx(want_norm, rel=gu.RTOL_NORM)
        got_th, got_m, got_v = (gu.to_host_f64(x) for x in (theta, m, v))
        off = 0
        for i, (name, k) in enumerate(shapes):
            sl = slice(off, off + k)
            st = ora.State(h_th[sl], ocfg, h_m[sl], h_v[sl], t_opt=3 * step)
            grads = [g[sl] for g in h_g]
            trace = {}
            with np.errstate(all="ignore"):
                ora.active_step(st, gcfg, lambda w, th: grads[w], round_f32=True, trace=trace)
                sat = ~np.isfinite(trace["scale"]) | (np.abs(trace["scale"]) > 1e30)
                # lr = 1e-3 against theta ~ N(0, 0.02): among 80M coordinates thousands have a step larger
                # than the parameter, so theta1's magnitude (and rounding) exceeds that of both end points
                slack = gu.displacement_slack(h_th[sl], trace["theta2"], trace["scale"], gcfg.alpha,
                                              theta1=trace["theta1"])
            what = f"step {step}, tensor {i} ({name})"
            nsat += gu.assert_close(got_th[sl], st.theta, what + " theta", rtol=2e-6, saturated=sat, extra_abs=slack)
            gu.assert_close(got_m[sl], st.m, what + " m")
            gu.assert_close(got_v[sl], st.v, what + " v")
            off += k
    assert nsat < 1e-3 * 2 * d
    assert ctx.optimizer_steps() == 6
    ctx.close()
