"""The paper's diagonal-quadratic sanity check (Corollary 1) run on the GPU through
the C ABI, the fused surrogate kernel, and the host-resident entry point."""
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


def _f32_grad_fn(a, b):
    """g = a * theta - b in float32 with a rounding after the product and after the
    difference: what the device harness kernel computes, bit for bit."""
    def fn(which, theta64):
        t = theta64.astype(np.float32)
        return ((a * t).astype(np.float32) - b).astype(np.float32).astype(np.float64)
    return fn


class Surrogate:
    def __init__(self, b, n, seed, K, alpha, eta=0.1, placement=0):
        import torch
        self.b, self.n, self.K, self.alpha, self.eta = b, n, K, alpha, eta
        self.a_np, self.b_np, self.t0_np = workloads.quadratic_surrogate(n, seed)
        self.a, self.bb, self.theta = (gu.to_dev(x) for x in (self.a_np, self.b_np, self.t0_np))
        self.work = torch.empty_like(self.theta)
        self.g0, self.g1, self.gs = (torch.empty_like(self.theta) for _ in range(3))
        cfg, opt = b.make_cfg(kind=b.OPT_GD, lr=eta, K=K, alpha=alpha, delta=1e-8, placement=placement)
        self.cfg, self.opt = cfg, opt
        self.ctx = b.Context(cfg, opt, b.F32)
        self.ctx.bind([b.tensor_ptrs(self.theta, self.work, None, None, self.g0, self.g1, self.gs)])
        self.live1 = self.work if placement == 0 else self.theta

    def grad(self, at, out):
        self.b.quad_grad(at.data_ptr(), self.a.data_ptr(), self.bb.data_ptr(), out.data_ptr(), self.n)

    def active_step(self):
        """Algorithm 1's active branch with the harness standing in for the backward passes."""
        self.grad(self.theta, self.g0)
        self.ctx.probe_step(0)
        self.grad(self.live1, self.g1)
        self.ctx.probe_step(1)
        self.ctx.extrapolate()
        self.grad(self.theta, self.gs)
        self.ctx.slow_step()
        return self.ctx.gate_update()

    def closed_form(self, steps):
        a, b, t0 = (x.astype(np.float64) for x in (self.a_np, self.b_np, self.t0_np))
        star, r = b / a, 1.0 - self.eta * a
        return star + (r * (1.0 - self.alpha + self.alpha * r ** self.K)) ** steps * (t0 - star)


@pytest.mark.parametrize("K", [3, 5, 10])
@pytest.mark.parametrize("alpha", [1.0, 0.5])
@pytest.mark.parametrize("placement", [0, 1])
def test_config0_one_active_step_vs_closed_form_and_oracle(K, alpha, placement):
    b = _binding()
    s = Surrogate(b, 4096, seed=0, K=K, alpha=alpha, placement=placement)
    res = s.active_step()
    got = gu.to_host_f64(s.theta)
    # closed form: theta* + r (1 - alpha + alpha r^K) (theta0 - theta*); alpha = 1 -> (K+1)-th GD iterate
    gu.assert_close(got, s.closed_form(1), "vs closed form", rtol=2e-6)
    gcfg, ocfg = gu.ora_cfgs(s.cfg, s.opt)
    st = ora.State(s.t0_np, ocfg)
    trace = {}
    nrm = ora.active_step(st, gcfg, _f32_grad_fn(s.a_np, s.b_np), round_f32=True, trace=trace)
    slack = gu.displacement_slack(s.t0_np.astype(np.float64), trace["theta2"], trace["scale"], gcfg.alpha)
    gu.assert_close(got, st.theta, "vs oracle", extra_abs=slack)
    assert res.norm == pytest.approx(nrm, rel=gu.RTOL_NORM)
    s.ctx.close()


def test_config0_fused_surrogate_kernel():
    import torch
    b = _binding()
    for K, alpha in [(3, 1.0), (5, 0.5), (10, 1.0)]:
        s = Surrogate(b, 4096, seed=0, K=K, alpha=alpha)
        scratch = torch.zeros(b.quad_scratch_bytes(), dtype=torch.uint8, device="cuda")
        sumsq = torch.zeros(1, dtype=torch.float64, device="cuda")
        theta = s.theta.clone()
        b.quad_active_step(theta.data_ptr(), s.a.data_ptr(), s.bb.data_ptr(), s.n, s.eta, K, alpha, 1e-8,
                           0.0, sumsq.data_ptr(), scratch.data_ptr())
        res = s.active_step()
        got = gu.to_host_f64(theta)
        gu.assert_close(got, s.closed_form(1), "fused vs closed form", rtol=2e-6)
        # same arithmetic as the four-call path, element for element
        np.testing.assert_array_equal(got, gu.to_host_f64(s.theta))
        assert math.sqrt(float(sumsq.item())) == pytest.approx(res.norm, rel=1e-12)
        s.ctx.close()


def test_config1_twenty_active_steps_at_1e8():
    """n = 1e8, 20 consecutive active steps: closed form on every element, oracle on
    sampled windows (the update is per-coordinate, so a window's oracle run is the
    full run restricted to it)."""
    import torch
    b = _binding()
    n, K, steps = 100_000_000, 5, 20
    s = Surrogate(b, n, seed=0, K=K, alpha=1.0)
    norms = [s.active_step().norm for _ in range(steps)]
    torch.cuda.synchronize()
    got = s.theta.cpu().numpy().astype(np.float64)
    want = s.closed_form(steps)                       # theta* + r^((K+1) m) (theta0 - theta*)
    gu.assert_close(got, want, "20 steps vs closed form", rtol=2e-5)
    # ||g_slow|| of the last step from the closed form: g_slow = a (theta_tilde - theta*)
    a64, b64, t64 = (x.astype(np.float64) for x in (s.a_np, s.b_np, s.t0_np))
    star, r = b64 / a64, 1.0 - s.eta * a64
    tilde = star + r ** ((K + 1) * (steps - 1) + K) * (t64 - star)
    assert norms[-1] == pytest.approx(float(np.sqrt(np.sum((a64 * (tilde - star)) ** 2))), rel=1e-4)
    assert all(x > y for x, y in zip(norms, norms[1:]))          # contraction: norms decrease
    # oracle on windows: start, a chunk boundary, the ragged end
    gcfg, ocfg = gu.ora_cfgs(s.cfg, s.opt)
    for lo, hi in [(0, 70000), (32768 * 1000 - 500, 32768 * 1000 + 500), (n - 66000, n)]:
        st = ora.State(s.t0_np[lo:hi], ocfg)
        fn = _f32_grad_fn(s.a_np[lo:hi], s.b_np[lo:hi])
        for _ in range(steps):
            ora.active_step(st, gcfg, fn, round_f32=True)
        gu.assert_close(got[lo:hi], st.theta, f"window [{lo},{hi}) vs oracle", rtol=5e-6)
    s.ctx.close()


@pytest.mark.parametrize("kind,grad_dtype", [("adamw", "bf16"), ("gd", "f32")])
def test_step_host_matches_device_path_and_oracle(kind, grad_dtype):
    import torch
    b = _binding()
    n = 5 * 32768 + 77
    sizes = [n, 1000, 32768]
    kw = dict(kind=b.OPT_ADAMW if kind == "adamw" else b.OPT_GD, lr=1e-3, K=5, alpha=0.5, tau=0.5)
    gd = b.BF16 if grad_dtype == "bf16" else b.F32
    host, dev, hold = [], [], []
    for i, k in enumerate(sizes):
        arrs = workloads.llm_inputs_numpy(k, 300 + i, grad_dtype, warm_state=True)
        pr = gu.Problem(*arrs)
        dev.append(pr)
        pinned = []
        for j, x in enumerate(arrs):
            t = torch.from_numpy(x.view(np.int16).copy() if x.dtype == np.uint16 else x.copy()).pin_memory()
            pinned.append(t)
        hold.append(pinned)
        th, m, v, g0, g1, gs = pinned
        host.append(b.tensor_ptrs(th, None, m, v, g0, g1, gs))
    cfg, opt = b.make_cfg(**kw)
    ctx_d = b.Context(cfg, opt, gd)
    ctx_d.bind([p.ptrs() for p in dev])
    ctx_h = b.Context(cfg, opt, gd)
    for step in range(3):
        rd = ctx_d.active_step(allow_nonfinite=True)
        rh = ctx_h.step_host(host, staging_elems=65536, allow_nonfinite=True)
        assert rh.norm == pytest.approx(rd.norm, rel=1e-12) and rh.t == rd.t == step + 1
        for p, pinned in zip(dev, hold):
            np.testing.assert_array_equal(pinned[0].numpy(), p.theta.cpu().numpy())
            if kind == "adamw":
                np.testing.assert_array_equal(pinned[1].numpy(), p.m.cpu().numpy())
                np.testing.assert_array_equal(pinned[2].numpy(), p.v.cpu().numpy())
    assert ctx_h.optimizer_steps() == 9
    ctx_d.close()
    ctx_h.close()
