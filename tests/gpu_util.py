"""Helpers shared by the GPU parity tests: move seeded numpy inputs to the
device, run the CUDA library through its C ABI, run the CPU oracle on the same
bits, and compare element by element."""
from __future__ import annotations

import numpy as np

from oracle import gxpo_oracle as ora

RTOL_ELEM = 1e-6      # float32 elementwise outputs (relative, per element)
RTOL_NORM = 1e-5      # reduced norms


def to_dev(x: np.ndarray, bf16: bool = False):
    import torch
    if bf16:                                    # uint16 bit patterns -> bfloat16 tensor
        return torch.from_numpy(x.view(np.int16).copy()).cuda().view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(x)).cuda()


def grad_to_f64(g: np.ndarray) -> np.ndarray:
    return ora.bf16_bits_to_f64(g) if g.dtype == np.uint16 else g.astype(np.float64)


def to_host_f64(t) -> np.ndarray:
    import torch
    if t.dtype == torch.bfloat16:
        return ora.bf16_bits_to_f64(t.view(torch.int16).cpu().numpy().view(np.uint16))
    return t.detach().cpu().numpy().astype(np.float64)


def ulp32(x):
    """Spacing of float32 numbers at |x| (float64 array in, float64 out)."""
    return np.spacing(np.abs(np.asarray(x, dtype=np.float64)).astype(np.float32)).astype(np.float64)


def displacement_slack(theta0, theta2, scale, alpha, ulps=4.0, theta1=None):
    """Absolute slack for outputs that contain (theta2 - theta0) * scale when theta2
    itself was produced by an earlier float32 call: theta2 carries up to a couple of
    ulps of its own rounding, the subtraction cancels the leading digits, and the
    scale factor multiplies what is left.  This is the conditioning of the formula,
    not an error of either implementation.  The ulp is that of the largest point on
    the way: where a step is as large as the parameter itself, theta1 can be several
    times larger than both theta0 and theta2, and its rounding (at its own magnitude)
    is what theta2 inherits -- pass theta1 where such coordinates occur."""
    big = np.maximum(np.abs(theta0), np.abs(theta2))
    if theta1 is not None:
        big = np.maximum(big, np.abs(theta1))
    with np.errstate(invalid="ignore", over="ignore"):
        return ulps * ulp32(big) * abs(alpha) * np.abs(scale)


def assert_close(gpu, want, what="", rtol=RTOL_ELEM, saturated=None, extra_abs=None):
    """|gpu - want| <= rtol |want| + rtol rms(want) (+ extra_abs) per element.
    Elements the oracle marks as saturated (float32 cannot hold the scale factor or
    the result) must be non-finite, huge, or still match."""
    gpu = np.asarray(gpu, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert gpu.shape == want.shape, what
    sat = ~np.isfinite(want) | (np.abs(want) > 1e30)
    if saturated is not None:
        sat |= saturated
    fin = ~sat
    rms = float(np.sqrt(np.mean(want[fin] ** 2))) if fin.any() else 0.0
    err = np.abs(gpu - want)
    tol = rtol * np.abs(want) + rtol * rms
    if extra_abs is not None:
        with np.errstate(invalid="ignore"):
            tol = tol + np.where(np.isfinite(extra_abs), extra_abs, 0.0)
    with np.errstate(invalid="ignore"):
        bad = fin & ~(err <= tol)
        sat_bad = sat & np.isfinite(gpu) & (np.abs(gpu) <= 1e29) & ~(err <= tol)
    if bad.any() or sat_bad.any():
        i = int(np.argmax(bad | sat_bad))
        raise AssertionError(
            f"{what}: {int(bad.sum())} of {gpu.size} elements out of tolerance "
            f"(+{int(sat_bad.sum())} saturated mismatches); first at {i}: gpu={gpu[i]!r} "
            f"oracle={want[i]!r} err={err[i]:.3e} tol={tol[i]:.3e}")
    return int(sat.sum())


class Problem:
    """One flat parameter vector on the device plus its oracle twin."""

    def __init__(self, theta, m, v, g0, g1, gs, offset_elems: int = 0):
        import torch
        self.np_in = dict(theta=theta, m=m, v=v, g0=g0, g1=g1, gs=gs)
        self.bf16 = g0.dtype == np.uint16
        n = theta.size

        def dev(x, bf16=False):
            # offset_elems > 0 places the data at a misaligned address inside a
            # larger allocation (exercises the scalar path)
            if x is None:
                return None
            t = to_dev(x, bf16)
            if offset_elems:
                big = torch.empty(n + offset_elems + 64, dtype=t.dtype, device="cuda")
                big[offset_elems:offset_elems + n] = t
                return big[offset_elems:offset_elems + n]
            return t

        self.theta = dev(theta)
        self.work = dev(np.full(n, np.nan, dtype=np.float32))
        self.m = dev(m)
        self.v = dev(v)
        self.g0 = dev(g0, self.bf16)
        self.g1 = dev(g1, self.bf16)
        self.gs = dev(gs, self.bf16)
        self.n = n

    def ptrs(self):
        from paper_2605_06755_b200 import binding
        return binding.tensor_ptrs(self.theta, self.work, self.m, self.v, self.g0, self.g1, self.gs)

    def oracle_state(self, opt: ora.OptCfg, t_opt: int = 0) -> ora.State:
        i = self.np_in
        return ora.State(i["theta"], opt, i["m"], i["v"], t_opt)

    def oracle_grads(self):
        i = self.np_in
        return [grad_to_f64(i["g0"]), grad_to_f64(i["g1"]), grad_to_f64(i["gs"])]


def ora_cfgs(cfg, opt):
    """Oracle configuration objects mirroring binding.Cfg / binding.OptCfg (the
    float32 hyper-parameters are widened exactly)."""
    o = ora.OptCfg(kind="adamw" if opt.kind == 1 else "gd", lr=float(opt.lr),
                   beta1=float(opt.beta1), beta2=float(opt.beta2), eps=float(opt.eps),
                   weight_decay=float(opt.weight_decay))
    g = ora.GxpoCfg(K=cfg.K, alpha=float(cfg.alpha), delta=float(cfg.delta),
                    den_eps=float(cfg.den_eps), tau=cfg.tau, gate_eps=cfg.gate_eps,
                    window=cfg.window, min_history=cfg.min_history, std_ddof=cfg.std_ddof)
    return g, o
