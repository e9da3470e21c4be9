"""ctypes front end of the GXPO oracle (oracle/gxpo_oracle.cpp).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU
baseline leg import this; the product package never does.  This file holds no
arithmetic of the method beyond calling the C++ functions in the order
Algorithm 1 gives; it marshals numpy float64 arrays and compiles the shared
object with g++ when it is missing or stale.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gxpo_oracle.cpp")
_LIB = os.path.join(_HERE, "libgxpo_oracle.so")

_f64p = ctypes.POINTER(ctypes.c_double)
_i64 = ctypes.c_int64


def build(force: bool = False) -> str:
    """Compile the oracle; -ffp-contract=off keeps the written operation order."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fno-fast-math", "-shared",
             "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        L.gxo_optim_step_gd.argtypes = [_f64p, _f64p, _i64, ctypes.c_double, ctypes.c_int]
        L.gxo_optim_step_gd.restype = None
        L.gxo_optim_step_adamw.argtypes = [_f64p, _f64p, _f64p, _f64p, _i64, _i64] + \
            [ctypes.c_double] * 5 + [ctypes.c_int]
        L.gxo_optim_step_adamw.restype = None
        L.gxo_extrapolate.argtypes = [_f64p] * 7 + [_i64, ctypes.c_int] + \
            [ctypes.c_double] * 3 + [ctypes.c_int]
        L.gxo_extrapolate.restype = None
        L.gxo_sum_squares.argtypes = [_f64p, _i64]
        L.gxo_sum_squares.restype = ctypes.c_double
        L.gxo_l2norm.argtypes = [_f64p, _i64]
        L.gxo_l2norm.restype = ctypes.c_double
        L.gxo_round_to_bf16.argtypes = [_f64p, ctypes.POINTER(ctypes.c_uint16), _i64]
        L.gxo_round_to_bf16.restype = None
        L.gxo_clip_coef.argtypes = [ctypes.c_double, ctypes.c_double]
        L.gxo_clip_coef.restype = ctypes.c_double
        L.gxo_active_diagnostics.argtypes = [_f64p] * 5 + [_i64, ctypes.c_int, ctypes.c_double,
                                             ctypes.c_double, _f64p]
        L.gxo_active_diagnostics.restype = None
        L.gxo_gate_create.argtypes = [ctypes.c_double, ctypes.c_double, ctypes.c_int,
                                      ctypes.c_int, ctypes.c_int]
        L.gxo_gate_create.restype = ctypes.c_void_p
        L.gxo_gate_destroy.argtypes = [ctypes.c_void_p]
        L.gxo_gate_destroy.restype = None
        L.gxo_gate_active.argtypes = [ctypes.c_void_p]
        L.gxo_gate_active.restype = ctypes.c_int
        L.gxo_gate_s_star.argtypes = [ctypes.c_void_p]
        L.gxo_gate_s_star.restype = _i64
        L.gxo_gate_t.argtypes = [ctypes.c_void_p]
        L.gxo_gate_t.restype = _i64
        L.gxo_gate_update.argtypes = [ctypes.c_void_p, ctypes.c_double, _f64p, _f64p, _f64p]
        L.gxo_gate_update.restype = ctypes.c_int
        L.gxo_gate_fallback_tick.argtypes = [ctypes.c_void_p]
        L.gxo_gate_fallback_tick.restype = None
        L.gxo_backward_budget.argtypes = [_i64, _i64]
        L.gxo_backward_budget.restype = _i64
        _lib = L
    return _lib


def _p(a: np.ndarray):
    assert a.dtype == np.float64 and a.flags["C_CONTIGUOUS"], "oracle arrays are contiguous float64"
    return a.ctypes.data_as(_f64p)


def as_f64(a) -> np.ndarray:
    """Exact widening of fp32 / fp64 numpy data to a fresh contiguous float64 array."""
    return np.array(a, dtype=np.float64, order="C", copy=True)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """uint16 bfloat16 bit patterns -> float64, exactly (a data-format conversion)."""
    u = bits.astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


@dataclass
class OptCfg:
    kind: str = "adamw"          # "gd" or "adamw"
    lr: float = 1e-7
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    weight_decay: float = 0.01


@dataclass
class GxpoCfg:
    K: int = 5
    alpha: float = 0.5
    delta: float = 1e-8
    den_eps: float = 0.0
    tau: float = 0.5
    gate_eps: float = 1e-8
    window: int = 20
    min_history: int = 2
    std_ddof: int = 0


def optim_step_gd(theta, g, lr, round_f32=False):
    lib().gxo_optim_step_gd(_p(theta), _p(g), theta.size, float(lr), int(round_f32))


def optim_step_adamw(theta, m, v, g, t_opt, opt: OptCfg, round_f32=False):
    lib().gxo_optim_step_adamw(_p(theta), _p(m), _p(v), _p(g), theta.size, int(t_opt),
                               float(opt.lr), float(opt.beta1), float(opt.beta2),
                               float(opt.eps), float(opt.weight_decay), int(round_f32))


def extrapolate(theta0, theta2, g0, g1, K, alpha, delta, den_eps=0.0, round_f32=False,
                want_aux=False):
    n = theta0.size
    out = np.empty(n, dtype=np.float64)
    tk = np.empty(n, dtype=np.float64) if want_aux else None
    sc = np.empty(n, dtype=np.float64) if want_aux else None
    lib().gxo_extrapolate(_p(out), _p(tk) if want_aux else None, _p(sc) if want_aux else None,
                          _p(theta0), _p(theta2), _p(g0), _p(g1), n, int(K), float(alpha),
                          float(delta), float(den_eps), int(round_f32))
    return (out, tk, sc) if want_aux else out


def sum_squares(g) -> float:
    return float(lib().gxo_sum_squares(_p(g), g.size))


def l2norm(g) -> float:
    return float(lib().gxo_l2norm(_p(g), g.size))


def round_to_bf16(theta) -> np.ndarray:
    """float64 array of float32 values -> uint16 bfloat16 patterns (round to nearest even)."""
    theta = np.ascontiguousarray(theta, dtype=np.float64)
    out = np.empty(theta.size, dtype=np.uint16)
    lib().gxo_round_to_bf16(_p(theta), out.ctypes.data_as(ctypes.POINTER(ctypes.c_uint16)), theta.size)
    return out


def clip_coef(norm: float, max_norm: float) -> float:
    """min(1, max_norm / (norm + 1e-6)): the global-norm clipping coefficient."""
    return float(lib().gxo_clip_coef(float(norm), float(max_norm)))


DIAG_FIELDS = ("g0_norm", "g1_norm", "gslow_norm", "cos_g0_gslow", "ratio_mean", "ratio_std",
               "scale_mean", "disp_ratio", "inactive_frac", "n_active", "n_irregular")


def active_diagnostics(theta0, theta2, g0, g1, g_slow, K, delta, den_eps=0.0) -> dict:
    """The appendix's active-phase diagnostics for one step (see the C++ header comment)."""
    out = np.empty(len(DIAG_FIELDS), dtype=np.float64)
    lib().gxo_active_diagnostics(_p(theta0), _p(theta2), _p(g0), _p(g1), _p(g_slow), theta0.size,
                                 int(K), float(delta), float(den_eps), _p(out))
    return dict(zip(DIAG_FIELDS, out.tolist()))


def backward_budget(s_star: int, T: int) -> int:
    return int(lib().gxo_backward_budget(int(s_star), int(T)))


class Gate:
    """Rolling z-score gate; one instance per training run."""

    def __init__(self, cfg: GxpoCfg):
        self._h = lib().gxo_gate_create(float(cfg.tau), float(cfg.gate_eps), int(cfg.window),
                                        int(cfg.min_history), int(cfg.std_ddof))
        if not self._h:
            raise ValueError("invalid gate configuration")

    def __del__(self):
        if getattr(self, "_h", None):
            lib().gxo_gate_destroy(self._h)
            self._h = None

    @property
    def active(self) -> bool:
        return bool(lib().gxo_gate_active(self._h))

    @property
    def s_star(self) -> int:
        return int(lib().gxo_gate_s_star(self._h))

    @property
    def t(self) -> int:
        return int(lib().gxo_gate_t(self._h))

    def update(self, norm: float):
        z = ctypes.c_double()
        mu = ctypes.c_double()
        sg = ctypes.c_double()
        tripped = lib().gxo_gate_update(self._h, float(norm), ctypes.byref(z), ctypes.byref(mu),
                                        ctypes.byref(sg))
        return bool(tripped), z.value, mu.value, sg.value

    def fallback_tick(self):
        lib().gxo_gate_fallback_tick(self._h)


class State:
    """theta / optimizer state of one parameter vector, held as float64 arrays."""

    def __init__(self, theta, opt: OptCfg, m=None, v=None, t_opt: int = 0):
        self.opt = opt
        self.theta = as_f64(theta)
        n = self.theta.size
        if opt.kind == "adamw":
            self.m = as_f64(m) if m is not None else np.zeros(n)
            self.v = as_f64(v) if v is not None else np.zeros(n)
        else:
            self.m = self.v = None
        self.t_opt = int(t_opt)

    def optim_step(self, g, round_f32):
        """OptimStep(theta, g) of Algorithm 1 with the configured base optimizer."""
        if self.opt.kind == "gd":
            optim_step_gd(self.theta, g, self.opt.lr, round_f32)
        else:
            self.t_opt += 1
            optim_step_adamw(self.theta, self.m, self.v, g, self.t_opt, self.opt, round_f32)


def active_step(state: State, cfg: GxpoCfg, grad_fn, round_f32=False, trace=None):
    """One active step of Algorithm 1.

    `grad_fn(which, theta)` returns the float64 gradient for backward pass
    `which` in (0, 1, 2) evaluated at `theta` (the caller's three backward
    passes: at theta^t, theta^{t,1} and theta-tilde).  Returns ||g_slow||_2.
    `trace`, if a dict, receives copies of the intermediate points.
    """
    theta0 = state.theta.copy()
    g0 = as_f64(grad_fn(0, state.theta))
    state.optim_step(g0, round_f32)                      # first fast step
    if trace is not None:
        trace["theta1"] = state.theta.copy()
    g1 = as_f64(grad_fn(1, state.theta))
    state.optim_step(g1, round_f32)                      # second fast step
    if trace is not None:
        trace["theta2"] = state.theta.copy()
    if trace is not None:
        tilde, tk, sc = extrapolate(theta0, state.theta, g0, g1, cfg.K, cfg.alpha, cfg.delta,
                                    cfg.den_eps, round_f32, want_aux=True)
        trace["theta_K"], trace["scale"], trace["theta_tilde"] = tk, sc, tilde.copy()
    else:
        tilde = extrapolate(theta0, state.theta, g0, g1, cfg.K, cfg.alpha, cfg.delta,
                            cfg.den_eps, round_f32)
    state.theta = tilde                                  # reposition
    g_slow = as_f64(grad_fn(2, state.theta))
    state.optim_step(g_slow, round_f32)                  # slow correction
    return l2norm(g_slow)


def fallback_step(state: State, grad_fn, round_f32=False):
    """Single-pass step of the fallback phase: theta <- OptimStep(theta, g^{t,0})."""
    g0 = as_f64(grad_fn(0, state.theta))
    state.optim_step(g0, round_f32)


def train_step(state: State, gate: Gate, cfg: GxpoCfg, grad_fn, round_f32=False):
    """One iteration of Algorithm 1's outer loop.  Returns a small record."""
    if gate.active:
        nrm = active_step(state, cfg, grad_fn, round_f32)
        tripped, z, mu, sg = gate.update(nrm)
        return {"phase": "active", "norm": nrm, "z": z, "mu": mu, "sigma": sg,
                "tripped": tripped, "backward_passes": 3}
    fallback_step(state, grad_fn, round_f32)
    gate.fallback_tick()
    return {"phase": "fallback", "backward_passes": 1}
