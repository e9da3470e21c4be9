"""ctypes binding of the GXPO C ABI (include/gxpo.h).

Argument marshalling only: every step of the update runs in the CUDA kernels of
libgxpo.so.  There is no fallback of any kind: if the shared library is missing
this module raises at import.  Tensors are passed as raw device pointers
(`tensor.data_ptr()`); torch is used by callers for memory and streams only.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional, Sequence

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libgxpo.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2605_06755_b200.build` "
        "(or __graft_entry__.build()).  There is no CPU fallback.")

_lib = ctypes.CDLL(LIB_PATH)

OK, ERR_INVALID_ARG, ERR_ALIGNMENT, ERR_STATE, ERR_CUDA, ERR_TIMEOUT, ERR_NONFINITE = range(7)
OPT_GD, OPT_ADAMW = 0, 1
F32, BF16 = 0, 1
PLACE_PINGPONG, PLACE_SNAPSHOT = 0, 1
BF16_BESIDE, BF16_ONLY_THETA1, BF16_ONLY_PROBE_POINTS = 0, 1, 2


class OptCfg(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int), ("lr", ctypes.c_double), ("beta1", ctypes.c_double),
                ("beta2", ctypes.c_double), ("eps", ctypes.c_double),
                ("weight_decay", ctypes.c_double)]


class Cfg(ctypes.Structure):
    _fields_ = [("K", ctypes.c_int), ("alpha", ctypes.c_float), ("delta", ctypes.c_float),
                ("den_eps", ctypes.c_float), ("tau", ctypes.c_double),
                ("gate_eps", ctypes.c_double), ("window", ctypes.c_int),
                ("min_history", ctypes.c_int), ("std_ddof", ctypes.c_int),
                ("placement", ctypes.c_int)]


class Tensor(ctypes.Structure):
    _fields_ = [("theta", ctypes.c_void_p), ("work", ctypes.c_void_p), ("m", ctypes.c_void_p),
                ("v", ctypes.c_void_p), ("g0", ctypes.c_void_p), ("g1", ctypes.c_void_p),
                ("g_slow", ctypes.c_void_p), ("n", ctypes.c_longlong)]


class GateResult(ctypes.Structure):
    _fields_ = [("active", ctypes.c_int), ("tripped", ctypes.c_int), ("t", ctypes.c_longlong),
                ("s_star", ctypes.c_longlong), ("norm", ctypes.c_double), ("z", ctypes.c_double),
                ("mu", ctypes.c_double), ("sigma", ctypes.c_double)]


class Diagnostics(ctypes.Structure):
    _fields_ = [(k, ctypes.c_double) for k in
                ("g0_norm", "g1_norm", "gslow_norm", "cos_g0_gslow", "ratio_mean", "ratio_std",
                 "scale_mean", "disp_ratio", "inactive_frac")] + \
               [(k, ctypes.c_longlong) for k in ("n", "n_active", "n_irregular")]


class SweepInfo(ctypes.Structure):
    _fields_ = [("kernel", ctypes.c_char * 48), ("staged", ctypes.c_int), ("grid", ctypes.c_int),
                ("bytes_read_per_param", ctypes.c_int), ("bytes_written_per_param", ctypes.c_int),
                ("extra_launches", ctypes.c_int), ("valid", ctypes.c_int)]


_vp = ctypes.c_void_p
_sigs = {
    "gxpo_default_cfg": (None, [ctypes.POINTER(Cfg), ctypes.POINTER(OptCfg)]),
    "gxpo_create": (ctypes.c_int, [ctypes.POINTER(Cfg), ctypes.POINTER(OptCfg), ctypes.c_int,
                                   ctypes.POINTER(_vp)]),
    "gxpo_destroy": (None, [_vp]),
    "gxpo_bind": (ctypes.c_int, [_vp, ctypes.POINTER(Tensor), ctypes.c_int]),
    "gxpo_bind_model_weights": (ctypes.c_int, [_vp, ctypes.POINTER(_vp), ctypes.c_int, ctypes.c_int]),
    "gxpo_probe_step": (ctypes.c_int, [_vp, ctypes.c_int, _vp]),
    "gxpo_probe_step_deferred": (ctypes.c_int, [_vp, _vp]),
    "gxpo_extrapolate": (ctypes.c_int, [_vp, _vp]),
    "gxpo_probe_extrapolate": (ctypes.c_int, [_vp, _vp]),
    "gxpo_slow_step": (ctypes.c_int, [_vp, _vp]),
    "gxpo_gate_update": (ctypes.c_int, [_vp, _vp, ctypes.POINTER(GateResult)]),
    "gxpo_gate_update_async": (ctypes.c_int, [_vp, _vp]),
    "gxpo_gate_last": (ctypes.c_int, [_vp, ctypes.POINTER(GateResult)]),
    "gxpo_set_sumsq_buffer": (ctypes.c_int, [_vp, _vp]),
    "gxpo_set_grad_scale": (ctypes.c_int, [_vp, ctypes.c_int, _vp]),
    "gxpo_clip_grad_norm": (ctypes.c_int, [_vp, ctypes.c_int, ctypes.c_double, _vp]),
    "gxpo_enable_diagnostics": (ctypes.c_int, [_vp, ctypes.c_int]),
    "gxpo_set_gradients_persist": (ctypes.c_int, [_vp, ctypes.c_int]),
    "gxpo_get_diagnostics": (ctypes.c_int, [_vp, _vp, ctypes.POINTER(Diagnostics)]),
    "gxpo_gate_peek": (ctypes.c_int, [_vp, ctypes.POINTER(ctypes.c_int),
                                      ctypes.POINTER(ctypes.c_longlong),
                                      ctypes.POINTER(ctypes.c_longlong)]),
    "gxpo_optimizer_steps": (ctypes.c_longlong, [_vp]),
    "gxpo_backward_passes": (ctypes.c_longlong, [_vp]),
    "gxpo_state_export": (ctypes.c_int, [_vp, _vp, ctypes.POINTER(ctypes.c_size_t)]),
    "gxpo_state_import": (ctypes.c_int, [_vp, _vp, ctypes.c_size_t]),
    "gxpo_step_host": (ctypes.c_int, [_vp, ctypes.POINTER(Tensor), ctypes.c_int,
                                      ctypes.c_longlong, _vp, ctypes.POINTER(GateResult)]),
    "gxpo_tune": (ctypes.c_int, [_vp, ctypes.c_int, ctypes.c_int, ctypes.c_int]),
    "gxpo_selftest_bounded_wait": (ctypes.c_int, [_vp, _vp]),
    "gxpo_selftest_inject_timeout": (ctypes.c_int, [_vp, _vp]),
    "gxpo_launch_count": (ctypes.c_longlong, [_vp]),
    "gxpo_last_sweep": (ctypes.c_int, [_vp, ctypes.POINTER(SweepInfo)]),
    "gxpo_last_error": (ctypes.c_char_p, [_vp]),
    "gxpo_status_string": (ctypes.c_char_p, [ctypes.c_int]),
    "gxpo_quad_grad": (ctypes.c_int, [_vp, _vp, _vp, _vp, ctypes.c_longlong, _vp]),
    "gxpo_quad_active_step": (ctypes.c_int, [_vp, _vp, _vp, ctypes.c_longlong, ctypes.c_float,
                                             ctypes.c_int, ctypes.c_float, ctypes.c_float,
                                             ctypes.c_float, _vp, _vp, _vp]),
    "gxpo_quad_scratch_bytes": (ctypes.c_size_t, []),
    "gxpo_slow_step_noalloc": (ctypes.c_int, [_vp, _vp, _vp, _vp, ctypes.c_longlong, ctypes.c_int,
                                              ctypes.POINTER(OptCfg), ctypes.c_longlong, _vp, _vp,
                                              ctypes.c_char_p, ctypes.c_size_t]),
}
for _name, (_res, _args) in _sigs.items():
    _f = getattr(_lib, _name)
    _f.restype = _res
    _f.argtypes = _args

EXPORTED_SYMBOLS = tuple(_sigs)


class GxpoError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"gxpo status {status} ({_lib.gxpo_status_string(status).decode()}): {message}")
        self.status = status


def default_cfg():
    cfg, opt = Cfg(), OptCfg()
    _lib.gxpo_default_cfg(ctypes.byref(cfg), ctypes.byref(opt))
    return cfg, opt


def make_cfg(**kw):
    """Defaults of gxpo_default_cfg with keyword overrides; optimizer fields are
    kind/lr/beta1/beta2/eps/weight_decay, everything else goes to the GXPO cfg."""
    cfg, opt = default_cfg()
    opt_fields = {f[0] for f in OptCfg._fields_}
    for k, v in kw.items():
        if k in opt_fields:
            setattr(opt, k, v)
        elif k in {f[0] for f in Cfg._fields_}:
            setattr(cfg, k, v)
        else:
            raise TypeError(f"unknown configuration field {k!r}")
    return cfg, opt


@dataclass
class TensorPtrs:
    """Raw pointers of one parameter tensor (device pointers for `bind`, host
    pointers for `step_host`)."""
    theta: int
    work: int
    m: int
    v: int
    g0: int
    g1: int
    g_slow: int
    n: int


def _pack(list_: Sequence[TensorPtrs]):
    arr = (Tensor * max(1, len(list_)))()
    for i, t in enumerate(list_):
        arr[i] = Tensor(t.theta or None, t.work or None, t.m or None, t.v or None,
                        t.g0 or None, t.g1 or None, t.g_slow or None, t.n)
    return arr


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        return None
    if isinstance(stream, int):
        return stream or None
    return int(stream.cuda_stream) or None       # torch.cuda.Stream


class Context:
    """Owns one gxpo_ctx.  Method names follow the C entry points."""

    def __init__(self, cfg: Cfg, opt: OptCfg, grad_dtype: int):
        self._h = _vp()
        st = _lib.gxpo_create(ctypes.byref(cfg), ctypes.byref(opt), grad_dtype,
                              ctypes.byref(self._h))
        if st != OK:
            self._h = _vp()
            raise GxpoError(st, "gxpo_create rejected the configuration or could not allocate")
        self.cfg, self.opt, self.grad_dtype = cfg, opt, grad_dtype

    def close(self):
        if self._h:
            _lib.gxpo_destroy(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int):
        if st != OK:
            raise GxpoError(st, _lib.gxpo_last_error(self._h).decode())

    def bind(self, tensors: Sequence[TensorPtrs]):
        self._check(_lib.gxpo_bind(self._h, _pack(tensors), len(tensors)))

    def bind_model_weights(self, ptrs, only_bf16_theta1: bool = False, bf16_only: int = 0):
        """ptrs: device pointers of the bfloat16 copies, one per bound tensor (0 = none),
        or None to unbind.  bf16_only: BF16_BESIDE, BF16_ONLY_THETA1 (also selected by
        only_bf16_theta1=True) or BF16_ONLY_PROBE_POINTS."""
        if ptrs is None:
            self._check(_lib.gxpo_bind_model_weights(self._h, None, 0, 0))
            return
        arr = (_vp * max(1, len(ptrs)))(*[p or None for p in ptrs])
        mode = int(bf16_only) if bf16_only else (1 if only_bf16_theta1 else 0)
        self._check(_lib.gxpo_bind_model_weights(self._h, arr, len(ptrs), mode))

    def probe_step(self, which: int, stream=None):
        self._check(_lib.gxpo_probe_step(self._h, which, _stream_ptr(stream)))

    def probe_step_deferred(self, stream=None):
        self._check(_lib.gxpo_probe_step_deferred(self._h, _stream_ptr(stream)))

    def extrapolate(self, stream=None):
        self._check(_lib.gxpo_extrapolate(self._h, _stream_ptr(stream)))

    def probe_extrapolate(self, stream=None):
        self._check(_lib.gxpo_probe_extrapolate(self._h, _stream_ptr(stream)))

    def slow_step(self, stream=None):
        self._check(_lib.gxpo_slow_step(self._h, _stream_ptr(stream)))

    def gate_update(self, stream=None, allow_nonfinite: bool = False) -> GateResult:
        res = GateResult()
        st = _lib.gxpo_gate_update(self._h, _stream_ptr(stream), ctypes.byref(res))
        if st == ERR_NONFINITE and allow_nonfinite:
            return res
        self._check(st)
        return res

    def gate_update_async(self, stream=None):
        self._check(_lib.gxpo_gate_update_async(self._h, _stream_ptr(stream)))

    def gate_last(self, allow_nonfinite: bool = False) -> GateResult:
        res = GateResult()
        st = _lib.gxpo_gate_last(self._h, ctypes.byref(res))
        if st == ERR_NONFINITE and allow_nonfinite:
            return res
        self._check(st)
        return res

    def set_sumsq_buffer(self, dev_ptr: int):
        self._check(_lib.gxpo_set_sumsq_buffer(self._h, dev_ptr or None))

    def set_grad_scale(self, which: int, scale_ptr: int):
        self._check(_lib.gxpo_set_grad_scale(self._h, which, scale_ptr or None))

    def clip_grad_norm(self, which: int, max_norm: float, stream=None):
        self._check(_lib.gxpo_clip_grad_norm(self._h, which, max_norm, _stream_ptr(stream)))

    def enable_diagnostics(self, on: bool = True):
        self._check(_lib.gxpo_enable_diagnostics(self._h, 1 if on else 0))

    def set_gradients_persist(self, on: bool):
        self._check(_lib.gxpo_set_gradients_persist(self._h, 1 if on else 0))

    def get_diagnostics(self, stream=None) -> Diagnostics:
        out = Diagnostics()
        self._check(_lib.gxpo_get_diagnostics(self._h, _stream_ptr(stream), ctypes.byref(out)))
        return out

    def gate_peek(self):
        a, s, t = ctypes.c_int(), ctypes.c_longlong(), ctypes.c_longlong()
        self._check(_lib.gxpo_gate_peek(self._h, ctypes.byref(a), ctypes.byref(s), ctypes.byref(t)))
        return bool(a.value), s.value, t.value

    def optimizer_steps(self) -> int:
        return _lib.gxpo_optimizer_steps(self._h)

    def backward_passes(self) -> int:
        return _lib.gxpo_backward_passes(self._h)

    def state_export(self) -> bytes:
        n = ctypes.c_size_t(0)
        self._check(_lib.gxpo_state_export(self._h, None, ctypes.byref(n)))
        buf = ctypes.create_string_buffer(n.value)
        self._check(_lib.gxpo_state_export(self._h, buf, ctypes.byref(n)))
        return buf.raw[:n.value]

    def state_import(self, blob: bytes):
        buf = ctypes.create_string_buffer(blob, len(blob))
        self._check(_lib.gxpo_state_import(self._h, buf, len(blob)))

    def step_host(self, tensors: Sequence[TensorPtrs], staging_elems: int = 0, stream=None,
                  allow_nonfinite: bool = False) -> GateResult:
        res = GateResult()
        st = _lib.gxpo_step_host(self._h, _pack(tensors), len(tensors), staging_elems,
                                 _stream_ptr(stream), ctypes.byref(res))
        if st == ERR_NONFINITE and allow_nonfinite:
            return res
        self._check(st)
        return res

    def tune(self, ctas_per_sm: int = 0, variant: int = 0, unit_tiles: int = 0):
        self._check(_lib.gxpo_tune(self._h, ctas_per_sm, variant, unit_tiles))

    def selftest_bounded_wait(self, stream=None) -> int:
        """Returns the status code (ERR_TIMEOUT is the expected outcome)."""
        return _lib.gxpo_selftest_bounded_wait(self._h, _stream_ptr(stream))

    def selftest_inject_timeout(self, stream=None):
        self._check(_lib.gxpo_selftest_inject_timeout(self._h, _stream_ptr(stream)))

    def launch_count(self) -> int:
        return _lib.gxpo_launch_count(self._h)

    def last_sweep(self) -> SweepInfo:
        out = SweepInfo()
        self._check(_lib.gxpo_last_sweep(self._h, ctypes.byref(out)))
        return out

    # -- convenience: the calls of one active step in Algorithm 1's order, for callers
    #    whose three gradient buffers are already filled (benchmarks, replay) --------
    def active_step(self, stream=None, allow_nonfinite: bool = False, fused: bool = False,
                    deferred: bool = False) -> GateResult:
        if deferred:
            self.probe_step_deferred(stream)
            self.probe_extrapolate(stream)
        elif fused:
            self.probe_step(0, stream)
            self.probe_extrapolate(stream)
        else:
            self.probe_step(0, stream)
            self.probe_step(1, stream)
            self.extrapolate(stream)
        self.slow_step(stream)
        return self.gate_update(stream, allow_nonfinite)


def quad_grad(theta_ptr: int, a_ptr: int, b_ptr: int, g_ptr: int, n: int, stream=None):
    st = _lib.gxpo_quad_grad(theta_ptr, a_ptr, b_ptr, g_ptr, n, _stream_ptr(stream))
    if st != OK:
        raise GxpoError(st, "gxpo_quad_grad")


def quad_scratch_bytes() -> int:
    return _lib.gxpo_quad_scratch_bytes()


def quad_active_step(theta_ptr, a_ptr, b_ptr, n, lr, K, alpha, delta, den_eps, sumsq_ptr,
                     scratch_ptr, stream=None):
    st = _lib.gxpo_quad_active_step(theta_ptr, a_ptr, b_ptr, n, lr, K, alpha, delta, den_eps,
                                    sumsq_ptr, scratch_ptr, _stream_ptr(stream))
    if st != OK:
        raise GxpoError(st, "gxpo_quad_active_step")


NOALLOC_MAX_PARAMS = 2147483648


def slow_step_noalloc(theta_ptr, m_ptr, v_ptr, g_slow_ptr, n, grad_dtype, opt: OptCfg, t_opt,
                      sumsq_ptr, stream=None):
    """gxpo_slow_step_noalloc: the slow correction on one flat buffer, in place, with
    sum(g_slow^2) written to the device double at `sumsq_ptr`.  Needs no Context and
    allocates nothing; see include/gxpo.h for the size limit and the sharing rules."""
    err = ctypes.create_string_buffer(512)
    st = _lib.gxpo_slow_step_noalloc(theta_ptr or None, m_ptr or None, v_ptr or None,
                                     g_slow_ptr or None, n, grad_dtype, ctypes.byref(opt), t_opt,
                                     sumsq_ptr or None, _stream_ptr(stream), err, len(err))
    if st != OK:
        raise GxpoError(st, err.value.decode())


def tensor_ptrs(theta, work, m, v, g0, g1, g_slow) -> TensorPtrs:
    """TensorPtrs from objects with data_ptr()/numel() (torch tensors, device or
    pinned host); m, v and work may be None."""
    def p(x):
        return 0 if x is None else int(x.data_ptr())
    return TensorPtrs(p(theta), p(work), p(m), p(v), p(g0), p(g1), p(g_slow), int(theta.numel()))
