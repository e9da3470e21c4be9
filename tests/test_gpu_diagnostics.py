"""Per-step diagnostics gathered inside the extrapolation sweep, against the oracle's
plain definitions on the same seeded inputs, for every call sequence; and the sweeps'
outputs must not change when diagnostics are switched on."""
import math

import numpy as np
import pytest

from oracle import gxpo_oracle as ora
from paper_2605_06755_b200 import workloads
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

SIZES = [3 * 32768 + 5, 2047, 1, 40003, 512, 70001]
OFFSETS = [0, 0, 0, 1, 0, 0]


def _binding():
    from paper_2605_06755_b200 import binding
    return binding


def _problems(grad_dtype, tame):
    probs = []
    for i, (n, off) in enumerate(zip(SIZES, OFFSETS)):
        if tame:                                     # ratios in [0.2, 1.2], like the paper's 0.5 +- 0.7
            rng = np.random.default_rng(900 + i)
            th = (0.02 * rng.standard_normal(n)).astype(np.float32)
            g0 = (1e-3 * rng.standard_normal(n)).astype(np.float32)
            g1 = (g0 * rng.uniform(0.2, 1.2, n)).astype(np.float32)
            gs = (g0 * rng.uniform(0.5, 1.0, n) + 1e-4 * rng.standard_normal(n)).astype(np.float32)
            g0[rng.random(n) < 0.03] = 0.0
            z = np.zeros(n, dtype=np.float32)
            arrs = (th, z, z.copy(), g0, g1, gs)
            if grad_dtype == "bf16":
                arrs = arrs[:3] + tuple(workloads.f32_to_bf16_bits(x) for x in arrs[3:])
        else:                                        # the benchmark recipe: heavy-tailed ratios
            arrs = workloads.llm_inputs_numpy(n, 900 + i, grad_dtype, zero_frac=0.03, warm_state=True)
        probs.append(gu.Problem(*arrs, offset_elems=off))
    return probs


def _oracle_diag(probs, gcfg, ocfg):
    """Oracle active step per tensor (for theta^{t,2}), then the diagnostics on the
    concatenation of all tensors."""
    th0, th2, g0, g1, gs = [], [], [], [], []
    for p in probs:
        st = p.oracle_state(ocfg)
        grads = p.oracle_grads()
        trace = {}
        ora.active_step(st, gcfg, lambda w, th: grads[w], round_f32=True, trace=trace)
        th0.append(p.np_in["theta"].astype(np.float64)); th2.append(trace["theta2"])
        g0.append(grads[0]); g1.append(grads[1]); gs.append(grads[2])
    cat = lambda xs: np.ascontiguousarray(np.concatenate(xs))
    return ora.active_diagnostics(cat(th0), cat(th2), cat(g0), cat(g1), cat(gs), gcfg.K, gcfg.delta, gcfg.den_eps)


@pytest.mark.parametrize("flow", ["deferred", "fused", "unfused"])
@pytest.mark.parametrize("grad_dtype,kind,tame", [("bf16", "adamw", True), ("bf16", "adamw", False),
                                                   ("f32", "gd", True)])
@pytest.mark.parametrize("K", [3, 5, 10])
@pytest.mark.parametrize("variant", [0, 3])            # 3: the shared-memory staged sweeps gather them too
def test_diagnostics_match_the_oracle(flow, grad_dtype, kind, tame, K, variant):
    b = _binding()
    probs = _problems(grad_dtype, tame)
    cfg, opt = b.make_cfg(kind=b.OPT_ADAMW if kind == "adamw" else b.OPT_GD, lr=1e-3, K=K, alpha=0.5)
    ctx = b.Context(cfg, opt, b.BF16 if grad_dtype == "bf16" else b.F32)
    ctx.bind([p.ptrs() for p in probs])
    ctx.tune(0, variant, 0)
    ctx.enable_diagnostics(True)
    gcfg, ocfg = gu.ora_cfgs(cfg, opt)
    want = _oracle_diag(probs, gcfg, ocfg)
    res = ctx.active_step(allow_nonfinite=True, fused=(flow == "fused"), deferred=(flow == "deferred"))
    got = ctx.get_diagnostics()
    n = sum(SIZES)
    assert got.n == n and got.n_active == want["n_active"]
    # a ratio or scale within a rounding of the float32 overflow threshold may be classed
    # differently by float32 and float64 arithmetic: allow a couple of such coordinates
    assert abs(got.n_irregular - want["n_irregular"]) <= 2
    assert got.inactive_frac == pytest.approx(want["inactive_frac"], abs=1e-12)
    assert 0.02 < got.inactive_frac < 0.05
    for k in ("g0_norm", "g1_norm", "gslow_norm"):
        assert getattr(got, k) == pytest.approx(want[k], rel=gu.RTOL_NORM), k
    assert got.gslow_norm == pytest.approx(res.norm, rel=1e-12)
    assert got.cos_g0_gslow == pytest.approx(want["cos_g0_gslow"], rel=1e-5, abs=1e-7)
    if tame:
        # theta^{t,2} - theta^t carries the float32 rounding of two optimizer steps, so the
        # displacement figure is compared at 1e-4; ratio and scale are exact to rounding
        assert got.n_irregular == want["n_irregular"]
        assert got.ratio_mean == pytest.approx(want["ratio_mean"], rel=1e-5)
        assert got.ratio_std == pytest.approx(want["ratio_std"], rel=1e-5)
        assert got.scale_mean == pytest.approx(want["scale_mean"], rel=1e-5)
        assert got.disp_ratio == pytest.approx(want["disp_ratio"], rel=1e-4)
        assert 0.6 < got.ratio_mean < 0.8
    elif got.n_irregular == want["n_irregular"]:
        # heavy tails: a handful of enormous ratios carry the sums; same coordinates, same sums
        assert got.ratio_mean == pytest.approx(want["ratio_mean"], rel=1e-4)
        assert got.ratio_std == pytest.approx(want["ratio_std"], rel=1e-4)
        assert got.scale_mean == pytest.approx(want["scale_mean"], rel=1e-4)
    ctx.close()


@pytest.mark.parametrize("variant", [0, 3])
def test_switching_diagnostics_on_changes_no_output_and_call_order_is_checked(variant):
    b = _binding()
    outs = []
    for on in (False, True):
        probs = _problems("bf16", tame=False)
        cfg, opt = b.make_cfg(lr=1e-3, K=5)
        ctx = b.Context(cfg, opt, b.BF16)
        ctx.bind([p.ptrs() for p in probs])
        ctx.tune(0, variant, 0)
        with pytest.raises(b.GxpoError) as e:
            ctx.get_diagnostics()
        assert e.value.status == b.ERR_STATE
        ctx.enable_diagnostics(on)
        res = ctx.active_step(allow_nonfinite=True, deferred=True)
        if on:
            d = ctx.get_diagnostics()
            assert d.n == sum(SIZES) and d.g0_norm > 0
            ctx.probe_step_deferred()
            with pytest.raises(b.GxpoError) as e:
                ctx.enable_diagnostics(False)            # mid-step
            assert e.value.status == b.ERR_STATE
            with pytest.raises(b.GxpoError):
                ctx.get_diagnostics()
        else:
            with pytest.raises(b.GxpoError):
                ctx.get_diagnostics()
        outs.append(([gu.to_host_f64(p.theta) for p in probs], [gu.to_host_f64(p.m) for p in probs], res.norm))
        ctx.close()
    for a, c in zip(outs[0][0] + outs[0][1], outs[1][0] + outs[1][1]):
        np.testing.assert_array_equal(a, c)
    assert outs[0][2] == outs[1][2]


def test_cosine_is_nan_when_g_slow_shares_g0s_buffer():
    b = _binding()
    n = 50000
    th, m, v, g0, g1, gs = workloads.llm_inputs_numpy(n, 5, "bf16")
    pr = gu.Problem(th, m, v, g0, g1, gs)
    cfg, opt = b.make_cfg(lr=1e-3)
    ctx = b.Context(cfg, opt, b.BF16)
    ctx.bind([b.tensor_ptrs(pr.theta, pr.work, pr.m, pr.v, pr.g0, pr.g1, pr.g0)])
    ctx.enable_diagnostics(True)
    ctx.active_step(allow_nonfinite=True, deferred=True)
    d = ctx.get_diagnostics()
    assert math.isnan(d.cos_g0_gslow)
    assert d.gslow_norm == pytest.approx(d.g0_norm, rel=1e-6)      # float32 partial sums inside the slow sweep
    ctx.close()


def test_long_list_diagnostics_in_the_default_launch_configuration():
    """A flat list long enough that the default picks the shared-memory staged sweep
    (200,000,003 parameters, ragged tail): the counts against a library count of
    |g0| > delta, the norms against float64 library reductions, every figure against the
    register-staged sweep's (whose figures the oracle checks above), and the outputs
    bit for bit against a run with diagnostics off."""
    import argparse
    import gc

    import torch

    import bench
    b = _binding()
    runs = {}
    for name, variant, on in (("staged", 0, True), ("registers", 2, True), ("plain", 0, False)):
        gc.collect()
        torch.cuda.empty_cache()
        args = argparse.Namespace(workload="flat", layers=0, params=200_000_003)
        free, _ = torch.cuda.mem_get_info()
        shapes, desc, alias = bench.plan_workload(args, free)
        d, ptrs, keep = bench.build_device_workload(torch, b, shapes, 77, alias)
        assert d == 200_000_003
        cfg, opt = b.make_cfg(lr=1e-3, K=5, alpha=0.5)
        ctx = b.Context(cfg, opt, b.BF16)
        ctx.bind(ptrs)
        ctx.tune(0, variant, 0)
        ctx.enable_diagnostics(on)
        ctx.set_gradients_persist(name == "staged")      # not used while diagnostics are on: no effect
        g0, g1 = keep[4], keep[5]
        if name == "staged":
            n_active = 0
            sq0 = sq1 = 0.0
            for s in range(0, d, 1 << 26):
                a, c = g0[s:s + (1 << 26)].double(), g1[s:s + (1 << 26)].double()
                n_active += int((a.abs() > cfg.delta).sum().item())
                sq0 += float(torch.dot(a, a).item())
                sq1 += float(torch.dot(c, c).item())
                del a, c
        res = ctx.active_step(allow_nonfinite=True, deferred=True)
        diag = ctx.get_diagnostics() if on else None
        runs[name] = (diag, res.norm, keep[0].clone(), keep[2].clone(), keep[3].clone())
        ctx.close()
        del keep, g0, g1
    got, ref = runs["staged"][0], runs["registers"][0]
    assert got.n == 200_000_003 and got.n_active == n_active
    # a vector's 8 squares are added up in float32 before they reach the float64 sums
    assert got.g0_norm == pytest.approx(math.sqrt(sq0), rel=1e-6)
    assert got.g1_norm == pytest.approx(math.sqrt(sq1), rel=1e-6)
    assert got.gslow_norm == pytest.approx(runs["staged"][1], rel=1e-12)
    for k in ("n", "n_active", "n_irregular"):
        assert getattr(got, k) == getattr(ref, k), k
    # float64 sums of the same float32 terms, grouped by a different grid
    for k in ("g0_norm", "g1_norm", "gslow_norm", "ratio_mean", "ratio_std", "scale_mean", "disp_ratio",
              "cos_g0_gslow", "inactive_frac"):
        assert getattr(got, k) == pytest.approx(getattr(ref, k), rel=1e-9), k
    for i in (2, 3, 4):
        assert torch.equal(runs["staged"][i], runs["plain"][i])
        assert torch.equal(runs["staged"][i], runs["registers"][i])
    assert runs["staged"][1] == runs["plain"][1]


@pytest.mark.parametrize("variant", [0, 3])
@pytest.mark.parametrize("K", [3, 5])
def test_terms_beyond_float32_squares_are_summed_in_float64(K, variant):
    """The vector paths pre-sum a vector's terms in float32 and must notice when that
    would overflow: planted coordinates with r = 1e16 (r^2 = 1e32), g0 = 1e16 and
    (d * scale)^2 far above 3e38 still give the oracle's float64 figures."""
    b = _binding()
    probs = _problems("f32", tame=True)
    big = probs[0]
    g0, g1 = big.np_in["g0"].copy(), big.np_in["g1"].copy()
    for idx, a, c in ((100, 1e-3, 1e13), (8 * 4096 + 3, 1e16, 5e15), (70000, 1e-3, 2e13)):
        g0[idx], g1[idx] = a, c
    probs[0] = gu.Problem(big.np_in["theta"], big.np_in["m"], big.np_in["v"], g0, g1, big.np_in["gs"])
    cfg, opt = b.make_cfg(kind=b.OPT_GD, lr=1e-3, K=K, alpha=0.5)
    ctx = b.Context(cfg, opt, b.F32)
    ctx.bind([p.ptrs() for p in probs])
    ctx.tune(0, variant, 0)
    ctx.enable_diagnostics(True)
    gcfg, ocfg = gu.ora_cfgs(cfg, opt)
    want = _oracle_diag(probs, gcfg, ocfg)
    ctx.active_step(allow_nonfinite=True, deferred=True)
    got = ctx.get_diagnostics()
    assert got.n_active == want["n_active"] and got.n_irregular == want["n_irregular"]
    assert want["g0_norm"] > 9e15                                       # the planted terms carry the sums
    if K == 3:                                                           # (for K = 5 the scale of r = 1e16 is not a float32)
        assert want["ratio_std"] > 1e12 and want["n_irregular"] == 0
    for k in ("g0_norm", "g1_norm", "ratio_mean", "ratio_std", "scale_mean", "disp_ratio"):
        assert math.isfinite(getattr(got, k)), k
        assert getattr(got, k) == pytest.approx(want[k], rel=1e-5), k
    ctx.close()
