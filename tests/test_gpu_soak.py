"""Many consecutive steps, four ways at once: the register-staged sweeps, the shared-memory
staged pair under the gradients-persist promise, the same with bfloat16-only probe points,
and the library's default dispatch.  The staged kernels hand tiles between a producer thread
and eight consumer warps through mbarriers; a race there would show up rarely and as a few
wrong elements, so the runs are long (120 steps, hundreds of tiles per CTA, gradients that
change every step) and compared bit for bit -- theta, m, v and the bfloat16 copies -- every
20 steps.  (The elementwise results of the register-staged sweeps are what the oracle parity
tests check.)"""
import numpy as np
import pytest

from paper_2605_06755_b200 import workloads
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def _make(b, torch, n_list, seed, variant, persist, mode):
    probs = [gu.Problem(*workloads.llm_inputs_numpy(n, seed + i, "bf16", zero_frac=0.03, warm_state=True))
             for i, n in enumerate(n_list)]
    cfg, opt = b.make_cfg(lr=1e-4, K=5, alpha=0.5, tau=1e9)           # the gate never trips
    ctx = b.Context(cfg, opt, b.BF16)
    ctx.bind([p.ptrs() for p in probs])
    ctx.tune(0, variant, 0)
    ctx.set_gradients_persist(persist)
    wbs = None
    if mode is not None:
        wbs = [torch.zeros(p.n, dtype=torch.bfloat16, device="cuda") for p in probs]
        ctx.bind_model_weights([w.data_ptr() for w in wbs], bf16_only=mode)
    return probs, ctx, wbs


@pytest.mark.parametrize("n_list", [[12_000_003], [3_000_017, 4_345_678, 65_536, 458_752, 7, 5_000_000]])
def test_staged_and_register_staged_sweeps_stay_bit_identical_over_many_steps(n_list):
    import torch
    from paper_2605_06755_b200 import binding as b
    ref = _make(b, torch, n_list, 900, 2, False, b.BF16_BESIDE)
    alts = [_make(b, torch, n_list, 900, 3, True, b.BF16_BESIDE),
            _make(b, torch, n_list, 900, 3, True, b.BF16_ONLY_PROBE_POINTS),
            _make(b, torch, n_list, 900, 0, True, None)]
    steps = 120
    for step in range(steps):
        for grp in [ref] + alts:                  # the gradients drift a little every step, the same everywhere
            for p in grp[0]:
                p.g1.mul_(1.0009765625)
                p.gs.mul_(0.9990234375)
        r0 = ref[1].active_step(allow_nonfinite=True, deferred=True)
        rs = [a[1].active_step(allow_nonfinite=True, deferred=True) for a in alts]
        if step % 20 == 19:
            torch.cuda.synchronize()
            for ai, a in enumerate(alts):
                for pi, (p, q) in enumerate(zip(ref[0], a[0])):
                    for nm in ("theta", "m", "v"):
                        x, y = getattr(p, nm).view(torch.int32), getattr(q, nm).view(torch.int32)
                        assert torch.equal(x, y), f"configuration {ai}, step {step}, tensor {pi}: {nm} differs"
                if a[2] is not None:
                    for w0, w1 in zip(ref[2], a[2]):
                        assert torch.equal(w0.view(torch.int16), w1.view(torch.int16))
                assert rs[ai].norm == pytest.approx(r0.norm, rel=1e-9)
    assert ref[1].optimizer_steps() == 3 * steps
    for grp in [ref] + alts:
        grp[1].close()
