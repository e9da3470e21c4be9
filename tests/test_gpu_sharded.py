"""The sharded step on the GPU (one process per GPU in production; here both shards'
contexts live on the one GPU, which needs no peer memory and no kernel that waits on
another): a tensor list is cut in two by sharding.partition_by_slice / partition_by_tensor,
each half is bound to a context of its own with a caller-owned sum-of-squares scalar
(gxpo_set_sumsq_buffer), and between gxpo_slow_step and gxpo_gate_update the two scalars
are added on the stream -- the one exchange of the sharded update, which NCCL performs
across GPUs.  Over a 12-step stream whose ||g_slow|| jumps by 8x at step 8

  * both gates must flip at the oracle's step, and with the unsharded context's gate,
  * every element of theta, m, v must equal the unsharded context's bit for bit, and
  * must match the CPU oracle within the chained-step tolerance.
"""
import math

import numpy as np
import pytest

from oracle import gxpo_oracle as ora
from paper_2605_06755_b200 import sharding, workloads
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

SIZES = [4096, 70001, 512, 33000 + 3 * 32768, 17]
STEPS, JUMP_AT = 12, 8


def _inputs():
    out = []
    for i, n in enumerate(SIZES):
        rng = np.random.default_rng(400 + i)
        th = (0.02 * rng.standard_normal(n)).astype(np.float32)
        g0 = (1e-3 * rng.standard_normal(n)).astype(np.float32)
        g1 = (g0 * rng.uniform(0.2, 1.2, n)).astype(np.float32)
        gs = (g0 * rng.uniform(0.5, 1.0, n)).astype(np.float32)
        z = np.zeros(n, dtype=np.float32)
        out.append((th, z, z.copy(), workloads.f32_to_bf16_bits(g0), workloads.f32_to_bf16_bits(g1),
                    workloads.f32_to_bf16_bits(gs)))
    return out


def _oracle_run(data):
    """Algorithm 1 over the whole list on the CPU; returns (s_star, phases, norms, states)."""
    cfg = ora.GxpoCfg(K=5, alpha=0.5, delta=float(np.float32(1e-8)), tau=0.5, window=20)
    opt = ora.OptCfg(kind="adamw", lr=1e-3)
    gate = ora.Gate(cfg)
    states = [ora.State(d[0], opt, d[1], d[2]) for d in data]
    grads = [[ora.bf16_bits_to_f64(g) for g in d[3:]] for d in data]
    phases, norms = [], []
    for t in range(STEPS):
        mult = 8.0 if t == JUMP_AT else 1.0
        if gate.active:
            total = 0.0
            for st, g in zip(states, grads):
                gg = [g[0], g[1], g[2] * mult]
                ora.active_step(st, cfg, lambda w, th, gg=gg: gg[w], round_f32=True)
                total += ora.sum_squares(gg[2])
            norms.append(math.sqrt(total))
            gate.update(norms[-1])
            phases.append("a")
        else:
            for st, g in zip(states, grads):
                ora.fallback_step(st, lambda w, th, g=g: g[w], round_f32=True)
            gate.fallback_tick()
            phases.append("f")
    return gate.s_star, "".join(phases), norms, states


def _step_calls(ctx, flow):
    if flow == "unfused":
        ctx.probe_step(0)
        ctx.probe_step(1)
        ctx.extrapolate()
    else:
        ctx.probe_step_deferred()
        ctx.probe_extrapolate()


@pytest.mark.parametrize("mode", ["slice", "tensor"])
@pytest.mark.parametrize("flow,variant", [("unfused", 0), ("deferred", 0), ("deferred", 3)])
def test_two_shards_on_one_gpu_flip_together_and_equal_the_unsharded_run(mode, flow, variant):
    import torch
    from paper_2605_06755_b200 import binding as b
    data = _inputs()
    s_ref, phases_ref, norms_ref, ora_states = _oracle_run(data)
    assert s_ref == JUMP_AT + 1 and phases_ref == "a" * (JUMP_AT + 1) + "f" * (STEPS - JUMP_AT - 1)

    whole = [gu.Problem(*d) for d in data]        # what the unsharded context updates
    split = [gu.Problem(*d) for d in data]        # what the two shard contexts update, piece by piece
    cfg, opt = b.make_cfg(lr=1e-3, K=5, alpha=0.5)

    def make_ctx(ptrs):
        ctx = b.Context(cfg, opt, b.BF16)
        ctx.tune(0, variant, 0)
        ctx.bind(ptrs)
        ctx.set_gradients_persist(flow == "deferred")   # with variant 3: m, v written once, by the replaying slow sweep
        return ctx

    ref = make_ctx([p.ptrs() for p in whole])
    parts = (sharding.partition_by_slice if mode == "slice" else sharding.partition_by_tensor)(SIZES, 2)
    sharding.check_partition(SIZES, parts)
    assert all(len(pieces) > 0 for pieces in parts)
    sums = [torch.full((1,), float("nan"), dtype=torch.float64, device="cuda") for _ in parts]
    shards = []
    for pieces, buf in zip(parts, sums):
        ptrs = []
        for pc in pieces:
            p = split[pc.tensor]
            o = pc.offset
            ptrs.append(b.TensorPtrs(p.theta.data_ptr() + 4 * o, p.work.data_ptr() + 4 * o, p.m.data_ptr() + 4 * o,
                                     p.v.data_ptr() + 4 * o, p.g0.data_ptr() + 2 * o, p.g1.data_ptr() + 2 * o,
                                     p.gs.data_ptr() + 2 * o, pc.length))
        ctx = make_ctx(ptrs)
        ctx.set_sumsq_buffer(buf.data_ptr())
        shards.append(ctx)

    phases, norms = [], []
    for t in range(STEPS):
        mult = 8.0 if t == JUMP_AT else 1.0
        peeks = [c.gate_peek() for c in [ref] + shards]
        assert len({pk[0] for pk in peeks}) == 1 and all(pk[2] == t for pk in peeks)
        if peeks[0][0]:
            for c in [ref] + shards:
                _step_calls(c, flow)
            for probs in (whole, split):
                for p in probs:
                    p.gs.mul_(mult)                         # the third backward pass writes g_slow (x8 is exact)
            for c in [ref] + shards:
                c.slow_step()
            # the exchange: every shard ends up with the sum over all shards (an all-reduce across
            # GPUs in production), enqueued on the same stream between the two calls
            total = sums[0] + sums[1]
            for buf in sums:
                buf.copy_(total)
            res = [c.gate_update() for c in [ref] + shards]
            for probs in (whole, split):
                for p in probs:
                    p.gs.div_(mult)
            assert res[1].norm == res[2].norm               # both shards saw the same scalar
            assert res[1].norm == pytest.approx(res[0].norm, rel=1e-12)
            assert len({(r.tripped, r.s_star, r.active) for r in res}) == 1
            norms.append(res[1].norm)
            phases.append("a")
        else:
            for c in [ref] + shards:
                c.probe_step(-1)
            phases.append("f")
    torch.cuda.synchronize()
    assert "".join(phases) == phases_ref
    for c in [ref] + shards:
        assert c.gate_peek()[1] == s_ref
        assert c.optimizer_steps() == 3 * (JUMP_AT + 1) + (STEPS - JUMP_AT - 1)
    for got, want in zip(norms, norms_ref):
        assert got == pytest.approx(want, rel=gu.RTOL_NORM)
    for i, (pw, ps, st) in enumerate(zip(whole, split, ora_states)):
        for name in ("theta", "m", "v"):
            a, s_ = getattr(pw, name), getattr(ps, name)
            assert torch.equal(a, s_), f"tensor {i} {name}: sharded and unsharded runs differ"
        # 12 chained steps: the bound the other multi-step tests use
        gu.assert_close(gu.to_host_f64(ps.theta), st.theta, f"tensor {i} theta after {STEPS} steps", rtol=5e-6)
        gu.assert_close(gu.to_host_f64(ps.m), st.m, f"tensor {i} m", rtol=5e-6)
        gu.assert_close(gu.to_host_f64(ps.v), st.v, f"tensor {i} v", rtol=5e-6)
    for c in [ref] + shards:
        c.close()


def test_sumsq_buffer_can_be_set_and_restored_only_between_norm_and_gate():
    import torch
    from paper_2605_06755_b200 import binding as b
    data = _inputs()[:2]
    probs = [gu.Problem(*d) for d in data]
    cfg, opt = b.make_cfg(lr=1e-3)
    ctx = b.Context(cfg, opt, b.BF16)
    ctx.bind([p.ptrs() for p in probs])
    buf = torch.zeros(2, dtype=torch.float64, device="cuda")
    with pytest.raises(b.GxpoError) as e:
        ctx.set_sumsq_buffer(buf.data_ptr() + 4)             # not 8-byte aligned
    assert e.value.status == b.ERR_ALIGNMENT
    ctx.set_sumsq_buffer(buf.data_ptr())
    ctx.probe_step(0); ctx.probe_step(1); ctx.extrapolate(); ctx.slow_step()
    with pytest.raises(b.GxpoError) as e:
        ctx.set_sumsq_buffer(0)                              # a norm is pending in the caller's buffer
    assert e.value.status == b.ERR_STATE
    r1 = ctx.gate_update()
    want = math.sqrt(sum(ora.sum_squares(ora.bf16_bits_to_f64(d[5])) for d in data))
    assert r1.norm == pytest.approx(want, rel=gu.RTOL_NORM)
    assert math.sqrt(float(buf[0].item())) == r1.norm        # the gate read exactly what the buffer holds
    ctx.set_sumsq_buffer(0)                                  # back to the internal scalar
    buf.fill_(float("nan"))
    r2 = ctx.active_step()
    assert r2.norm == pytest.approx(want, rel=gu.RTOL_NORM) and math.isnan(float(buf[0].item()))
    ctx.close()
