"""The multi-GPU path on CPU: two `gloo` ranks each own a shard of a tensor list,
run Algorithm 1 on it (the CPU oracle stands in for the kernels), exchange only
sum(g_slow^2), and must (a) flip their gates at the same step as an unsharded run
and (b) hold exactly the unsharded parameters restricted to their shard."""
import os
import socket
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from oracle import gxpo_oracle as ora  # noqa: E402
from paper_2605_06755_b200 import sharding, workloads  # noqa: E402

SIZES = [4096, 70001, 512, 33000, 17]
STEPS, JUMP_AT = 12, 8


def _inputs():
    out = []
    for i, n in enumerate(SIZES):
        rng = np.random.default_rng(400 + i)
        th = (0.02 * rng.standard_normal(n)).astype(np.float32)
        g0 = (1e-3 * rng.standard_normal(n)).astype(np.float32)
        g1 = (g0 * rng.uniform(0.2, 1.2, n)).astype(np.float32)
        gs = (g0 * rng.uniform(0.5, 1.0, n)).astype(np.float32)
        out.append((th, workloads.f32_to_bf16_bits(g0), workloads.f32_to_bf16_bits(g1),
                    workloads.f32_to_bf16_bits(gs)))
    return out


def _run(pieces, reduce_fn):
    """Algorithm 1 for STEPS steps on the given pieces; `reduce_fn` turns the local
    sum of squares into the global one.  Returns (s_star, phases, thetas)."""
    data = _inputs()
    cfg = ora.GxpoCfg(K=5, alpha=0.5, delta=1e-8, tau=0.5, window=20)
    opt = ora.OptCfg(kind="adamw", lr=1e-3)
    gate = ora.Gate(cfg)
    states, grads = [], []
    for p in pieces:
        th, g0, g1, gs = (x[p.offset:p.offset + p.length] for x in data[p.tensor])
        states.append(ora.State(th, opt))
        grads.append([ora.bf16_bits_to_f64(g) for g in (g0, g1, gs)])
    phases = []
    for t in range(STEPS):
        mult = 8.0 if t == JUMP_AT else 1.0
        if gate.active:
            local = 0.0
            for st, g in zip(states, grads):
                gg = [g[0], g[1], g[2] * mult]
                ora.active_step(st, cfg, lambda w, th, gg=gg: gg[w], round_f32=True)
                local += ora.sum_squares(gg[2])
            gate.update(float(np.sqrt(reduce_fn(local))))
            phases.append("a")
        else:
            for st, g in zip(states, grads):
                ora.fallback_step(st, lambda w, th, g=g: g[w], round_f32=True)
            gate.fallback_tick()
            phases.append("f")
    return gate.s_star, "".join(phases), [st.theta.copy() for st in states]


def _worker(rank, world, port, mode, outdir):
    import torch
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    parts = (sharding.partition_by_tensor if mode == "tensor" else sharding.partition_by_slice)(SIZES, world)

    def reduce_fn(local):
        t = torch.tensor([local], dtype=torch.float64)
        sharding.allreduce_sumsq(t)
        return float(t.item())

    s_star, phases, thetas = _run(parts[rank], reduce_fn)
    np.savez(os.path.join(outdir, f"rank{rank}.npz"), s_star=s_star, phases=phases,
             **{f"theta{i}": th for i, th in enumerate(thetas)})
    dist.barrier()
    dist.destroy_process_group()


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.mark.parametrize("mode", ["tensor", "slice"])
def test_two_ranks_flip_together_and_match_the_unsharded_run(mode, tmp_path):
    import torch.multiprocessing as mp
    world = 2
    whole = [sharding.Piece(i, 0, n) for i, n in enumerate(SIZES)]
    s_ref, phases_ref, thetas_ref = _run(whole, lambda x: x)
    assert s_ref == JUMP_AT + 1 and phases_ref == "a" * (JUMP_AT + 1) + "f" * (STEPS - JUMP_AT - 1)
    mp.spawn(_worker, args=(world, _free_port(), mode, str(tmp_path)), nprocs=world, join=True)
    parts = (sharding.partition_by_tensor if mode == "tensor" else sharding.partition_by_slice)(SIZES, world)
    sharding.check_partition(SIZES, parts)
    for rank in range(world):
        got = np.load(os.path.join(tmp_path, f"rank{rank}.npz"))
        assert int(got["s_star"]) == s_ref and str(got["phases"]) == phases_ref
        assert len(parts[rank]) > 0
        for i, p in enumerate(parts[rank]):
            np.testing.assert_array_equal(got[f"theta{i}"],
                                          thetas_ref[p.tensor][p.offset:p.offset + p.length])


def test_partitions_tile_every_tensor_once_and_balance():
    qwen = [n for _, n in workloads.qwen25_7b_shapes()]
    for world in (1, 2, 3, 4, 8):
        for fn in (sharding.partition_by_tensor, sharding.partition_by_slice):
            parts = fn(qwen, world)
            assert len(parts) == world
            sharding.check_partition(qwen, parts)
            loads = [sum(p.length for p in pieces) for pieces in parts]
            assert sum(loads) == sum(qwen)
            if fn is sharding.partition_by_slice:
                assert max(loads) - min(loads) <= 2 * sharding.ALIGN_ELEMS
                for pieces in parts:
                    assert all(p.offset % sharding.ALIGN_ELEMS == 0 for p in pieces)
            else:
                assert max(loads) <= 1.25 * sum(qwen) / world + max(qwen)
    with pytest.raises(ValueError):
        sharding.check_partition([10], [[sharding.Piece(0, 0, 6)], [sharding.Piece(0, 5, 5)]])
    with pytest.raises(ValueError):
        sharding.partition_by_slice([4, -1], 2)
    assert sharding.partition_by_slice([], 2) == [[], []]
