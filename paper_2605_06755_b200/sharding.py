"""Host-side helpers for running the update sharded over several GPUs, one process
per GPU.

Every step of the update is per-coordinate, so any partition of the parameters
works; the one quantity that crosses shards is sum(g_slow^2), which feeds the gate
(Eq. (z_score)).  This module only cuts a tensor list into per-rank pieces and
wraps the 8-byte exchange; it holds none of the method's arithmetic.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Sequence, Tuple

# Slice boundaries are multiples of this many elements so that a slice of a
# 32-byte-aligned bfloat16 or float32 array is still 32-byte aligned (vector path).
ALIGN_ELEMS = 16


@dataclass(frozen=True)
class Piece:
    """`length` elements of tensor `tensor`, starting at element `offset`."""
    tensor: int
    offset: int
    length: int


def partition_by_tensor(sizes: Sequence[int], world: int) -> List[List[Piece]]:
    """Whole tensors to ranks, largest first onto the least loaded rank (ties go to
    the lowest rank).  Deterministic; every tensor appears exactly once."""
    if world < 1:
        raise ValueError("world must be >= 1")
    load = [0] * world
    out: List[List[Piece]] = [[] for _ in range(world)]
    order = sorted(range(len(sizes)), key=lambda i: (-sizes[i], i))
    for i in order:
        if sizes[i] < 0:
            raise ValueError("negative tensor size")
        r = min(range(world), key=lambda k: (load[k], k))
        out[r].append(Piece(i, 0, sizes[i]))
        load[r] += sizes[i]
    for pieces in out:
        pieces.sort(key=lambda p: p.tensor)
    return out


def partition_by_slice(sizes: Sequence[int], world: int) -> List[List[Piece]]:
    """Contiguous slices of the concatenated parameter space, equal up to alignment:
    rank k owns global elements [cut[k], cut[k+1]).  Cuts inside a tensor fall on
    multiples of ALIGN_ELEMS relative to that tensor's start."""
    if world < 1:
        raise ValueError("world must be >= 1")
    if any(n < 0 for n in sizes):
        raise ValueError("negative tensor size")
    total = sum(sizes)
    starts, acc = [], 0
    for n in sizes:
        starts.append(acc)
        acc += n
    cuts = [0]
    for k in range(1, world):
        c = total * k // world
        # move the cut to an aligned position inside the tensor that holds it
        t = _tensor_at(starts, sizes, c)
        if t is not None:
            inside = c - starts[t]
            c = starts[t] + inside // ALIGN_ELEMS * ALIGN_ELEMS
        cuts.append(max(c, cuts[-1]))
    cuts.append(total)
    out: List[List[Piece]] = []
    for k in range(world):
        lo, hi = cuts[k], cuts[k + 1]
        pieces = []
        for t, (s, n) in enumerate(zip(starts, sizes)):
            a, b = max(lo, s), min(hi, s + n)
            if b > a:
                pieces.append(Piece(t, a - s, b - a))
        out.append(pieces)
    return out


def _tensor_at(starts, sizes, g):
    for t, (s, n) in enumerate(zip(starts, sizes)):
        if s <= g < s + n:
            return t
    return None


def check_partition(sizes: Sequence[int], parts: Sequence[Sequence[Piece]]) -> None:
    """Raise unless the pieces tile every tensor exactly once."""
    seen: List[List[Tuple[int, int]]] = [[] for _ in sizes]
    for pieces in parts:
        for p in pieces:
            if p.length <= 0 or p.offset < 0 or p.offset + p.length > sizes[p.tensor]:
                raise ValueError(f"piece out of range: {p}")
            seen[p.tensor].append((p.offset, p.offset + p.length))
    for t, spans in enumerate(seen):
        spans.sort()
        pos = 0
        for a, b in spans:
            if a != pos:
                raise ValueError(f"tensor {t}: gap or overlap at element {pos}")
            pos = b
        if pos != sizes[t]:
            raise ValueError(f"tensor {t}: covered {pos} of {sizes[t]} elements")


def allreduce_sumsq(sumsq, group=None):
    """Sum the per-shard sum(g_slow^2) over all ranks, in place.  `sumsq` is a
    one-element float64 tensor: on the device with NCCL (enqueued on the current
    stream, between gxpo_slow_step and gxpo_gate_update), on the host with gloo."""
    import torch.distributed as dist
    dist.all_reduce(sumsq, op=dist.ReduceOp.SUM, group=group)
    return sumsq
