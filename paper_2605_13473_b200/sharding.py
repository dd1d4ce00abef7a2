"""Host-side helpers for running the layer on several GPUs.

Every (sequence, head) chain of the layer is independent of every other one, so a batch is
sharded by sequences (or a benchmark gives every rank a batch of its own) and no collective is
needed on the data path.  The only cross-rank communication is the reduction of timings.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist


def shard_sequences(seq_lens: Sequence[int], rank: int, world: int) -> Tuple[List[int], int]:
    """Greedy longest-first assignment of sequences to ranks, balanced by token count.

    Returns (indices of the sequences of `rank`, tokens of `rank`).  Deterministic; every sequence
    is assigned to exactly one rank.
    """
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    order = sorted(range(len(seq_lens)), key=lambda i: (-int(seq_lens[i]), i))
    load = [0] * world
    mine: List[int] = []
    for i in order:
        r = min(range(world), key=lambda j: (load[j], j))
        load[r] += int(seq_lens[i])
        if r == rank:
            mine.append(i)
    return sorted(mine), load[rank]


def aggregate_throughput(local_units: float, local_ms: float, device=None) -> Tuple[float, float, float]:
    """(total units over all ranks, max time in ms over ranks, units per second of the whole job)."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        t = torch.tensor([float(local_units), 0.0], dtype=torch.float64, device=device)
        m = torch.tensor([float(local_ms)], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        dist.all_reduce(m, op=dist.ReduceOp.MAX)
        units, ms = float(t[0]), float(m[0])
    else:
        units, ms = float(local_units), float(local_ms)
    return units, ms, units / (ms * 1e-3) if ms > 0 else float("inf")
