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


# ---------------------------------------------------------------------------------------------
# One sequence over several GPUs: consecutive segments of T, the recurrent state handed on
# ---------------------------------------------------------------------------------------------
# The layer is a recurrence over tokens, so cutting a sequence along T gives a pipeline, not a parallel
# speed-up for one sequence: rank r runs its segment once rank r - 1 has sent the state S and the
# preconditioner d at the cut (`final_state`, `precond_out` of osdn_fwd are exactly that hand-off,
# `init_state`, `precond_in` take it up; backward the cotangents travel the other way through
# `dfinal_state` / `dprecond_out` and `dinit_state` / `dprecond_in`).  With several micro-batches
# (sequences) in flight the ranks overlap: rank r works on micro-batch m while rank r + 1 works on m - 1.
# What crosses the link per micro-batch and cut is [B, H, V, K] + [B, H, K] floats, point to point
# (NCCL send / recv over NVLink on GPUs; gloo in the CPU tests).

def segment_bounds(T: int, world: int, chunk: int = 64) -> List[Tuple[int, int]]:
    """Token range [lo, hi) of every rank: cuts on chunk boundaries, as even as those allow; ranks
    beyond the end of a short sequence get an empty range (they pass the state through)."""
    if T < 0 or world < 1:
        raise ValueError("bad arguments")
    per = -(-(-(-T // chunk)) // world) * chunk if T > 0 else 0   # ceil(ceil(T / chunk) / world) chunks
    out = []
    for r in range(world):
        lo = min(r * per, T)
        out.append((lo, min(lo + per, T)))
    return out


def forward_handoff(run_segment, state_in, precond_in, rank: int, world: int, group=None):
    """Forward of this rank's segment for one micro-batch.

    `run_segment(S, d) -> (result, S_out, d_out)` runs the layer on the rank's tokens from the state
    and preconditioner at the left cut and returns them at the right cut.  `state_in`, `precond_in`:
    tensors of the hand-off shapes; rank 0 uses their contents as the initial values, the other ranks
    receive into them.  Returns (result, S_out, d_out); the send to rank + 1 is complete on return.
    """
    if rank > 0:
        dist.recv(state_in, src=rank - 1, group=group)
        dist.recv(precond_in, src=rank - 1, group=group)
    result, s_out, d_out = run_segment(state_in, precond_in)
    if rank < world - 1:
        dist.send(s_out.contiguous(), dst=rank + 1, group=group)
        dist.send(d_out.contiguous(), dst=rank + 1, group=group)
    return result, s_out, d_out


def backward_handoff(run_segment_bwd, dstate_out, dprecond_out, rank: int, world: int, group=None):
    """Backward of this rank's segment: the mirror image of `forward_handoff`.

    `run_segment_bwd(dS, dd) -> (grads, dS_in, dd_in)` takes the cotangents of the state and the
    preconditioner at the right cut and returns those at the left cut.  The last rank uses the
    contents of `dstate_out`, `dprecond_out`; the others receive into them from rank + 1.
    """
    if rank < world - 1:
        dist.recv(dstate_out, src=rank + 1, group=group)
        dist.recv(dprecond_out, src=rank + 1, group=group)
    grads, ds_in, dd_in = run_segment_bwd(dstate_out, dprecond_out)
    if rank > 0:
        dist.send(ds_in.contiguous(), dst=rank - 1, group=group)
        dist.send(dd_in.contiguous(), dst=rank - 1, group=group)
    return grads, ds_in, dd_in
