"""One sequence cut along T over three ranks, every segment computed by the library (osdn_fwd / osdn_bwd on
the GPU), the state and the preconditioner handed on through `final_state` -> `init_state` and the
cotangents back through `dinit_state` -> `dfinal_state`; the result is compared with the uncut fp64 oracle.

The ranks are three processes that take turns on one GPU: what is handed over travels through gloo on
the host (the hand-off protocol of `sharding.py`), and no kernel of one rank ever waits for a kernel of
another.  The device-to-device push over NVLink is not exercised here (one GPU per run).
"""
import copy
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

pytestmark = pytest.mark.gpu


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    import oracle
    import parity
    from paper_2605_13473_b200 import binding
    from paper_2605_13473_b200.sharding import backward_handoff, forward_handoff, segment_bounds
    from paper_2605_13473_b200.synth import OsdnHyper, draw
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        B, T, H, D = 2, 170, 2, 128
        hy = OsdnHyper(eta=0.3, apf_mode=1)
        inp = draw("handoff", 78, [T] * B, H, D, D, "bf16", dense_B=B, hyper=hy, with_dout=True, with_state=True,
                   with_state_cotangents=True)
        lo, hi = segment_bounds(T, world)[rank]

        def piece(b, S, d, dS=None, dd=None):
            """The rank's tokens of micro-batch b as an input bundle of its own."""
            sub = copy.copy(inp)
            sl = slice(b * T + lo, b * T + hi)
            for name in ("q", "k", "v", "beta", "gate", "dout"):
                setattr(sub, name, getattr(inp, name)[sl].contiguous())
            sub.seq_lens, sub.dense_B = [hi - lo], 1
            sub.init_state, sub.precond_in = S.float(), d.float()
            sub.dfinal_state, sub.dprecond_out = (None if dS is None else dS.float()), (None if dd is None else dd.float())
            return sub

        got = {k: [] for k in ("out", "dq", "dk", "dv", "dbeta", "dgate")}
        ends, saved = {}, []
        for b in range(B):   # micro-batches: one sequence each, the ranks form a pipeline
            S_in, d_in = inp.init_state[b:b + 1].clone(), inp.precond_in[b:b + 1].clone()

            def run(S, d):
                if hi == lo:
                    return None, S, d
                r = binding.run_inputs_fwd(piece(b, S, d))
                return r["out"], r["final_state"], r["precond_out"]
            res, S_out, d_out = forward_handoff(run, S_in, d_in, rank, world)
            saved.append((S_in.clone(), d_in.clone()))
            got["out"].append(res)
            ends[("S", b)], ends[("d", b)] = S_out, d_out
        for b in range(B):
            S_in, d_in = saved[b]
            dS, dd = inp.dfinal_state[b:b + 1].clone(), inp.dprecond_out[b:b + 1].clone()

            def run_bwd(dS_r, dd_r):
                if hi == lo:
                    return None, dS_r, dd_r
                g = binding.run_inputs_bwd(piece(b, S_in, d_in, dS_r, dd_r))
                return g, g["dinit_state"], g["dprecond_in"]
            g, dS_in, dd_in = backward_handoff(run_bwd, dS, dd, rank, world)
            for name in ("dq", "dk", "dv", "dbeta", "dgate"):
                got[name].append(None if g is None else g[name])
            ends[("dS", b)], ends[("dd", b)] = dS_in, dd_in
        # the uncut definition
        ref = oracle.fwd_inputs(inp)
        ref.update(oracle.bwd_inputs(inp))
        worst = {}
        for name, parts in got.items():
            for b, x in enumerate(parts):
                if x is not None:
                    e = parity.err(x.numpy(), ref[name][b * T + lo:b * T + hi], "bf16")
                    worst[name] = max(worst.get(name, 0.0), e)
        for b in range(B):
            if rank == world - 1:
                worst["final_state"] = max(worst.get("final_state", 0.0),
                                           parity.err(ends[("S", b)].numpy(), ref["final_state"][b:b + 1]))
                worst["precond_out"] = max(worst.get("precond_out", 0.0),
                                           parity.err(ends[("d", b)].numpy(), ref["precond_out"][b:b + 1]))
            if rank == 0:
                worst["dinit_state"] = max(worst.get("dinit_state", 0.0),
                                           parity.err(ends[("dS", b)].numpy(), ref["dinit_state"][b:b + 1]))
                worst["dprecond_in"] = max(worst.get("dprecond_in", 0.0),
                                           parity.err(ends[("dd", b)].numpy(), ref["dprecond_in"][b:b + 1]))
        out.put((rank, hi - lo, worst))
    finally:
        dist.destroy_process_group()


def test_sequence_cut_over_three_ranks_through_the_library():
    world = 3
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(q.get(timeout=300) for _ in range(world))
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert [r[1] for r in results] == [64, 64, 42]
    for rank, n, worst in results:
        bad = {k: v for k, v in worst.items() if not (v <= 2e-2)}
        assert not bad, (rank, worst)
    # every boundary quantity was checked by the rank that owns it
    assert "final_state" in results[2][2] and "dinit_state" in results[0][2]
