"""The N > 1 path on CPU: two gloo ranks shard a var-len batch by sequences, each checks its shard
against the whole-batch oracle result (chains are independent, so no data-path collective exists),
and the job throughput is reduced as sum(units) / max(time)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
import parity
from paper_2605_13473_b200.sharding import aggregate_throughput, shard_sequences
from paper_2605_13473_b200.synth import OsdnHyper, draw


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        inp = draw("multi", 31, [40, 7, 90, 13, 64], 2, 8, 8, "fp32", hyper=OsdnHyper(eta=0.3, apf_mode=1))
        mine, tokens = shard_sequences(inp.seq_lens, rank, world)
        sub, tok_t, hd = parity.subset(inp, mine, [0, 1])
        res = oracle.fwd_inputs(sub)                     # this rank's shard, alone
        full = oracle.fwd_inputs(inp)                    # the whole batch
        ref = parity.subset_result(full, mine, [0, 1], tok_t, hd)
        ok = all(np.array_equal(res[k], ref[k]) for k in ("out", "final_state", "precond_out"))
        # every sequence belongs to exactly one rank
        owned = torch.zeros(len(inp.seq_lens), dtype=torch.int64)
        owned[mine] = 1
        dist.all_reduce(owned)
        units, ms, value = aggregate_throughput(tokens, 10.0 * (rank + 1))
        out.put((rank, ok, owned.tolist(), tokens, units, ms, value))
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_by_sequence_and_reduce_timing():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    total = 40 + 7 + 90 + 13 + 64
    for rank, ok, owned, tokens, units, ms, value in results:
        assert ok
        assert owned == [1] * 5
        assert units == total and ms == 20.0 and abs(value - total / 0.02) < 1e-6
    assert sum(r[3] for r in results) == total
    assert abs(results[0][3] - results[1][3]) <= 40       # balanced by tokens


def test_shard_sequences_properties():
    lens = [5586, 16100, 976, 32768, 32768, 7605, 4227, 31042]
    for world in (1, 2, 4, 8):
        seen = []
        loads = []
        for r in range(world):
            mine, tokens = shard_sequences(lens, r, world)
            seen += mine
            loads.append(tokens)
            assert tokens == sum(lens[i] for i in mine)
        assert sorted(seen) == list(range(len(lens)))
        assert max(loads) <= max(max(lens), -(-sum(lens) // world) + max(lens))


# ---------------------------------------------------------------------------------------------
# one sequence cut along T over the ranks: the state and the preconditioner are handed on
# ---------------------------------------------------------------------------------------------
def _seq_worker(rank, world, port, out):
    from paper_2605_13473_b200.sharding import backward_handoff, forward_handoff, segment_bounds
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        B, T, H, K, V = 2, 150, 2, 8, 8
        hy = OsdnHyper(eta=0.3, apf_mode=2)
        inp = draw("seqshard", 77, [T] * B, H, K, V, "fp32", dense_B=B, hyper=hy, with_dout=True,
                   with_log_ret=True, with_state=True, with_state_cotangents=True)
        f64 = lambda t: None if t is None else t.double().numpy()
        x = {n: f64(getattr(inp, n)) for n in ("q", "k", "v", "beta", "gate", "log_ret", "dout", "init_state",
                                               "precond_in", "dfinal_state", "dprecond_out")}
        lo, hi = segment_bounds(T, world)[rank]
        ok = True
        worst = 0.0
        full_f = oracle.fwd(hy, [T] * B, x["q"], x["k"], x["v"], x["beta"], x["gate"], x["log_ret"],
                            x["init_state"], x["precond_in"])
        full_b = oracle.bwd(hy, [T] * B, x["q"], x["k"], x["v"], x["beta"], x["gate"], x["dout"], x["log_ret"],
                            x["init_state"], x["precond_in"], x["dfinal_state"], x["dprecond_out"])
        saved = []
        for b in range(B):   # micro-batches: one sequence each, the ranks form a pipeline
            sl = slice(b * T + lo, b * T + hi)
            S_in = torch.from_numpy(x["init_state"][b:b + 1].copy())
            d_in = torch.from_numpy(x["precond_in"][b:b + 1].copy())

            def run(S, d):
                if hi == lo:
                    return None, S, d
                r = oracle.fwd(hy, [hi - lo], x["q"][sl], x["k"][sl], x["v"][sl], x["beta"][sl], x["gate"][sl],
                               x["log_ret"][sl], S.numpy(), d.numpy())
                return r["out"], torch.from_numpy(r["final_state"]), torch.from_numpy(r["precond_out"])
            res, S_out, d_out = forward_handoff(run, S_in, d_in, rank, world)
            saved.append((S_in.clone(), d_in.clone()))
            if res is not None:
                worst = max(worst, float(np.abs(res - full_f["out"][sl]).max()))
            if rank == world - 1:
                worst = max(worst, float(np.abs(S_out.numpy() - full_f["final_state"][b:b + 1]).max()),
                            float(np.abs(d_out.numpy() - full_f["precond_out"][b:b + 1]).max()))
        for b in range(B):
            sl = slice(b * T + lo, b * T + hi)
            S_in, d_in = saved[b]
            dS = torch.from_numpy(x["dfinal_state"][b:b + 1].copy())
            dd = torch.from_numpy(x["dprecond_out"][b:b + 1].copy())

            def run_bwd(dS_r, dd_r):
                if hi == lo:
                    return None, dS_r, dd_r
                g = oracle.bwd(hy, [hi - lo], x["q"][sl], x["k"][sl], x["v"][sl], x["beta"][sl], x["gate"][sl],
                               x["dout"][sl], x["log_ret"][sl], S_in.numpy(), d_in.numpy(), dS_r.numpy(), dd_r.numpy())
                return g, torch.from_numpy(g["dinit_state"]), torch.from_numpy(g["dprecond_in"])
            g, dS_in, dd_in = backward_handoff(run_bwd, dS, dd, rank, world)
            if g is not None:
                for name in ("dq", "dk", "dv", "dbeta", "dgate", "dlog_ret"):
                    worst = max(worst, float(np.abs(g[name] - full_b[name][sl]).max()))
            if rank == 0:
                worst = max(worst, float(np.abs(dS_in.numpy() - full_b["dinit_state"][b:b + 1]).max()),
                            float(np.abs(dd_in.numpy() - full_b["dprecond_in"][b:b + 1]).max()))
        out.put((rank, ok, worst, hi - lo))
    finally:
        dist.destroy_process_group()


def test_sequence_cut_over_ranks_hands_state_and_cotangents_on():
    from paper_2605_13473_b200.sharding import segment_bounds
    assert segment_bounds(150, 3) == [(0, 64), (64, 128), (128, 150)]
    assert segment_bounds(65, 3) == [(0, 64), (64, 65), (65, 65)]
    assert segment_bounds(4096, 4)[2] == (2048, 3072)
    world = 3
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_seq_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(q.get(timeout=180) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[3] for r in results] == [64, 64, 22]
    for rank, ok, worst, n in results:
        assert ok and worst <= 1e-9, (rank, worst)
