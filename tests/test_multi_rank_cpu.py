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
