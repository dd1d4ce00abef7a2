#!/usr/bin/env python
"""Benchmark of the OSDN layer hot path: forward + backward tokens/s per layer on B200.

    python bench.py --gpus 1 --steps 20 --warmup 5
    python -m torch.distributed.run --nnodes=1 --nproc-per-node N ... bench.py --gpus N ...
    python bench.py --impl reference            # the fp64 CPU oracle, timed on the host cores

One step = one pass of the whole hot path (osdn_fwd with saved residuals + osdn_bwd) over one
synthetic batch of the 340M-model layer shape (B=8, T=2048, H=8, dk=dv=128, bf16).  Inputs are
resident in HBM for `value`; `e2e` goes through osdn_step_host with pinned host buffers.  With N
GPUs every rank runs its own batch (weak scaling, no data-path collective: chains are independent).
Rank 0 prints one JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

WORKLOADS = {
    "cfg1": dict(idx=1, bwd=False, desc="cfg1 340M layer forward: B=8 T=2048 H=8 dk=dv=128 bf16"),
    "cfg2": dict(idx=2, bwd=True, desc="cfg2 340M layer train step (fwd+bwd): B=8 T=2048 H=8 dk=dv=128 bf16"),
    "cfg3": dict(idx=3, bwd=True, desc="cfg3 1.3B layer fwd+bwd: B=4 T=4096 H=16 dk=dv=128 bf16, mixture gates"),
    "cfg4": dict(idx=4, bwd=True, desc="cfg4 varlen fwd+bwd: 8 packed sequences, 131072 tokens, H=8 dk=dv=128 bf16"),
    "osdn_1p3b": dict(idx=-3, bwd=True, desc="ungated 1.3B OSDN setting (g = 0, separate retention near 0.999, "
                                             "non-beta-aware step): B=4 T=4096 H=16 dk=dv=128 bf16"),
    "cfg2_lively": dict(idx=-2, bwd=True, desc="cfg2 shape with a moving preconditioner (eta=0.3, sparse keys, "
                                               "separate retention): B=8 T=2048 H=8 dk=dv=128 bf16"),
    "oskda": dict(idx=-4, bwd=True, desc="OSKDA extension (one gate per key channel, constant retention 0.999) at the "
                                         "cfg2 shape: B=8 T=2048 H=8 dk=dv=128 bf16, osdn_kda_fwd + osdn_kda_bwd"),
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def make_inputs(name):
    from paper_2605_13473_b200.synth import OsdnHyper, config, draw
    if name == "decode":
        return draw("decode_b512", 21, [1] * 512, 8, 128, 128, "bf16", dense_B=512, hyper=OsdnHyper(), with_state=True)
    w = WORKLOADS[name]
    if w["idx"] >= 0:
        return config(w["idx"])
    if w["idx"] == -3:
        hy = OsdnHyper(eta=0.003, apf_mode=2, beta_aware=0)
        return draw("osdn_1p3b", 13, [4096] * 4, 16, 128, 128, "bf16", dense_B=4, hyper=hy, gate_kind="zero",
                    with_dout=True, with_log_ret=True, log_ret_shift=7.0)
    if w["idx"] == -4:
        import math
        import torch
        hy = OsdnHyper(eta=0.003, apf_mode=2, channel_gate=1)
        inp = draw("oskda", 5, [2048] * 8, 8, 128, 128, "bf16", dense_B=8, hyper=hy, with_dout=True, with_log_ret=True)
        inp.log_ret = torch.full_like(inp.log_ret, math.log(0.999))   # the paper's setting for this extension
        return inp
    hy = OsdnHyper(eta=0.3, apf_mode=2)
    return draw("cfg2_lively", 12, [2048] * 8, 8, 128, 128, "bf16", dense_B=8, hyper=hy, key_kind="sparse",
                with_dout=True, with_log_ret=True)


# ---------------------------------------------------------------------------------------------
# Work of each kernel per launch, as a function of the workload.
#   method_bytes : the bytes of the METHOD that the kernel is the one to move -- user tensors it reads
#                  or writes and the per-chunk state the backward is entitled to (one bf16 state
#                  image per 64 tokens) -- independent of how this design splits the work.  The
#                  roofline fraction is computed from these.
#   kernel_model : the bytes this design makes the kernel read + write (its tiles included) and its
#                  tensor flops; reported beside the fraction as `design_bytes`, never as its numerator.
# ---------------------------------------------------------------------------------------------
def method_bytes(name, inp, with_bwd):
    """Method bytes per launch of one kernel (see above); None for kernels outside the table."""
    K, V = inp.K, inp.V
    es = 2 if inp.io_dtype == "bf16" else 4
    tokh = inp.T_total * inp.H
    state = V * K * 2 / 64.0          # one bf16 state image per 64-token chunk, per token-head
    per = {
        "phase1_spec": K * es + 8,                                   # k, beta, gate
        "phase1_seq": 0.0, "phase1_bwd_seq": 0.0, "build_table": 0.0,
        "tc_chunk_fwd": 2 * K * es + 8,                              # q, k, beta, gate
        "tc_chain_fwd": V * es + V * es + (state if with_bwd else 0),  # v in, out, saved state
        "tc_fwd": 2 * K * es + 8 + V * es + V * es + (state if with_bwd else 0),   # both passes in one launch
        # q, k, v, dout, beta, gate, the saved state in; dq, dk, dv, dbeta, dgate out
        "tc_bwd": (2 * K + 2 * V) * es + 8 + state + (2 * K + V) * es + 8,
        # channel-gate extension: q, k, v, beta, K gates in, out; the backward reads them again with dout and
        # writes dq, dk, dv, dbeta and K gate gradients
        "kda_fwd": (2 * K + 2 * V) * es + 4 + 4 * K,
        "kda_bwd": (2 * K + 2 * V) * es + 4 + 4 * K + (2 * K + V) * es + 4 + 4 * K,
    }
    return None if name not in per else per[name] * tokh


def kernel_model(name, inp, NT):
    """returns (design bytes, flops, bound) for one launch; NT = number of 64-token chunks (all heads excluded)."""
    H, K, V = inp.H, inp.K, inp.V
    T = inp.T_total
    es = 2 if inp.io_dtype == "bf16" else 4
    tiles = NT * H               # (chunk, head) tiles
    tokh = T * H                 # token-heads
    C = 64
    f = lambda m, n, k: 2.0 * m * n * k
    m = {}
    # CUDA-core (fp32 workspace) family
    m["phase1_fwd"] = (tokh * (K * es + 8 + K * 4) + tiles * K * 4, tokh * 9.0 * K, "hbm")
    m["simt_chunk_local_fwd"] = (tokh * (2 * K * es + K * 4 + V * es + 8) + tiles * 4 * (2 * C * C + C * K + C * V),
                                 tiles * (2 * f(C, C, K) + f(C, K, C) + f(C, V, C)), "alu")
    m["simt_chain_fwd"] = (tokh * (K * es + K * 4 + V * es + 8) + tiles * 4 * (C * K + 2 * C * V + C * C + V * K),
                           tiles * (2 * f(C, V, K) + f(C, V, C) + f(V, K, C)), "alu")
    m["simt_chain_bwd"] = (tokh * (K * es + K * 4 + V * es + 8) + tiles * 4 * (C * K + C * V + C * C + V * K),
                           tiles * (f(C, V, C) + f(C, V, K) + 2 * f(V, K, C)), "alu")
    m["simt_chunk_local_bwd"] = (tokh * (3 * K * es + K * 4 + 3 * V * es + 2 * K * 4 + 16)
                                 + tiles * 4 * (2 * C * C + 2 * C * V + 2 * V * K + 10 * C * K),
                                 tiles * (f(C, C, V) + 5 * f(C, K, V) + f(C, C, K) * 2 + f(C, C, V)
                                          + f(C, K, C) * 5 + f(C, V, C) + 2 * f(C, C, C)), "alu")
    m["build_table"] = (NT * 12, 0.0, "hbm")
    # phase 1 (both families)
    m["phase1_spec"] = (tokh * (2 * K * es + 16), tokh * 12.0 * K, "hbm")
    m["phase1_seq"] = (tiles * (16 + K * 4), 0.0, "hbm")          # pinned regime: flag words + chunk-start d
    m["phase1_bwd_seq"] = (tiles * 8, 0.0, "hbm")
    m["phase1_bwd_bulk"] = (tokh * (2 * K * 4 + K * es), tokh * 2.0 * K, "hbm")
    # tensor-core family: bytes of the tiles each kernel reads and writes in this design (bf16 images)
    raw = C * K * es                                               # one [64 x 128] user tile
    m["tc_chunk_fwd"] = (tiles * (3 * raw + 16384 + 8192 + 8192 + 8192 + 16384) + tokh * 8,
                         tiles * (f(128, 64, K) + f(128, 64, C)), "hbm")
    m["tc_chain_fwd"] = (tiles * (16384 + 8192 + 8192 + 3 * raw + raw + 32768 + 16384) + tokh * 4,
                         tiles * (f(128, 64, C) + 2 * f(128, 64, K) + f(128, 64, C) + f(128, 128, C)), "hbm")
    m["tc_fwd"] = (m["tc_chunk_fwd"][0] + m["tc_chain_fwd"][0], m["tc_chunk_fwd"][1] + m["tc_chain_fwd"][1], "hbm")
    # one launch: the reverse state chains (dout, ktil, W^T, P', Qg in; dS_n, ddU^T out) and the chunk-local
    # part (q, k, ktil, v, dout, dU^T, ddU^T, T, S_n, dS_n in; dq, dk, dv out)
    m["tc_bwd"] = (tiles * (2 * raw + 8192 + 16384 + 16384 + 32768 + 16384) + tokh * 4
                   + tiles * (5 * raw + 16384 + 16384 + 8192 + 32768 + 32768 + 3 * raw) + tokh * 24,
                   tiles * (f(128, 64, C) + f(128, 64, K) + 2 * f(128, 128, C))
                   + tiles * (2 * f(64, 64, K) + 3 * f(128, 64, K) + 2 * f(64, 64, K) + 2 * f(128, 64, C)
                              + 2 * f(64, 64, C) + 4 * f(128, 64, C)), "hbm")
    # channel-gate extension, token-recurrent on CUDA cores: per token and state row K decays, K + K + K fused
    # multiply-adds forward (read, write, output); the backward replays the forward's two and takes about
    # seven more per element for the adjoint
    m["kda_fwd"] = (tokh * ((2 * K + 2 * V) * es + 4 + 8 * K) + tiles * 4 * V * K, tokh * V * K * 8.0, "alu")
    m["kda_bwd"] = (tokh * ((4 * K + 3 * V) * es + 8 + 24 * K) + tiles * 4 * V * K, tokh * V * K * 20.0, "alu")
    return m.get(name)


def load_traffic(workload, kernel, measured_us=None, summary=None):
    """DRAM bytes (read + write) of one launch of `kernel` from the committed ncu summary of this
    workload (lines "- traffic_bytes <kernel> = <bytes>" and "- profile_us <kernel> = <duration>").
    The capture belongs to the build it was taken on: when the kernel's duration in the capture and the
    one measured now differ by more than 15 % the figure is stale and dropped.  Returns
    (bytes or None, a note naming the source)."""
    rel = os.path.join("profiles", summary or f"osdn_step_{workload}.md")
    nbytes, prof_us = None, None
    try:
        for line in open(os.path.join(ROOT, rel)):
            parts = line.split()
            if len(parts) >= 5 and parts[0] == "-" and parts[2] == kernel:
                if parts[1] == "traffic_bytes":
                    nbytes = float(parts[4])
                elif parts[1] == "profile_us":
                    prof_us = float(parts[4])
    except OSError:
        return None, "no ncu capture committed for this workload"
    if nbytes is None:
        return None, f"{rel} has no capture of this kernel"
    if prof_us is not None and measured_us:
        if abs(prof_us - measured_us) > 0.15 * measured_us:
            return None, (f"{rel} is stale: the captured launch took {prof_us:.1f} us, this build "
                          f"{measured_us:.1f} us")
        return nbytes, f"{rel} (ncu capture, {prof_us:.1f} us per launch there)"
    return nbytes, f"{rel} (ncu capture)"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.rows = []
        self.proc = None
        self.gpu = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        for r in self.rows:
            c = [x.strip() for x in r.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1])); mx.append(float(c[2])); power.append(float(c[3]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), c[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    power_w_max=max(power) if power else None, samples=len(sm), reasons=sorted(reasons))


def run_reference(args):
    """The oracle as it stands, timed on the host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import oracle
    inp = make_inputs(args.workload)
    w = WORKLOADS.get(args.workload) or dict(bwd=False, desc="decode: 512 sequences x 1 new token, H=8 dk=dv=128, "
                                                               "bf16 activations, fp32 state")
    tokens = inp.T_total

    def step():
        oracle.fwd_inputs(inp)
        if w["bwd"]:
            oracle.bwd_inputs(inp)

    oracle.build()
    for _ in range(args.warmup if args.warmup is not None else 1):
        step()
    steps = args.steps if args.steps is not None else 5
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    dt = time.perf_counter() - t0
    val = tokens * steps / dt
    cores = oracle.threads()
    line = {
        "impl": "reference",
        "metric": ("decode tokens/s per layer" if args.workload == "decode" else
                   "fwd+bwd tokens/s per layer" if w["bwd"] else "fwd tokens/s per layer"), "value": val, "unit": "tokens/s",
        "n_gpus": 0, "steps": steps, "warmup": args.warmup if args.warmup is not None else 1,
        "ms_per_step": 1e3 * dt / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": w["desc"], "note": "fp64 token-by-token CPU oracle, OpenMP over chains"},
        "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                         "sample": f"whole workload ({tokens} tokens x {inp.H} heads) per step"},
        "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def run_decode(args):
    """`--workload decode`: the recurrent step (osdn_decode_step) on a serving-sized cache: one new token
    for each of 512 sequences, H=8, dk=dv=128, bf16 activations, fp32 state (268 MB, larger than L2).
    Bound by reading and writing the state once per token."""
    import torch
    import torch.distributed as dist
    from paper_2605_13473_b200 import binding
    from paper_2605_13473_b200.build import build
    from paper_2605_13473_b200.sharding import aggregate_throughput
    from paper_2605_13473_b200.synth import OsdnHyper, draw

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        build()
    if world > 1:
        dist.barrier()
    steps = args.steps if args.steps is not None else 50
    warmup = max(args.warmup if args.warmup is not None else 5, 3)
    B, H, D = 512, 8, 128
    hy = OsdnHyper()
    inp = draw("decode_b512", 21 + rank, [1] * B, H, D, D, "bf16", dense_B=B, hyper=hy, with_state=True)
    p = binding.make_params(B=B, T=1, H=H, K=D, V=D, io_dtype="bf16", hyper=hy)
    hq, hk, hv = (x.to(torch.bfloat16).contiguous().pin_memory() for x in (inp.q, inp.k, inp.v))
    hb, hg = inp.beta.float().pin_memory(), inp.gate.float().pin_memory()
    q, k, v, beta, gate = (x.to(dev) for x in (hq, hk, hv, hb, hg))
    state, precond = inp.init_state.float().to(dev).contiguous(), inp.precond_in.float().to(dev).contiguous()
    out = torch.empty(B, H, D, device=dev, dtype=torch.bfloat16)
    hout = torch.empty(B, H, D, dtype=torch.bfloat16).pin_memory()

    def step():
        binding.osdn_decode_step(p, q, k, v, beta, gate, None, state, precond, out)

    def host_step():
        for dst, src in ((q, hq), (k, hk), (v, hv), (beta, hb), (gate, hg)):
            dst.copy_(src, non_blocking=True)
        step()
        hout.copy_(out, non_blocking=True)

    def sync_all():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn):
        sync_all()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        sync_all()
        return e0.elapsed_time(e1)

    for _ in range(warmup):
        step()
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    ms_total = timed(step)
    binding.stage_timing_enable(True)
    timed(step)
    stages = binding.stage_timing_collect()
    binding.stage_timing_enable(False)
    clocks = sampler.stop()
    for _ in range(2):
        host_step()
    ms_host = timed(host_step)
    total_tokens, ms_total, _ = aggregate_throughput(B * steps, ms_total, dev)
    _, ms_host, _ = aggregate_throughput(B * steps, ms_host, dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    peaks = load_peaks()
    durs = stages.get("decode_step", [])
    avg_s = (sum(durs) / len(durs) * 1e-3) if durs else ms_total / steps * 1e-3
    nbytes = B * H * (2 * D * D * 4 + 2 * D * 4 + (2 * D + 2 * D) * 2 + 8)   # state and d in+out, q k v out, beta gate
    ach = nbytes / avg_s / 1e9
    roofline = dict(kernel="decode_step", bound="hbm", achieved=ach, peak=peaks["hbm_gbs"], unit="GB/s",
                    frac=ach / peaks["hbm_gbs"], traffic=load_traffic("decode", "decode_step", avg_s * 1e6, "osdn_decode_b512.md")[0],
                    peak_source=peaks["source"], avg_us=avg_s * 1e6, algorithmic_bytes=nbytes)
    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        sys.path.insert(0, os.path.join(ROOT, "tests"))
        import oracle
        oracle.build()
        t0, reps = time.perf_counter(), 0
        while time.perf_counter() - t0 < 10.0 and reps < 200:
            oracle.fwd_inputs(inp)
            reps += 1
        dt = time.perf_counter() - t0
        cpu_baseline = dict(value=B * reps / dt, unit="tokens/s", cores=oracle.threads(), kind="oracle",
                            sample=f"whole workload ({B} sequences x {H} heads, one token each), {reps} repetitions, {dt:.1f} s")
    nb = lambda *ts: int(sum(t.numel() * t.element_size() for t in ts))
    line = {
        "metric": "decode tokens/s per layer", "value": total_tokens / (ms_total * 1e-3), "unit": "tokens/s",
        "n_gpus": world, "steps": steps, "warmup": warmup, "ms_per_step": ms_total / steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": "decode: 512 sequences x 1 new token, H=8 dk=dv=128, bf16 activations, fp32 state",
                   "l2": "state (268 MB) exceeds L2 (no flush)", "tokens_per_step_per_gpu": B,
                   "kernel_timing": "second pass of the same steps with an event between launches"},
        "clocks": clocks, "gpu_launches": steps,
        "e2e": {"value": total_tokens / (ms_host * 1e-3), "unit": "tokens/s",
                "h2d_bytes_per_step": nb(hq, hk, hv, hb, hg), "d2h_bytes_per_step": nb(hout),
                "note": "activations from and to pinned host memory every step; the state stays in its device cache"},
        "roofline": roofline, "cpu_baseline": cpu_baseline,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=list(WORKLOADS) + ["decode"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--simt", action="store_true", help="force the CUDA-core fp32 kernels")
    ap.add_argument("--no-graph", action="store_true", help="time plain launches instead of a graph replay")
    ap.add_argument("--no-lively", action="store_true", help="skip the moving-preconditioner sub-record of cfg2")
    ap.add_argument("--no-sustained", action="store_true", help="skip the two-second back-to-back run")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.workload == "decode":
        run_decode(args)
        return
    steps = args.steps if args.steps is not None else 20
    warmup = max(args.warmup if args.warmup is not None else 5, 3)

    import torch
    import torch.distributed as dist
    from paper_2605_13473_b200 import binding
    from paper_2605_13473_b200.build import build

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        build()
    if world > 1:
        dist.barrier()
    binding.load_library()

    w = WORKLOADS[args.workload]
    inp = make_inputs(args.workload)
    flags = binding.FLAG_FORCE_SIMT if args.simt else 0
    tokens = inp.T_total

    def sync_all():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def prepare(inputs, with_bwd):
        """Device bundle, a step function and (unless --no-graph) a CUDA graph holding one step."""
        bundle = binding.DeviceBundle(inputs, dev, need_bwd=with_bwd, flags=flags)

        def step():
            if with_bwd:
                bundle.fwd(save=True)
                n = binding.osdn_last_launch_count()
                bundle.bwd(residuals_valid=True)
                return n + binding.osdn_last_launch_count()
            bundle.fwd(save=False)
            return binding.osdn_last_launch_count()

        for _ in range(warmup):
            step()
        torch.cuda.synchronize()
        assert bundle.device_status() == 0, "device-side error recorded during warm-up"
        # One step (osdn_fwd + osdn_bwd through the C ABI) captured once as a CUDA graph and replayed:
        # the calls only enqueue kernels on the stream they are given, so the capture holds exactly
        # the launches of the plain call sequence, without the launch gaps between them.
        graph, per_step = None, 0
        if not args.no_graph:
            try:
                cap = torch.cuda.Stream()
                with torch.cuda.stream(cap):
                    graph = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(graph, stream=cap):
                        per_step = step()
                torch.cuda.synchronize()
                for _ in range(3):
                    graph.replay()
                torch.cuda.synchronize()
            except Exception as exc:   # report and time the plain call sequence instead
                print(f"bench: graph capture failed ({exc}); timing plain launches", file=sys.stderr)
                graph = None
                torch.cuda.synchronize()
        return bundle, step, graph, per_step

    def timed(step, graph, per_step, n):
        """n steps between two events on the current stream; returns (ms, launches)."""
        sync_all()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        launches = 0
        e0.record()
        for _ in range(n):
            if graph is not None:
                graph.replay()
                launches += per_step
            else:
                launches += step()
        e1.record()
        sync_all()
        return e0.elapsed_time(e1), launches

    def per_kernel(step, n):
        """The same steps once more with an event between every two launches (the events cost a few
        percent of a step, so they stay out of the region `value` is timed on)."""
        binding.stage_timing_enable(True)
        sync_all()
        for _ in range(n):
            step()
        sync_all()
        st = binding.stage_timing_collect()
        binding.stage_timing_enable(False)
        return st

    b, step, graph, per_step = prepare(inp, w["bwd"])
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    ms_total, launches = timed(step, graph, per_step, steps)
    stages = per_kernel(step, steps)
    clocks = sampler.stop()
    assert b.device_status() == 0, "device-side error recorded during the timed region"

    # ---- sustained: the same step back to back for at least two seconds, clocks sampled meanwhile ----
    sustained = None
    if not args.no_sustained:
        n_sus = max(steps, int(2000.0 / max(ms_total / steps, 1e-3)) + 1)
        sus_sampler = ClockSampler(local)
        sus_sampler.start()
        time.sleep(0.2)
        ms_sus, _ = timed(step, graph, per_step, n_sus)
        sus_clocks = sus_sampler.stop()
        mhz = sus_clocks.get("sm_mhz")
        sustained = dict(steps=n_sus, seconds=ms_sus * 1e-3, ms_per_step=ms_sus / n_sus,
                         tokens_per_s=tokens * n_sus / (ms_sus * 1e-3), sm_mhz_median=mhz,
                         ms_times_mhz=(ms_sus / n_sus * mhz) if mhz else None, power_w_max=sus_clocks.get("power_w_max"),
                         reasons=sus_clocks.get("reasons"))

    # ---- the same shape with a preconditioner that really moves (no token is skipped) --------------
    lively = None
    if args.workload == "cfg2" and not args.no_lively and not args.simt:
        linp = make_inputs("cfg2_lively")
        lb, lstep, lgraph, lper = prepare(linp, True)
        ms_l, _ = timed(lstep, lgraph, lper, steps)
        lst = per_kernel(lstep, steps)
        assert lb.device_status() == 0
        ltot = {k: sum(v) / len(v) * 1e3 for k, v in lst.items()}
        ldom = max(ltot, key=ltot.get) if ltot else None
        lively = dict(workload=WORKLOADS["cfg2_lively"]["desc"], ms_per_step=ms_l / steps,
                      tokens_per_s=linp.T_total * steps / (ms_l * 1e-3), dominant_kernel=ldom,
                      kernels_us={k: round(v, 1) for k, v in sorted(ltot.items(), key=lambda kv: -kv[1])})
        del lb, lstep, lgraph

    # ---- end to end through the host-buffer entry point --------------------------------------
    e2e = None
    if inp.log_ret is None:
        pin = lambda t: None if t is None else t.contiguous().pin_memory()
        io_dt = torch.bfloat16 if inp.io_dtype == "bf16" else torch.float32
        hq, hk, hv = (pin(x.to(io_dt)) for x in (inp.q, inp.k, inp.v))
        hb, hg = pin(inp.beta), pin(inp.gate)
        hdo = pin(inp.dout.to(io_dt)) if w["bwd"] else None
        hout = torch.empty(tokens, inp.H, inp.V, dtype=io_dt).pin_memory()
        if w["bwd"]:
            hdq, hdk = (torch.empty(tokens, inp.H, inp.K, dtype=io_dt).pin_memory() for _ in range(2))
            hdv = torch.empty(tokens, inp.H, inp.V, dtype=io_dt).pin_memory()
            hdb, hdg = (torch.empty(tokens, inp.H, dtype=torch.float32).pin_memory() for _ in range(2))
        else:
            hdq = hdk = hdv = hdb = hdg = None
        staging = torch.empty(binding.osdn_host_staging_bytes(b.params, w["bwd"]), device=dev, dtype=torch.uint8)
        b.params.flags = flags

        def host_step():
            binding.osdn_step_host(b.params, hq, hk, hv, hb, hg, hdo, hout, hdq, hdk, hdv, hdb, hdg, staging)

        for _ in range(2):
            host_step()
        sync_all()
        h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0.record()
        for _ in range(steps):
            host_step()
        h1.record()
        sync_all()
        ms_host = h0.elapsed_time(h1)
        nb = lambda *ts: int(sum(t.numel() * t.element_size() for t in ts if t is not None))
        e2e = dict(ms=ms_host, h2d=nb(hq, hk, hv, hb, hg, hdo), d2h=nb(hout, hdq, hdk, hdv, hdb, hdg))

    # ---- whole-job numbers: units summed over ranks, time = max over ranks ----------------------
    from paper_2605_13473_b200.sharding import aggregate_throughput
    total_tokens, ms_total, _ = aggregate_throughput(tokens * steps, ms_total, dev)
    if e2e:
        _, e2e["ms"], _ = aggregate_throughput(tokens * steps, e2e["ms"], dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    value = total_tokens / (ms_total * 1e-3)
    # dominant kernel and its roofline: method bytes (or flops) per launch over the measured duration
    totals = {k: sum(v) for k, v in stages.items()}
    NT = sum((L + 63) // 64 for L in inp.seq_lens)
    roofline = None
    kernel_table = {}
    if totals:
        all_ms = sum(totals.values())
        for k, v in sorted(totals.items(), key=lambda kv: -kv[1]):
            kernel_table[k] = dict(launches=len(stages[k]), avg_us=1e3 * v / len(stages[k]), share=v / all_ms)
        dom = max(totals, key=totals.get)
        avg_s = totals[dom] / len(stages[dom]) * 1e-3
        model = kernel_model(dom, inp, NT)
        mbytes = method_bytes(dom, inp, w["bwd"])
        if model:
            dbytes, flops, bound = model
            traffic, traffic_source = load_traffic(args.workload, dom, avg_s * 1e6)
            if bound == "tensor":
                ach, peak, unit = flops / avg_s / 1e12, peaks["bf16_tflops_sustained"], "TFLOP/s"
            elif bound == "alu":
                # fp32 FMA peak of the chip: 148 SMs x 128 lanes x 2 flop x 1.965 GHz
                ach, peak, unit = flops / avg_s / 1e12, 148 * 128 * 2 * 1.965e9 / 1e12, "TFLOP/s"
            else:
                nb = mbytes if mbytes is not None else dbytes
                ach, peak, unit = nb / avg_s / 1e9, peaks["hbm_gbs"], "GB/s"
            roofline = dict(kernel=dom, bound=bound, achieved=ach, peak=peak, unit=unit, frac=ach / peak,
                            traffic=traffic, traffic_source=traffic_source, peak_source=peaks["source"],
                            avg_us=avg_s * 1e6,
                            algorithmic_bytes=mbytes if (mbytes is not None and bound == "hbm") else dbytes,
                            algorithmic_bytes_kind=("method bytes moved by this kernel (user tensors and one bf16 "
                                                    "state image per chunk)" if (mbytes is not None and bound == "hbm")
                                                    else "bytes of the design's data flow"),
                            design_bytes=dbytes, design_frac=(dbytes / avg_s / 1e9 / peaks["hbm_gbs"]) if bound == "hbm" else None,
                            algorithmic_flops=flops)
    # whole-step roofline (the slower of the step's flops at tensor peak and its bytes at HBM peak), for
    # two byte counts: the least any implementation moves (inputs, outputs, gradients once) and the
    # method's count with one bf16 state image per chunk saved by the forward and read by the backward
    es = 2 if inp.io_dtype == "bf16" else 4
    tokh = tokens * inp.H
    state = inp.V * inp.K * 2 / 64.0
    if w["bwd"]:
        min_bytes = tokh * ((2 * inp.K + inp.V) * es * 2 + inp.V * es * 2 + 16 + 16) + 0.0
        fwd_b = (2 * inp.K + inp.V) * es + 8 + inp.V * es + state + 8
        bwd_b = (2 * inp.K + inp.V) * es + inp.V * es + state + 8 + (2 * inp.K + inp.V) * es + 8
        method_step_bytes = tokh * (fwd_b + bwd_b)
        step_flops = tokh * 0.67e6 * (inp.K * inp.V) / (128 * 128)
    else:
        min_bytes = tokh * ((2 * inp.K + 2 * inp.V) * es + 8)
        method_step_bytes = min_bytes
        step_flops = tokh * 139264.0 * (inp.K * inp.V) / (128 * 128)
    t_flop = step_flops / (peaks["bf16_tflops"] * 1e12)
    t_roof = max(min_bytes / (peaks["hbm_gbs"] * 1e9), t_flop)
    t_roof_m = max(method_step_bytes / (peaks["hbm_gbs"] * 1e9), t_flop)
    step_s = ms_total / steps * 1e-3
    step_roof = dict(roofline_us=t_roof * 1e6, measured_us=step_s * 1e6, frac=t_roof / step_s, min_bytes=min_bytes,
                     flops=step_flops, method_bytes=method_step_bytes, method_roofline_us=t_roof_m * 1e6,
                     method_frac=t_roof_m / step_s)

    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        sys.path.insert(0, os.path.join(ROOT, "tests"))
        import oracle
        oracle.build()
        t0 = time.perf_counter()
        reps = 0
        while True:
            oracle.fwd_inputs(inp)
            if w["bwd"]:
                oracle.bwd_inputs(inp)
            reps += 1
            if time.perf_counter() - t0 > 10.0 or reps >= 50:
                break
        dt = time.perf_counter() - t0
        cpu_baseline = dict(value=tokens * reps / dt, unit="tokens/s", cores=oracle.threads(), kind="oracle",
                            sample=f"whole workload ({tokens} tokens x {inp.H} heads), {reps} repetitions, {dt:.1f} s")

    line = {
        "metric": "fwd+bwd tokens/s per layer" if w["bwd"] else "fwd tokens/s per layer",
        "value": value, "unit": "tokens/s", "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": ms_total / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if inp.io_dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": w["desc"], "l2": "inputs + workspace exceed L2 (no flush)",
                   "path": "simt" if args.simt else "auto", "tokens_per_step_per_gpu": tokens,
                   "launch": "cuda graph replay of one captured step" if graph is not None else "plain launches",
                   "kernel_timing": "second pass of the same steps with an event between launches"},
        "clocks": clocks, "gpu_launches": launches,
        "e2e": ({"value": total_tokens / (e2e["ms"] * 1e-3), "unit": "tokens/s",
                 "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"]} if e2e else None),
        "roofline": roofline, "step_roofline": step_roof, "kernels": kernel_table, "lively": lively,
        "sustained": sustained, "cpu_baseline": cpu_baseline,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
