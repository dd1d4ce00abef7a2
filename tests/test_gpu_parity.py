"""GPU parity: the CUDA path (through the C ABI) against the fp64 oracle, element by element."""
import numpy as np
import pytest
import torch

import oracle
import parity
from paper_2605_13473_b200 import binding, run_inputs_bwd, run_inputs_fwd
from paper_2605_13473_b200.synth import OsdnHyper, config, draw, lively

pytestmark = pytest.mark.gpu

REPORT = {}


def teardown_module(module):
    """Writes every measure of every case as JSON to the file named by OSDN_PARITY_REPORT, if set."""
    parity.write_report(REPORT)


def _on_tensor_cores(inp, flags):
    return inp.io_dtype == "bf16" and inp.K == 128 and inp.V == 128 and not (flags & binding.FLAG_FORCE_SIMT)


def _check(inp, bwd, label, flags=0, tol=None, take_over_ties=True, rms_ceiling=None):
    got = run_inputs_bwd(inp, flags=flags) if bwd else run_inputs_fwd(inp, flags=flags)
    ref = parity.oracle_all(inp, bwd, got.get("projection_masks") if take_over_ties else None)
    keys = parity.FWD_KEYS + (parity.BWD_KEYS if bwd else ())
    return parity.compare(got, ref, inp.io_dtype, keys, label, tol=tol, report=REPORT,
                          tensor_core=_on_tensor_cores(inp, flags), rms_ceiling=rms_ceiling)


PATHS = [("simt", binding.FLAG_FORCE_SIMT), ("auto", 0)]


def test_cfg0_tiny_forward_fp32():
    _check(config(0), False, "cfg0")


def test_cfg0_shape_backward_fp32():
    inp = draw("cfg0_bwd", 10, [256], 1, 64, 64, "fp32", dense_B=1, with_dout=True,
               with_state=True, with_state_cotangents=True)
    _check(inp, True, "cfg0_bwd")


@pytest.mark.parametrize("path,flags", PATHS, ids=[p[0] for p in PATHS])
@pytest.mark.parametrize("idx", [1, 2, 3, 4])
def test_benchmark_configs_reduced(idx, path, flags):
    shrink = {1: dict(B=2, T=320, H=2), 2: dict(B=2, T=320, H=2), 3: dict(B=1, T=448, H=3),
              4: dict(nseq=5, lo=40, hi=700, total=1500, H=2)}[idx]
    inp = config(idx, shrink=shrink)
    _check(inp, idx >= 2, f"cfg{idx}_reduced_{path}", flags=flags)


@pytest.mark.parametrize("path,flags", PATHS, ids=[p[0] for p in PATHS])
@pytest.mark.parametrize("io", ["fp32", "bf16"])
@pytest.mark.parametrize("idx", [1, 2, 3, 4, 5, 6, 7])
def test_lively_sets(idx, io, path, flags):
    if io == "fp32" and path == "auto":
        pytest.skip("fp32 I/O always runs the CUDA-core kernels")
    inp = lively(idx, T=200, B=2, H=2, D=128, io_dtype=io)
    _check(inp, True, f"lively{idx}_{io}_{path}", flags=flags)


@pytest.mark.parametrize("io,D,seed,kind", [("bf16", 128, 2010, "alias"), ("fp32", 64, 2015, "sparse")],
                         ids=["tensor_core", "cuda_core"])
def test_backward_owes_nothing_to_the_gpu_masks(io, D, seed, kind):
    """One case per kernel family in which the oracle's reverse sweep takes every projection decision
    by itself: the seeds were chosen (on the CPU, from the oracle's own margins) so that the box is
    active for part of the coordinates and no pre-projection value lies within 1e-4 of a face."""
    if kind == "alias":
        hy, extra = OsdnHyper(eta=0.3, apf_mode=1), {}
    else:
        hy, extra = OsdnHyper(eta=0.3, apf_mode=2), dict(key_kind="sparse", with_log_ret=True)
    inp = draw("noties", seed, [100], 1, D, D, io, dense_B=1, hyper=hy, with_dout=True, with_state=True,
               with_state_cotangents=True, **extra)
    probe = oracle.fwd_inputs(inp, want_margin=True)
    assert probe["margin"].min() > 1e-4 and 0.02 < probe["mask"].mean() < 0.98
    _check(inp, True, f"no_ties_{io}", take_over_ties=False)


@pytest.mark.parametrize("path,flags", PATHS, ids=[p[0] for p in PATHS])
@pytest.mark.parametrize("K,V", [(64, 64), (64, 128), (128, 64)])
@pytest.mark.parametrize("T", [1, 63, 65, 200])
def test_shapes_and_ragged_tails(T, K, V, path, flags):
    hy = OsdnHyper(eta=0.3, apf_mode=1)
    inp = draw(f"shape_{T}_{K}_{V}", 700 + T + K + V, [T, T], 2, K, V, "bf16", dense_B=2, hyper=hy,
               with_dout=True, with_state=True, with_state_cotangents=True)
    _check(inp, True, f"shape_T{T}_K{K}_V{V}_{path}", flags=flags)


@pytest.mark.parametrize("io", ["fp32", "bf16"])
@pytest.mark.parametrize("K,V", [(64, 64), (64, 128)])
def test_vector_retention_small_heads_and_ragged_batch(K, V, io):
    """One log-retention per coordinate with K = 64 (two coordinates per lane), packed ragged batch
    with an empty sequence, forward and backward."""
    hy = OsdnHyper(eta=0.3, apf_mode=3)
    inp = draw(f"vec_{K}_{V}_{io}", 990 + K + V, [130, 0, 65, 1], 2, K, V, io, hyper=hy, key_kind="sparse",
               with_dout=True, with_log_ret=True, with_state=True, with_state_cotangents=True, log_ret_shift=3.0)
    _check(inp, True, f"vector_ret_K{K}_V{V}_{io}")


@pytest.mark.parametrize("path,flags", PATHS, ids=[p[0] for p in PATHS])
def test_degenerate_inputs(path, flags):
    hy = OsdnHyper(eta=0.3, apf_mode=1)
    inp = draw("degenerate", 900, [130, 0, 70, 3], 2, 128, 128, "bf16", hyper=hy, with_dout=True,
               with_state=True, with_state_cotangents=True)
    inp.beta[:40] = 0.0          # no-op writes
    inp.beta[40:60] = 1.0        # full-step writes
    inp.k[100:110] = 0.0         # zero keys: the eps floor of the normaliser
    inp.gate[120:125] = -20.0    # near-total forgetting
    _check(inp, True, f"degenerate_{path}", flags=flags)


def test_precond_update_alone():
    hy = OsdnHyper(eta=0.3, apf_mode=2)
    inp = draw("pu", 950, [150, 64, 7], 3, 128, 128, "bf16", hyper=hy, with_log_ret=True, with_state=True)
    dev = torch.device("cuda:0")
    b = binding.DeviceBundle(inp, dev, need_bwd=False)
    ktil = torch.empty_like(b.k)
    dout = torch.empty_like(b.precond_in)
    binding.osdn_precond_update(b.params, b.k, b.beta, b.log_ret, b.precond_in, ktil, dout)
    torch.cuda.synchronize()
    ref = oracle.precond_update(hy, inp.seq_lens, inp.k, inp.beta, None, inp.log_ret, inp.precond_in)
    assert parity.err(dout.cpu().numpy(), ref["precond_out"], "fp32") <= 1e-5
    assert parity.err(ktil.float().cpu().numpy(), ref["ktil"], "bf16") <= 2e-2
    # streaming: two calls with the preconditioner carried equal one call (dense, fp32)
    inp2 = draw("pu2", 951, [90], 2, 64, 64, "fp32", dense_B=1, hyper=OsdnHyper(eta=0.3, apf_mode=1))
    b2 = binding.DeviceBundle(inp2, dev, need_bwd=False)
    d_all = torch.empty(1, 2, 64, device=dev)
    binding.osdn_precond_update(b2.params, b2.k, b2.beta, b2.gate, None, None, d_all)
    p1 = binding.make_params(B=1, T=50, H=2, K=64, V=64, io_dtype="fp32", hyper=inp2.hyper)
    p2 = binding.make_params(B=1, T=40, H=2, K=64, V=64, io_dtype="fp32", hyper=inp2.hyper)
    d_mid = torch.empty(1, 2, 64, device=dev)
    binding.osdn_precond_update(p1, b2.k[:50].contiguous(), b2.beta[:50].contiguous(), b2.gate[:50].contiguous(),
                                None, None, d_mid)
    binding.osdn_precond_update(p2, b2.k[50:].contiguous(), b2.beta[50:].contiguous(), b2.gate[50:].contiguous(),
                                d_mid, None, d_mid)
    torch.cuda.synchronize()
    assert torch.equal(d_mid, d_all)


@pytest.mark.parametrize("io,K", [("bf16", 128), ("fp32", 64)])
def test_precond_update_vector_retention(io, K):
    """One log-retention per coordinate ([T,H,K]), packed batch with ragged sequences."""
    hy = OsdnHyper(eta=0.3, apf_mode=3)
    inp = draw(f"pu_vec_{io}", 952, [150, 64, 7], 3, K, K, io, hyper=hy, with_log_ret=True, with_state=True,
               key_kind="sparse", log_ret_shift=3.0)
    assert tuple(inp.log_ret.shape) == (221, 3, K)
    dev = torch.device("cuda:0")
    b = binding.DeviceBundle(inp, dev, need_bwd=False)
    ktil = torch.empty_like(b.k)
    dout = torch.empty_like(b.precond_in)
    binding.osdn_precond_update(b.params, b.k, b.beta, b.log_ret, b.precond_in, ktil, dout)
    torch.cuda.synchronize()
    ref = oracle.precond_update(hy, inp.seq_lens, inp.k, inp.beta, None, inp.log_ret, inp.precond_in)
    assert parity.err(dout.cpu().numpy(), ref["precond_out"], "fp32") <= 1e-5
    assert parity.err(ktil.float().cpu().numpy(), ref["ktil"], io) <= parity.TOL[io]
    # the sweep of osdn_fwd and the stand-alone update agree on the final preconditioner
    full = run_inputs_fwd(inp)
    assert parity.err(full["precond_out"].numpy(), dout.cpu().numpy(), "fp32") <= 1e-6


def test_split_sequence_state_carry_on_gpu():
    hy = OsdnHyper(eta=0.3, apf_mode=1)
    inp = draw("carry", 960, [192], 2, 128, 128, "fp32", dense_B=1, hyper=hy)
    full = run_inputs_fwd(inp)
    first = draw("carry", 960, [192], 2, 128, 128, "fp32", dense_B=1, hyper=hy)
    for name in ("q", "k", "v", "beta", "gate"):
        setattr(first, name, getattr(inp, name)[:128].contiguous())
    first.seq_lens = [128]
    r1 = run_inputs_fwd(first)
    second = draw("carry", 960, [192], 2, 128, 128, "fp32", dense_B=1, hyper=hy)
    for name in ("q", "k", "v", "beta", "gate"):
        setattr(second, name, getattr(inp, name)[128:].contiguous())
    second.seq_lens = [64]
    second.init_state, second.precond_in = r1["final_state"], r1["precond_out"]
    r2 = run_inputs_fwd(second)
    assert parity.err(torch.cat([r1["out"], r2["out"]]).numpy(), full["out"].numpy(), "fp32") <= 1e-5
    assert parity.err(r2["final_state"].numpy(), full["final_state"].numpy(), "fp32") <= 1e-5
    assert parity.err(r2["precond_out"].numpy(), full["precond_out"].numpy(), "fp32") <= 1e-6


def test_backward_with_and_without_saved_residuals_agree():
    inp = lively(1, T=150, B=1, H=2, D=128, io_dtype="bf16")
    a = run_inputs_bwd(inp, reuse_residuals=True)
    b = run_inputs_bwd(inp, reuse_residuals=False)
    for k in parity.BWD_KEYS:
        assert parity.err(a[k].numpy(), b[k].numpy(), "fp32") <= 1e-5, k


def test_run_to_run_determinism():
    inp = config(2, shrink=dict(B=1, T=256, H=2))
    a = run_inputs_bwd(inp)
    b = run_inputs_bwd(inp)
    for k in ("out", "final_state", "dq", "dv", "dinit_state"):
        assert torch.equal(a[k], b[k]), k


@pytest.mark.parametrize("case", ["many_chains_dense", "many_chains_packed", "long_tail_packed", "equal_packed"])
def test_forward_launch_variants_of_the_tensor_core_path(case):
    """The forward of phase 2 is one launch while enough SMs are left to feed the chains and two launches
    otherwise; packed batches go through the sorted tile list and the three-group variant, dense ones
    through the arithmetic order.  Every variant, forward and backward, against the oracle."""
    hy = OsdnHyper(eta=0.3, apf_mode=1)
    kw = dict(hyper=hy, with_dout=True, with_state=True, with_state_cotangents=True)
    if case == "many_chains_dense":      # 120 chains: no SMs left over, chunk-local pass and chains as two launches
        inp = draw(case, 301, [130] * 20, 6, 128, 128, "bf16", dense_B=20, **kw)
    elif case == "many_chains_packed":
        inp = draw(case, 302, [70, 40, 129, 64, 33] * 8, 3, 128, 128, "bf16", **kw)
    elif case == "long_tail_packed":     # one long sequence among short ones, an empty one, single-token ones
        inp = draw(case, 303, [700, 64, 0, 1, 130, 65, 1, 320], 2, 128, 128, "bf16", **kw)
    else:                                # equal lengths given as a packed batch
        inp = draw(case, 304, [192] * 4, 2, 128, 128, "bf16", **kw)
    # ragged sets with carried-in states: the largest elements stand 15-30 times above the rms, so the
    # third measure (largest error over rms) gets its own ceiling here; the other two gates are the usual ones
    _check(inp, True, "fwd_variants/" + case, rms_ceiling=0.16)


@pytest.mark.parametrize("case", ["k64_fp32", "two_groups_fp32", "packed_ragged_bf16", "vector_two_groups_fp32",
                                  "update_only_k64"])
def test_pipelined_stretches_of_the_sequential_passes(case):
    """Where nearly every token is processed the sequential preconditioner kernels hand a chain to three
    warps (stretches of up to eight chunks, blocks of 16 / 8 tokens through a ring).  Cases that the small
    sets above do not reach: K = 64, sequences longer than one group of 32 chunks (stretches end at group
    boundaries), packed sequences whose stretches start and end on ragged chunks, the vector retention,
    and the stand-alone update (the same pipeline over a whole sequence) with a block tail."""
    if case == "k64_fp32":
        hy = OsdnHyper(eta=0.3, apf_mode=2)
        inp = draw(case, 401, [333, 333], 2, 64, 64, "fp32", dense_B=2, hyper=hy, key_kind="sparse", with_dout=True,
                   with_log_ret=True, with_state=True, with_state_cotangents=True)
    elif case == "two_groups_fp32":
        hy = OsdnHyper(eta=0.3, apf_mode=2)
        inp = draw(case, 402, [2300], 1, 64, 64, "fp32", dense_B=1, hyper=hy, key_kind="sparse", with_dout=True,
                   with_log_ret=True, with_state=True, with_state_cotangents=True)
    elif case == "packed_ragged_bf16":
        hy = OsdnHyper(eta=0.3, apf_mode=2)
        inp = draw(case, 403, [700, 65, 130, 1, 577], 2, 128, 128, "bf16", hyper=hy, key_kind="sparse", with_dout=True,
                   with_log_ret=True, with_state=True, with_state_cotangents=True)
    elif case == "vector_two_groups_fp32":
        hy = OsdnHyper(eta=0.3, apf_mode=3)
        inp = draw(case, 404, [2100], 1, 64, 64, "fp32", dense_B=1, hyper=hy, key_kind="sparse", with_dout=True,
                   with_log_ret=True, with_state=True, with_state_cotangents=True, log_ret_shift=3.0)
    else:
        hy = OsdnHyper(eta=0.3, apf_mode=2)
        inp = draw(case, 405, [203, 16, 1], 3, 64, 64, "fp32", hyper=hy, key_kind="sparse", with_log_ret=True, with_state=True)
        dev = "cuda:0"
        b = binding.DeviceBundle(inp, dev, need_bwd=False)
        ktil = torch.empty_like(b.k)
        d_out = torch.empty_like(b.precond_in)
        binding.osdn_precond_update(b.params, b.k, b.beta, b.log_ret, b.precond_in, ktil, d_out)
        torch.cuda.synchronize()
        ref = oracle.precond_update(hy, inp.seq_lens, inp.k, inp.beta, None, inp.log_ret, inp.precond_in)
        assert parity.err(ktil.float().cpu().numpy(), ref["ktil"], "fp32") <= 1e-4
        assert parity.err(d_out.cpu().numpy(), ref["precond_out"], "fp32") <= 1e-4
        return
    _check(inp, True, "pipelined/" + case, rms_ceiling=0.16 if inp.io_dtype == "bf16" else None)
