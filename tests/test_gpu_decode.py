"""osdn_decode_step: the recurrent step on a cached state and preconditioner.

1. Against the fp64 token-by-token oracle started from the same cache (the decode step is the
   recurrence itself, so the fp32 tolerance applies to the cache even for bf16 activations).
2. The paper's two equivalence checks between the recurrent and the chunk schedule (appendix
   "Numerical equivalence with the chunk forward"): T = 64 from an empty cache, and a prefill of 128
   tokens with the chunk path followed by one recurrent token against a chunk-only forward of 129.
"""
import numpy as np
import pytest
import torch

import oracle
import parity
from paper_2605_13473_b200 import binding
from paper_2605_13473_b200.synth import OsdnHyper, draw

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _io(t, io):
    return t.to(torch.bfloat16 if io == "bf16" else torch.float32).to(DEV).contiguous()


def _decode(inp, state, precond):
    """Runs the decode step over all tokens of a dense bundle; returns out and the updated cache."""
    B, L = inp.dense_B, inp.seq_lens[0]
    p = binding.make_params(B=B, T=L, H=inp.H, K=inp.K, V=inp.V, io_dtype=inp.io_dtype, hyper=inp.hyper)
    q, k, v = (_io(x, inp.io_dtype) for x in (inp.q, inp.k, inp.v))
    beta, gate = inp.beta.float().to(DEV), inp.gate.float().to(DEV)
    lr = None if inp.log_ret is None else inp.log_ret.float().to(DEV)
    st = state.float().to(DEV).contiguous().clone()
    dd = precond.float().to(DEV).contiguous().clone()
    out = torch.empty(B * L, inp.H, inp.V, device=DEV, dtype=q.dtype)
    binding.osdn_decode_step(p, q, k, v, beta, gate, lr, st, dd, out)
    torch.cuda.synchronize()
    assert binding.osdn_last_launch_count() == 1
    return out.float().cpu().numpy(), st.cpu().numpy(), dd.cpu().numpy()


def _rel(x, y):
    """Relative error in the Euclidean norm, the reading taken of the paper's "relative error" between
    two bf16 schedules (the max-normalised measure of the parity gate is also checked, at its own bound)."""
    x, y = np.asarray(x, dtype=np.float64), np.asarray(y, dtype=np.float64)
    return float(np.linalg.norm((x - y).ravel()) / max(np.linalg.norm(y.ravel()), 1e-300))


CASES = [
    # io, K, V, B, H, L, apf, clamp, beta_aware, eta
    ("fp32", 64, 64, 2, 2, 1, 1, 1, 1, 0.3),
    ("fp32", 128, 128, 2, 3, 7, 2, 1, 1, 0.3),
    ("fp32", 128, 64, 1, 2, 64, 0, 1, 0, 0.2),
    ("fp32", 64, 128, 3, 1, 5, 1, 0, 1, 0.05),
    ("bf16", 128, 128, 2, 2, 1, 1, 1, 1, 0.003),
    ("bf16", 128, 128, 2, 2, 33, 1, 1, 1, 0.3),
    ("bf16", 64, 64, 1, 4, 64, 2, 1, 1, 0.3),
    ("fp32", 128, 128, 2, 2, 9, 3, 1, 1, 0.3),    # vector retention
    ("bf16", 64, 128, 2, 2, 40, 3, 1, 0, 0.3),
]


@pytest.mark.parametrize("io,K,V,B,H,L,apf,clamp,ba,eta", CASES)
def test_decode_matches_oracle(io, K, V, B, H, L, apf, clamp, ba, eta):
    hy = OsdnHyper(eta=eta, apf_mode=apf, clamp=clamp, beta_aware=ba)
    inp = draw(f"decode_{io}_{K}_{V}_{L}", 900 + L + K, [L] * B, H, K, V, io, dense_B=B, hyper=hy,
               with_log_ret=(apf >= 2), with_state=True)
    got_out, got_S, got_d = _decode(inp, inp.init_state, inp.precond_in)
    ref = oracle.fwd_inputs(inp)
    assert parity.err(got_S, ref["final_state"]) <= 1e-4
    assert parity.err(got_d, ref["precond_out"]) <= 1e-4
    assert parity.err(got_out, ref["out"]) <= parity.TOL[io]


@pytest.mark.parametrize("L", [1, 64])
def test_decode_in_place_preconditioner_over_many_waves(L):
    """The preconditioner is advanced in place while every slice of a chain reads it: with a grid of
    several waves (512 chains x 8 slices) and a preconditioner that really moves (large step, no
    projection) a slice that started late must still see the vector the call was entered with."""
    hy = OsdnHyper(eta=0.3, apf_mode=1, clamp=0)
    B, H, D = 64, 8, 128
    inp = draw(f"decode_waves_{L}", 4100 + L, [L] * B, H, D, D, "bf16", dense_B=B, hyper=hy, with_state=True)
    got_out, got_S, got_d = _decode(inp, inp.init_state, inp.precond_in)
    ref = oracle.fwd_inputs(inp)
    assert parity.err(got_d, ref["precond_out"]) <= 1e-4
    assert parity.err(got_S, ref["final_state"]) <= 1e-4
    assert parity.err(got_out, ref["out"]) <= parity.TOL["bf16"]


def test_decode_continues_in_place_across_calls():
    """Two calls of 3 and 4 tokens equal one call of 7: the cache carries everything."""
    hy = OsdnHyper(eta=0.3, apf_mode=1)
    inp = draw("decode_split", 77, [7, 7], 2, 128, 128, "fp32", dense_B=2, hyper=hy, with_state=True)
    out7, S7, d7 = _decode(inp, inp.init_state, inp.precond_in)

    def part(lo, hi):
        import copy
        sub = copy.copy(inp)
        sel = lambda x: x.reshape(2, 7, *x.shape[1:])[:, lo:hi].reshape(2 * (hi - lo), *x.shape[1:]).contiguous()
        sub.q, sub.k, sub.v, sub.beta, sub.gate = (sel(x) for x in (inp.q, inp.k, inp.v, inp.beta, inp.gate))
        sub.seq_lens = [hi - lo, hi - lo]
        return sub
    o1, S1, d1 = _decode(part(0, 3), inp.init_state, inp.precond_in)
    o2, S2, d2 = _decode(part(3, 7), torch.from_numpy(S1), torch.from_numpy(d1))
    assert np.array_equal(S2, S7) and np.array_equal(d2, d7)
    full = out7.reshape(2, 7, 2, 128)
    assert np.array_equal(o1.reshape(2, 3, 2, 128), full[:, :3]) and np.array_equal(o2.reshape(2, 4, 2, 128), full[:, 3:])


@pytest.mark.parametrize("apf", [0, 1])
def test_recurrent_and_chunk_schedules_agree_T64(apf):
    """T = 64, bf16 activations, fp32 state, both decay modes: output, final state and final d of
    the two schedules within the paper's bounds (6.5e-3, 6.7e-3, 2.0e-3)."""
    hy = OsdnHyper(eta=0.003, apf_mode=apf)
    inp = draw("equiv64", 640 + apf, [64] * 4, 4, 128, 128, "bf16", dense_B=4, hyper=hy)
    chunk = binding.run_inputs_fwd(inp, DEV)
    S0 = torch.zeros(4, 4, 128, 128)
    d0 = torch.ones(4, 4, 128)
    out, S, d = _decode(inp, S0, d0)
    assert _rel(out, chunk["out"].numpy()) <= 6.5e-3
    assert _rel(S, chunk["final_state"].numpy()) <= 6.7e-3
    assert _rel(d, chunk["precond_out"].numpy()) <= 2.0e-3
    assert parity.err(out, chunk["out"].numpy()) <= parity.TOL["bf16"]
    assert parity.err(S, chunk["final_state"].numpy()) <= parity.TOL["bf16"]


@pytest.mark.parametrize("apf", [0, 1])
def test_prefill_128_then_one_recurrent_token_equals_chunk_129(apf):
    hy = OsdnHyper(eta=0.003, apf_mode=apf)
    B, H, D = 3, 4, 128
    full = draw("equiv129", 1290 + apf, [129] * B, H, D, D, "bf16", dense_B=B, hyper=hy)
    ref = binding.run_inputs_fwd(full, DEV)
    import copy
    cut = lambda x, lo, hi: x.reshape(B, 129, *x.shape[1:])[:, lo:hi].reshape(B * (hi - lo), *x.shape[1:]).contiguous()
    pre, last = copy.copy(full), copy.copy(full)
    for dst, lo, hi in ((pre, 0, 128), (last, 128, 129)):
        dst.q, dst.k, dst.v, dst.beta, dst.gate = (cut(x, lo, hi) for x in (full.q, full.k, full.v, full.beta, full.gate))
        dst.seq_lens = [hi - lo] * B
    prefill = binding.run_inputs_fwd(pre, DEV)
    out, S, d = _decode(last, prefill["final_state"], prefill["precond_out"])
    want = ref["out"].numpy().reshape(B, 129, H, D)[:, 128]
    assert _rel(out.reshape(B, H, D), want) <= 5.8e-3
    assert _rel(S, ref["final_state"].numpy()) <= 6.7e-3
    assert _rel(d, ref["precond_out"].numpy()) <= 2.0e-3
    assert parity.err(out.reshape(B, H, D), want) <= parity.TOL["bf16"]
