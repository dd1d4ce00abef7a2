"""Helpers shared by the GPU parity tests: error measures, tolerances, chain sub-sampling."""
from __future__ import annotations

import copy

import numpy as np
import torch

import oracle

# Tolerances of the parity gate.
#   fp32 I/O : max|x - y| / max|y|  <= 1e-4  per tensor
#   bf16 I/O : max|x - y| / rms(y)  <= 2e-2  per tensor, i.e. a maximum absolute error of 2e-2 after
#              the tensor is brought to unit scale (gradients are normalised by their own rms the
#              same way).  Tensors the ABI returns in bf16 storage (out, dq, dk, dv) carry an
#              unavoidable final rounding of up to half a bf16 ulp, 2^-8 |y| per element -- already
#              2.1e-2 rms for an element 5.4 rms large -- so for those the bound applies to the
#              error in excess of that storage rounding: |x - y| - 2^-8 |y| <= 2e-2 rms(y).
TOL = {"fp32": 1e-4, "bf16": 2e-2}
BF16_STORED = ("out", "dq", "dk", "dv")

FWD_KEYS = ("out", "final_state", "precond_out")
BWD_KEYS = ("dq", "dk", "dv", "dbeta", "dgate", "dlog_ret", "dinit_state", "dprecond_in")


def err(x, y, io_dtype, bf16_stored=False):
    x = np.asarray(x, dtype=np.float64)
    y = np.asarray(y, dtype=np.float64)
    if y.size == 0:
        return 0.0
    ad = np.abs(x - y)
    if bf16_stored:
        ad = np.maximum(ad - 2.0 ** -8 * np.abs(y), 0.0)
    diff = ad.max()
    if not np.isfinite(x).all():
        return float("inf")
    if io_dtype == "fp32":
        den = np.abs(y).max()
    else:
        den = np.sqrt(np.mean(y * y))
    if den < 1e-30:
        return float(diff)  # reference is identically zero: absolute error
    return float(diff / den)


def subset(inp, seqs, heads):
    """Restrict an input bundle to some sequences and heads (chains are independent)."""
    out = copy.copy(inp)
    cu = np.concatenate([[0], np.cumsum(inp.seq_lens)])
    tok = np.concatenate([np.arange(cu[s], cu[s + 1]) for s in seqs]) if len(seqs) else np.zeros(0, int)
    tok_t = torch.as_tensor(tok, dtype=torch.long)
    hd = torch.as_tensor(list(heads), dtype=torch.long)

    def tk(x):
        return None if x is None else x.index_select(0, tok_t).index_select(1, hd).contiguous()

    def st(x):
        return None if x is None else x.index_select(0, torch.as_tensor(list(seqs))).index_select(1, hd).contiguous()

    for name in ("q", "k", "v", "beta", "gate", "log_ret", "dout"):
        setattr(out, name, tk(getattr(inp, name)))
    for name in ("init_state", "precond_in", "dfinal_state", "dprecond_out"):
        setattr(out, name, st(getattr(inp, name)))
    out.seq_lens = [inp.seq_lens[s] for s in seqs]
    out.H = len(heads)
    out.dense_B = 0
    return out, tok_t, hd


def subset_result(res, seqs, heads, tok_t, hd):
    sq = torch.as_tensor(list(seqs))
    out = {}
    for k, v in res.items():
        v = torch.as_tensor(v)
        if k in ("final_state", "precond_out", "dinit_state", "dprecond_in"):
            out[k] = v.index_select(0, sq).index_select(1, hd).numpy()
        else:
            out[k] = v.index_select(0, tok_t).index_select(1, hd).numpy()
    return out


def oracle_all(inp, bwd: bool):
    ref = oracle.fwd_inputs(inp)
    if bwd:
        ref.update(oracle.bwd_inputs(inp))
    return ref


def compare(got, ref, io_dtype, keys, label="", tol=None, report=None):
    tol = TOL[io_dtype] if tol is None else tol
    worst = {}
    for k in keys:
        if k not in ref or k not in got:
            continue
        e = err(got[k], ref[k], io_dtype, io_dtype == "bf16" and k in BF16_STORED)
        worst[k] = e
    if report is not None:
        report[label] = worst
    bad = {k: e for k, e in worst.items() if not (e <= tol)}
    assert not bad, f"{label}: parity failed {bad} (tol {tol}); all: {worst}"
    return worst
