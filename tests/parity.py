"""Helpers shared by the GPU parity tests: error measures, tolerances, chain sub-sampling."""
from __future__ import annotations

import copy

import numpy as np
import torch

import oracle

# Tolerances of the parity gate: per tensor, max|x - y| / max|y| (the maximum absolute error after
# the reference tensor is scaled to unit magnitude)
#   fp32 I/O : <= 1e-4
#   bf16 I/O : <= 2e-2   (bf16 operands, fp32 accumulation)
# The report also records max|x - y| / rms(y), which is stricter by the tensor's crest factor.
TOL = {"fp32": 1e-4, "bf16": 2e-2}

FWD_KEYS = ("out", "final_state", "precond_out")
BWD_KEYS = ("dq", "dk", "dv", "dbeta", "dgate", "dlog_ret", "dinit_state", "dprecond_in")


def err(x, y, io_dtype=None, norm="max"):
    """max|x - y| normalised by max|y| (default) or rms(y); absolute if the reference is all zero."""
    x = np.asarray(x, dtype=np.float64)
    y = np.asarray(y, dtype=np.float64)
    if y.size == 0:
        return 0.0
    if not np.isfinite(x).all():
        return float("inf")
    diff = np.abs(x - y).max()
    den = np.abs(y).max() if norm == "max" else np.sqrt(np.mean(y * y))
    if den < 1e-30:
        return float(diff)
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
        if v is None:
            continue
        v = torch.as_tensor(v)
        if k in ("final_state", "precond_out", "dinit_state", "dprecond_in"):
            out[k] = v.index_select(0, sq).index_select(1, hd).numpy()
        else:
            out[k] = v.index_select(0, tok_t).index_select(1, hd).numpy()
    return out


TIE = 2e-6   # |pre-projection value - box face| below which fp32 and fp64 may decide differently


def oracle_all(inp, bwd: bool, gpu_masks=None):
    """Oracle forward (and backward).  The gradient is discontinuous where a pre-projection value of
    the preconditioner touches a face of the box.  Where the oracle's fp64 value is within TIE of a
    face the decision is not unique at fp32 resolution: there (and only there) the oracle's reverse
    sweep takes the decision the CUDA path took (`gpu_masks`); everywhere else the two must agree."""
    if not bwd:
        return oracle.fwd_inputs(inp)
    ref = oracle.fwd_inputs(inp, want_margin=True)
    override = None
    if gpu_masks is not None and inp.hyper.clamp:
        gm = np.asarray(gpu_masks, dtype=np.uint8)
        near = ref["margin"] <= TIE
        disagree = (gm != ref["mask"]) & ~near
        assert not disagree.any(), f"{int(disagree.sum())} projection decisions differ away from any tie"
        override = np.where(near, gm, 255).astype(np.uint8)
        ref["near_ties"] = int(near.sum())
    ref.update(oracle.bwd_inputs(inp, mask_override=override))
    return ref


def compare(got, ref, io_dtype, keys, label="", tol=None, report=None):
    tol = TOL[io_dtype] if tol is None else tol
    worst = {}
    for k in keys:
        if k not in ref or k not in got:
            continue
        worst[k] = err(got[k], ref[k], io_dtype)
    if report is not None:
        report[label] = dict(worst)
        report[label + "/rms_normalised"] = {k: err(got[k], ref[k], io_dtype, "rms") for k in worst}
    bad = {k: e for k, e in worst.items() if not (e <= tol)}
    assert not bad, f"{label}: parity failed {bad} (tol {tol}); all: {worst}"
    return worst
