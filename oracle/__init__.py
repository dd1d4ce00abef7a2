"""ctypes front end of the fp64 CPU oracle (``osdn_oracle.c``).

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports this module;
it is used by the tests, by the smoke check and by the CPU-baseline leg of the
benchmark.  It never touches the CUDA library.

``build()`` compiles the C file with gcc (OpenMP over the independent
(sequence, head) chains).  All arrays cross the boundary as contiguous float64
numpy arrays in the packed layout ``[T_total, H, *]``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "osdn_oracle.c")
_SO = os.path.join(_HERE, "liboracle.so")
_lib = None


class _Hyper(ctypes.Structure):
    _fields_ = [("eta", ctypes.c_double), ("d_min", ctypes.c_double), ("d_max", ctypes.c_double),
                ("eps", ctypes.c_double), ("scale", ctypes.c_double),
                ("beta_aware", ctypes.c_int), ("apf_mode", ctypes.c_int), ("clamp", ctypes.c_int),
                ("channel_gate", ctypes.c_int)]


def build(force: bool = False) -> str:
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-shared", "-fPIC", "-o", _SO, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _SO


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.osdn_oracle_threads.restype = ctypes.c_int
    return _lib


def threads() -> int:
    return int(_load().osdn_oracle_threads())


def _hyper(hy, K: int) -> _Hyper:
    scale = float(hy.scale) if hy.scale and hy.scale > 0 else float(K) ** -0.5
    return _Hyper(float(hy.eta), float(hy.d_min), float(hy.d_max), float(hy.eps), scale,
                  int(hy.beta_aware), int(hy.apf_mode), int(hy.clamp), int(_channel_gate(hy)))


def _channel_gate(hy) -> bool:
    """OSKDA: `gate` holds one log-gate per key channel, [T, H, K]; the aliased retention mode is undefined."""
    cg = bool(getattr(hy, "channel_gate", False))
    assert not (cg and hy.apf_mode == 1), "the preconditioner's retention is separate from a channel gate"
    return cg


def _f64(x) -> Optional[np.ndarray]:
    if x is None:
        return None
    if hasattr(x, "detach"):
        x = x.detach().cpu().to(dtype=__import__("torch").float64).numpy()
    return np.ascontiguousarray(np.asarray(x, dtype=np.float64))


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _cu(seq_lens: Sequence[int]) -> np.ndarray:
    return np.concatenate([[0], np.cumsum(np.asarray(seq_lens, dtype=np.int64))]).astype(np.int32)


def fwd(hy, seq_lens, q, k, v, beta, gate, log_ret=None, init_state=None, precond_in=None,
        want_ktil: bool = False, want_dtraj: bool = False, want_margin: bool = False) -> dict:
    """Token-by-token forward.  Returns dict(out, final_state, precond_out[, ktil, d_traj])."""
    lib = _load()
    q, k, v, beta, gate = map(_f64, (q, k, v, beta, gate))
    log_ret, init_state, precond_in = map(_f64, (log_ret, init_state, precond_in))
    T, H, K = q.shape
    V = v.shape[-1]
    cu = _cu(seq_lens)
    nseq = len(seq_lens)
    assert cu[-1] == T
    assert gate.shape == ((T, H, K) if _channel_gate(hy) else (T, H))
    if hy.apf_mode == 2:
        assert log_ret is not None and log_ret.shape == (T, H)
    if hy.apf_mode == 3:
        assert log_ret is not None and log_ret.shape == (T, H, K)
    out = np.zeros((T, H, V))
    S = np.zeros((nseq, H, V, K))
    d = np.zeros((nseq, H, K))
    ktil = np.zeros((T, H, K)) if want_ktil else None
    dtraj = np.zeros((T, H, K)) if want_dtraj else None
    margin = np.zeros((T, H, K)) if want_margin else None
    mask = np.zeros((T, H, K), dtype=np.uint8) if want_margin else None
    hp = _hyper(hy, K)
    lib.osdn_oracle_fwd(ctypes.c_int(nseq), _p(cu), ctypes.c_int(H), ctypes.c_int(K),
                        ctypes.c_int(V), ctypes.byref(hp), _p(q), _p(k), _p(v), _p(beta), _p(gate),
                        _p(log_ret), _p(init_state), _p(precond_in), _p(out), _p(S), _p(d),
                        _p(ktil), _p(dtraj), _p(margin), _p(mask))
    res = dict(out=out, final_state=S, precond_out=d)
    if want_margin:
        res["margin"] = margin
        res["mask"] = mask
    if want_ktil:
        res["ktil"] = ktil
    if want_dtraj:
        res["d_traj"] = dtraj
    return res


def residual_ratio(hy, seq_lens, k, v, beta, gate, log_ret=None, init_state=None, precond_in=None) -> np.ndarray:
    """q_t = f_t(S_t) / f_t(exp(g_t) S_{t-1}) with f_t(S) = |S k_t - v_t|^2 / 2, from the states
    themselves (the definition; not the closed form).  Returns [T, H]."""
    lib = _load()
    k, v, beta, gate = map(_f64, (k, v, beta, gate))
    log_ret, init_state, precond_in = map(_f64, (log_ret, init_state, precond_in))
    T, H, K = k.shape
    V = v.shape[-1]
    assert not _channel_gate(hy)
    cu = _cu(seq_lens)
    out = np.zeros((T, H))
    hp = _hyper(hy, K)
    lib.osdn_oracle_residual_ratio(ctypes.c_int(len(seq_lens)), _p(cu), ctypes.c_int(H), ctypes.c_int(K),
                                   ctypes.c_int(V), ctypes.byref(hp), _p(k), _p(v), _p(beta), _p(gate),
                                   _p(log_ret), _p(init_state), _p(precond_in), _p(out))
    return out


def precond_update(hy, seq_lens, k, beta, gate=None, log_ret=None, precond_in=None) -> dict:
    lib = _load()
    k, beta, gate, log_ret, precond_in = map(_f64, (k, beta, gate, log_ret, precond_in))
    T, H, K = k.shape
    cu = _cu(seq_lens)
    nseq = len(seq_lens)
    ktil = np.zeros((T, H, K))
    d = np.zeros((nseq, H, K))
    hp = _hyper(hy, K)
    lib.osdn_oracle_precond_update(ctypes.c_int(nseq), _p(cu), ctypes.c_int(H), ctypes.c_int(K),
                                   ctypes.byref(hp), _p(k), _p(beta), _p(gate), _p(log_ret),
                                   _p(precond_in), _p(ktil), _p(d))
    return dict(ktil=ktil, precond_out=d)


def bwd(hy, seq_lens, q, k, v, beta, gate, dout, log_ret=None, init_state=None, precond_in=None,
        dfinal_state=None, dprecond_out=None, mask_override=None) -> dict:
    """Reverse sweep.  mask_override: uint8 [T,H,K], 0/1 force a projection pass decision, 255 = default.
  Returns dict(dq, dk, dv, dbeta, dgate, dlog_ret, dinit_state, dprecond_in)."""
    lib = _load()
    q, k, v, beta, gate, dout = map(_f64, (q, k, v, beta, gate, dout))
    log_ret, init_state, precond_in = map(_f64, (log_ret, init_state, precond_in))
    dfinal_state, dprecond_out = map(_f64, (dfinal_state, dprecond_out))
    T, H, K = q.shape
    V = v.shape[-1]
    cu = _cu(seq_lens)
    nseq = len(seq_lens)
    dq, dk, dv = np.zeros((T, H, K)), np.zeros((T, H, K)), np.zeros((T, H, V))
    assert gate.shape == ((T, H, K) if _channel_gate(hy) else (T, H))
    dbeta, dgate = np.zeros((T, H)), np.zeros((T, H, K) if _channel_gate(hy) else (T, H))
    dlr = np.zeros((T, H, K)) if hy.apf_mode == 3 else np.zeros((T, H))
    dS0, dd0 = np.zeros((nseq, H, V, K)), np.zeros((nseq, H, K))
    hp = _hyper(hy, K)
    mo = None if mask_override is None else np.ascontiguousarray(mask_override, dtype=np.uint8)
    lib.osdn_oracle_bwd(ctypes.c_int(nseq), _p(cu), ctypes.c_int(H), ctypes.c_int(K),
                        ctypes.c_int(V), ctypes.byref(hp), _p(q), _p(k), _p(v), _p(beta), _p(gate),
                        _p(log_ret), _p(init_state), _p(precond_in), _p(dout), _p(dfinal_state),
                        _p(dprecond_out), _p(mo), _p(dq), _p(dk), _p(dv), _p(dbeta), _p(dgate), _p(dlr),
                        _p(dS0), _p(dd0))
    return dict(dq=dq, dk=dk, dv=dv, dbeta=dbeta, dgate=dgate, dlog_ret=dlr,
                dinit_state=dS0, dprecond_in=dd0)


def fwd_inputs(inp, **kw) -> dict:
    """Forward on an ``OsdnInputs`` bundle from the synthetic generator."""
    return fwd(inp.hyper, inp.seq_lens, inp.q, inp.k, inp.v, inp.beta, inp.gate, inp.log_ret,
               inp.init_state, inp.precond_in, **kw)


def bwd_inputs(inp, mask_override=None) -> dict:
    return bwd(inp.hyper, inp.seq_lens, inp.q, inp.k, inp.v, inp.beta, inp.gate, inp.dout,
               inp.log_ret, inp.init_state, inp.precond_in, inp.dfinal_state, inp.dprecond_out,
               mask_override=mask_override)
