"""ctypes binding of ``libosdn.so`` (argument marshalling only)."""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libosdn.so")
_lib = None

FLAG_SAVE_RESIDUALS = 1
FLAG_RESIDUALS_VALID = 2
FLAG_FORCE_SIMT = 4

EXPORTS = [
    "osdn_workspace_bytes", "osdn_fwd", "osdn_bwd", "osdn_precond_update", "osdn_host_staging_bytes",
    "osdn_step_host", "osdn_read_device_status", "osdn_status_string", "osdn_last_launch_count",
    "osdn_stage_timing_enable", "osdn_stage_timing_read", "osdn_workspace_region",
    "osdn_fwd_static", "osdn_decode_step", "osdn_residual_ratio", "osdn_read_static_status",
    "osdn_selftest_wait_timeout", "osdn_kda_workspace_bytes", "osdn_kda_fwd", "osdn_kda_bwd",
]


class OsdnParams(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("T", ctypes.c_int32), ("H", ctypes.c_int32), ("K", ctypes.c_int32),
        ("V", ctypes.c_int32), ("chunk", ctypes.c_int32), ("io_dtype", ctypes.c_int32),
        ("eta", ctypes.c_float), ("d_min", ctypes.c_float), ("d_max", ctypes.c_float),
        ("eps", ctypes.c_float), ("scale", ctypes.c_float),
        ("beta_aware", ctypes.c_int32), ("apf_mode", ctypes.c_int32), ("clamp", ctypes.c_int32),
        ("nseq", ctypes.c_int32), ("cu_seqlens", ctypes.c_void_p), ("flags", ctypes.c_int32),
    ]


def load_library(path: Optional[str] = None):
    """Loads libosdn.so (building nothing: run ``build.py`` / ``__graft_entry__.build`` first)."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    path = path or _LIB_PATH
    if not os.path.exists(path):
        raise RuntimeError(f"{path} not found: build the CUDA library first "
                           "(python paper_2605_13473_b200/build.py); there is no fallback path")
    lib = ctypes.CDLL(path)
    vp, sz, ci = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
    pp = ctypes.POINTER(OsdnParams)
    lib.osdn_workspace_bytes.restype = sz
    lib.osdn_workspace_bytes.argtypes = [pp, ci]
    lib.osdn_host_staging_bytes.restype = sz
    lib.osdn_host_staging_bytes.argtypes = [pp, ci]
    lib.osdn_fwd.restype = ci
    lib.osdn_fwd.argtypes = [pp] + [vp] * 11 + [vp, sz, vp]
    lib.osdn_fwd_static.restype = ci
    lib.osdn_fwd_static.argtypes = [pp] + [vp] * 11 + [vp]
    lib.osdn_bwd.restype = ci
    lib.osdn_bwd.argtypes = [pp] + [vp] * 19 + [vp, sz, vp]
    lib.osdn_precond_update.restype = ci
    lib.osdn_precond_update.argtypes = [pp] + [vp] * 6 + [vp]
    lib.osdn_residual_ratio.restype = ci
    lib.osdn_residual_ratio.argtypes = [pp] + [vp] * 7 + [vp]
    lib.osdn_decode_step.restype = ci
    lib.osdn_decode_step.argtypes = [pp] + [vp] * 9 + [vp]
    lib.osdn_step_host.restype = ci
    lib.osdn_step_host.argtypes = [pp] + [vp] * 12 + [vp, sz, vp]
    lib.osdn_read_device_status.restype = ci
    lib.osdn_read_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int32)]
    lib.osdn_read_static_status.restype = ci
    lib.osdn_read_static_status.argtypes = [ctypes.POINTER(ctypes.c_int32)]
    lib.osdn_selftest_wait_timeout.restype = ci
    lib.osdn_selftest_wait_timeout.argtypes = [vp, ctypes.c_uint32, vp]
    lib.osdn_status_string.restype = ctypes.c_char_p
    lib.osdn_status_string.argtypes = [ci]
    lib.osdn_last_launch_count.restype = ci
    lib.osdn_last_launch_count.argtypes = []
    lib.osdn_stage_timing_enable.restype = None
    lib.osdn_stage_timing_enable.argtypes = [ci]
    lib.osdn_stage_timing_read.restype = ci
    lib.osdn_stage_timing_read.argtypes = [ci, ctypes.POINTER(ctypes.c_char_p), ctypes.POINTER(ctypes.c_float)]
    lib.osdn_workspace_region.restype = ci
    lib.osdn_workspace_region.argtypes = [pp, ci, ctypes.c_char_p, ctypes.POINTER(sz), ctypes.POINTER(sz)]
    if path == _LIB_PATH:
        _lib = lib
    return lib


def status_string(code: int) -> str:
    return load_library().osdn_status_string(code).decode()


def _check(code: int, what: str):
    if code != 0:
        raise RuntimeError(f"{what} failed: {status_string(code)} ({code})")


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_contiguous():
        raise ValueError("tensors passed to the OSDN library must be contiguous")
    return ctypes.c_void_p(t.data_ptr())


def _stream_ptr():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def make_params(*, B: int, T: int, H: int, K: int, V: int, io_dtype: str, hyper=None,
                cu_seqlens: Optional[torch.Tensor] = None, flags: int = 0) -> OsdnParams:
    """``hyper``: any object with eta, d_min, d_max, eps, scale, beta_aware, apf_mode, clamp, chunk."""
    p = OsdnParams()
    p.B, p.T, p.H, p.K, p.V = B, T, H, K, V
    p.chunk = getattr(hyper, "chunk", 64)
    p.io_dtype = {"fp32": 0, "bf16": 1}[io_dtype]
    p.eta = getattr(hyper, "eta", 0.003)
    p.d_min = getattr(hyper, "d_min", 0.5)
    p.d_max = getattr(hyper, "d_max", 2.0)
    p.eps = getattr(hyper, "eps", 1e-6)
    p.scale = getattr(hyper, "scale", 0.0)
    p.beta_aware = getattr(hyper, "beta_aware", 1)
    p.apf_mode = getattr(hyper, "apf_mode", 1)
    p.clamp = getattr(hyper, "clamp", 1)
    if cu_seqlens is not None:
        assert cu_seqlens.dtype == torch.int32 and cu_seqlens.is_cuda
        p.nseq = cu_seqlens.numel() - 1
        p.cu_seqlens = cu_seqlens.data_ptr()
    else:
        p.nseq = 0
        p.cu_seqlens = None
    p.flags = flags
    return p


def osdn_workspace_bytes(p: OsdnParams, need_bwd: bool) -> int:
    return int(load_library().osdn_workspace_bytes(ctypes.byref(p), int(need_bwd)))


def osdn_host_staging_bytes(p: OsdnParams, with_bwd: bool) -> int:
    return int(load_library().osdn_host_staging_bytes(ctypes.byref(p), int(with_bwd)))


def osdn_last_launch_count() -> int:
    return int(load_library().osdn_last_launch_count())


def stage_timing_enable(on: bool):
    load_library().osdn_stage_timing_enable(int(on))


def stage_timing_collect() -> dict:
    """{kernel name: [durations in ms]} of the marks recorded since the last enable (sync first)."""
    lib = load_library()
    name, ms = ctypes.c_char_p(), ctypes.c_float()
    n = lib.osdn_stage_timing_read(-1, None, None)
    out = {}
    for i in range(max(n - 1, 0)):
        lib.osdn_stage_timing_read(i, ctypes.byref(name), ctypes.byref(ms))
        if name.value is not None:
            out.setdefault(name.value.decode(), []).append(float(ms.value))
    return out


def workspace_region(p: OsdnParams, name: str):
    """(offset, bytes) of a named region of a backward-capable workspace."""
    off, nb = ctypes.c_size_t(0), ctypes.c_size_t(0)
    _check(load_library().osdn_workspace_region(ctypes.byref(p), 1, name.encode(), ctypes.byref(off),
                                                ctypes.byref(nb)), "osdn_workspace_region")
    return int(off.value), int(nb.value)


def osdn_read_device_status(workspace: torch.Tensor) -> int:
    out = ctypes.c_int32(0)
    _check(load_library().osdn_read_device_status(_ptr(workspace), ctypes.byref(out)), "osdn_read_device_status")
    return int(out.value)


def osdn_fwd(p: OsdnParams, q, k, v, beta, gate, apf_log_ret, init_state, precond_in, out, final_state,
             precond_out, workspace: torch.Tensor):
    lib = load_library()
    rc = lib.osdn_fwd(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(gate), _ptr(apf_log_ret),
                      _ptr(init_state), _ptr(precond_in), _ptr(out), _ptr(final_state), _ptr(precond_out),
                      _ptr(workspace), ctypes.c_size_t(workspace.numel() * workspace.element_size()),
                      _stream_ptr())
    _check(rc, "osdn_fwd")


def osdn_kda_workspace_bytes(p: OsdnParams, need_bwd: bool) -> int:
    lib = load_library()
    lib.osdn_kda_workspace_bytes.restype = ctypes.c_size_t
    return int(lib.osdn_kda_workspace_bytes(ctypes.byref(p), ctypes.c_int(1 if need_bwd else 0)))


def osdn_kda_fwd(p: OsdnParams, q, k, v, beta, gate_k, apf_log_ret, init_state, precond_in, out, final_state,
                 precond_out, workspace: torch.Tensor):
    """Channel-gate variant (OSKDA extension): ``gate_k`` is [T,H,K] fp32; the rest as for ``osdn_fwd``."""
    lib = load_library()
    rc = lib.osdn_kda_fwd(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(gate_k), _ptr(apf_log_ret),
                          _ptr(init_state), _ptr(precond_in), _ptr(out), _ptr(final_state), _ptr(precond_out),
                          _ptr(workspace), ctypes.c_size_t(workspace.numel() * workspace.element_size()),
                          _stream_ptr())
    _check(rc, "osdn_kda_fwd")


def osdn_kda_bwd(p: OsdnParams, q, k, v, beta, gate_k, apf_log_ret, init_state, precond_in, dout, dfinal_state,
                 dprecond_out, dq, dk, dv, dbeta, dgate_k, dapf_log_ret, dinit_state, dprecond_in,
                 workspace: torch.Tensor):
    lib = load_library()
    rc = lib.osdn_kda_bwd(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(gate_k), _ptr(apf_log_ret),
                          _ptr(init_state), _ptr(precond_in), _ptr(dout), _ptr(dfinal_state), _ptr(dprecond_out),
                          _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dbeta), _ptr(dgate_k), _ptr(dapf_log_ret),
                          _ptr(dinit_state), _ptr(dprecond_in), _ptr(workspace),
                          ctypes.c_size_t(workspace.numel() * workspace.element_size()), _stream_ptr())
    _check(rc, "osdn_kda_bwd")


STATIC_SCRATCH_BYTES = 32 << 20


def osdn_fwd_static(p: OsdnParams, q, k, v, beta, gate, apf_log_ret, init_state, precond_in, out, final_state,
                    precond_out) -> int:
    """Forward pass on the library's built-in scratch array: for callers that cannot allocate a
    workspace.  Returns the status code (0 = ok, -6 = the problem does not fit the built-in scratch)
    instead of raising, so that a caller can fall back to ``osdn_fwd`` with its own workspace."""
    lib = load_library()
    return int(lib.osdn_fwd_static(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(gate),
                                   _ptr(apf_log_ret), _ptr(init_state), _ptr(precond_in), _ptr(out),
                                   _ptr(final_state), _ptr(precond_out), _stream_ptr()))


def osdn_read_static_status() -> int:
    """Device status word of the most recent ``osdn_fwd_static`` call on the current device
    (0 = no device-side error).  Synchronise the stream first."""
    lib = load_library()
    st = ctypes.c_int32(0)
    _check(lib.osdn_read_static_status(ctypes.byref(st)), "osdn_read_static_status")
    return int(st.value)


def osdn_selftest_wait_timeout(workspace: torch.Tensor, limit_us: int) -> None:
    """Launches the self-test of the bounded device-side wait on ``workspace`` (>= 256 bytes)."""
    lib = load_library()
    _check(lib.osdn_selftest_wait_timeout(_ptr(workspace), ctypes.c_uint32(limit_us), _stream_ptr()),
           "osdn_selftest_wait_timeout")


def osdn_bwd(p: OsdnParams, q, k, v, beta, gate, apf_log_ret, init_state, precond_in, dout, dfinal_state,
             dprecond_out, dq, dk, dv, dbeta, dgate, dapf_log_ret, dinit_state, dprecond_in,
             workspace: torch.Tensor):
    lib = load_library()
    rc = lib.osdn_bwd(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(gate), _ptr(apf_log_ret),
                      _ptr(init_state), _ptr(precond_in), _ptr(dout), _ptr(dfinal_state), _ptr(dprecond_out),
                      _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dbeta), _ptr(dgate), _ptr(dapf_log_ret),
                      _ptr(dinit_state), _ptr(dprecond_in), _ptr(workspace),
                      ctypes.c_size_t(workspace.numel() * workspace.element_size()), _stream_ptr())
    _check(rc, "osdn_bwd")


def osdn_precond_update(p: OsdnParams, k, beta, gate_or_log_ret, precond_in, k_tilde_out, precond_out):
    lib = load_library()
    rc = lib.osdn_precond_update(ctypes.byref(p), _ptr(k), _ptr(beta), _ptr(gate_or_log_ret), _ptr(precond_in),
                                 _ptr(k_tilde_out), _ptr(precond_out), _stream_ptr())
    _check(rc, "osdn_precond_update")


def osdn_residual_ratio(p: OsdnParams, k, beta, gate_or_log_ret, precond_in, ratio_out, log_ratio_sum, precond_out=None):
    lib = load_library()
    rc = lib.osdn_residual_ratio(ctypes.byref(p), _ptr(k), _ptr(beta), _ptr(gate_or_log_ret), _ptr(precond_in),
                                 _ptr(ratio_out), _ptr(log_ratio_sum), _ptr(precond_out), _stream_ptr())
    _check(rc, "osdn_residual_ratio")


def osdn_decode_step(p: OsdnParams, q, k, v, beta, gate, apf_log_ret, state, precond, out):
    """``state`` [B,H,V,K] and ``precond`` [B,H,K] (fp32, device) are updated in place."""
    lib = load_library()
    rc = lib.osdn_decode_step(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(gate), _ptr(apf_log_ret),
                              _ptr(state), _ptr(precond), _ptr(out), _stream_ptr())
    _check(rc, "osdn_decode_step")


def osdn_step_host(p: OsdnParams, q, k, v, beta, gate, dout, out, dq, dk, dv, dbeta, dgate,
                   staging: torch.Tensor):
    """All tensor arguments except ``staging`` are HOST tensors (pinned for async copies)."""
    lib = load_library()
    rc = lib.osdn_step_host(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(gate), _ptr(dout),
                            _ptr(out), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dbeta), _ptr(dgate), _ptr(staging),
                            ctypes.c_size_t(staging.numel() * staging.element_size()), _stream_ptr())
    _check(rc, "osdn_step_host")


# ---------------------------------------------------------------------------------------------
# Convenience used by tests, smoke and bench: move an input bundle to the device and call the ABI.
# ---------------------------------------------------------------------------------------------
def _io(t: Optional[torch.Tensor], io_dtype: str, dev):
    if t is None:
        return None
    dt = torch.bfloat16 if io_dtype == "bf16" else torch.float32
    return t.to(device=dev, dtype=dt).contiguous()


def _f32(t: Optional[torch.Tensor], dev):
    return None if t is None else t.to(device=dev, dtype=torch.float32).contiguous()


class DeviceBundle:
    """Device copies of an input bundle plus output / gradient buffers and the workspace."""

    def __init__(self, inp, device="cuda:0", need_bwd: bool = True, flags: int = 0):
        dev = torch.device(device)
        self.inp = inp
        io = inp.io_dtype
        self.q, self.k, self.v = _io(inp.q, io, dev), _io(inp.k, io, dev), _io(inp.v, io, dev)
        self.beta, self.gate = _f32(inp.beta, dev), _f32(inp.gate, dev)
        self.log_ret = _f32(inp.log_ret, dev)
        self.init_state, self.precond_in = _f32(inp.init_state, dev), _f32(inp.precond_in, dev)
        self.dout = _io(inp.dout, io, dev)
        self.dfinal_state, self.dprecond_out = _f32(inp.dfinal_state, dev), _f32(inp.dprecond_out, dev)
        T, H, K, V, S = inp.T_total, inp.H, inp.K, inp.V, inp.nseq
        if inp.dense_B > 0:
            self.cu = None
            self.params = make_params(B=inp.dense_B, T=T // inp.dense_B, H=H, K=K, V=V, io_dtype=io,
                                      hyper=inp.hyper, flags=flags)
        else:
            self.cu = inp.cu_seqlens.to(dev)
            self.params = make_params(B=1, T=T, H=H, K=K, V=V, io_dtype=io, hyper=inp.hyper,
                                      cu_seqlens=self.cu, flags=flags)
        dt = torch.bfloat16 if io == "bf16" else torch.float32
        self.out = torch.empty(T, H, V, device=dev, dtype=dt)
        self.final_state = torch.empty(S, H, V, K, device=dev, dtype=torch.float32)
        self.precond_out = torch.empty(S, H, K, device=dev, dtype=torch.float32)
        self.channel_gate = bool(getattr(inp.hyper, "channel_gate", 0))   # OSKDA extension: gate is [T,H,K]
        nbytes = (osdn_kda_workspace_bytes if self.channel_gate else osdn_workspace_bytes)(self.params, need_bwd)
        if nbytes == 0:
            raise RuntimeError("osdn_workspace_bytes rejected the parameters")
        self.workspace = torch.empty(nbytes, device=dev, dtype=torch.uint8)
        if need_bwd:
            self.dq = torch.empty(T, H, K, device=dev, dtype=dt)
            self.dk = torch.empty(T, H, K, device=dev, dtype=dt)
            self.dv = torch.empty(T, H, V, device=dev, dtype=dt)
            self.dbeta = torch.empty(T, H, device=dev, dtype=torch.float32)
            self.dgate = torch.empty((T, H, K) if self.channel_gate else (T, H), device=dev, dtype=torch.float32)
            mode = int(self.params.apf_mode)
            if mode >= 2:   # written in full by osdn_bwd ([T,H], or [T,H,K] for the vector retention)
                self.dlog_ret = torch.full((T, H, K) if mode == 3 else (T, H), float("nan"), device=dev)
            else:           # not touched by the library
                self.dlog_ret = torch.zeros(T, H, device=dev, dtype=torch.float32)
            self.dinit_state = torch.empty(S, H, V, K, device=dev, dtype=torch.float32)
            self.dprecond_in = torch.empty(S, H, K, device=dev, dtype=torch.float32)

    def fwd(self, save: bool = False):
        base = self.params.flags & FLAG_FORCE_SIMT
        self.params.flags = base | (FLAG_SAVE_RESIDUALS if save else 0)
        (osdn_kda_fwd if self.channel_gate else osdn_fwd)(
            self.params, self.q, self.k, self.v, self.beta, self.gate, self.log_ret, self.init_state,
            self.precond_in, self.out, self.final_state, self.precond_out, self.workspace)

    def bwd(self, residuals_valid: bool = False):
        base = self.params.flags & FLAG_FORCE_SIMT
        self.params.flags = base | (FLAG_RESIDUALS_VALID if residuals_valid else 0)
        (osdn_kda_bwd if self.channel_gate else osdn_bwd)(
            self.params, self.q, self.k, self.v, self.beta, self.gate, self.log_ret, self.init_state,
            self.precond_in, self.dout, self.dfinal_state, self.dprecond_out, self.dq, self.dk, self.dv,
            self.dbeta, self.dgate, self.dlog_ret, self.dinit_state, self.dprecond_in, self.workspace)

    def device_status(self) -> int:
        return osdn_read_device_status(self.workspace)

    def projection_masks(self) -> torch.Tensor:
        """uint8 [T,H,K] pass masks of the projection as the forward (with saved residuals) took them."""
        inp = self.inp
        T, H, K = inp.T_total, inp.H, inp.K
        o1, n1 = workspace_region(self.params, "p1_skip")
        o2, n2 = workspace_region(self.params, "p1_mask")
        skip = self.workspace[o1:o1 + n1].view(torch.int32).cpu().numpy().astype("uint32").reshape(-1, H, 2)
        words = self.workspace[o2:o2 + n2].view(torch.int32).cpu().numpy().astype("uint32").reshape(T, H, 32)
        import numpy as np
        R = K // 32   # bit r of word l <-> coordinate R * l + r
        bits = ((words[..., None] >> np.arange(R, dtype=np.uint32)) & 1).astype(np.uint8)   # [T,H,32,R]
        bits = np.ascontiguousarray(bits).reshape(T, H, K)
        skipped = np.zeros((T, H), dtype=bool)
        c = 0
        t0 = 0
        for L in inp.seq_lens:
            for j in range((L + 63) // 64):
                n = min(64, L - 64 * j)
                w = skip[c].astype(np.uint64)
                pair = w[:, 0] | (w[:, 1] << np.uint64(32))
                sk = ((pair[None, :] >> np.arange(n, dtype=np.uint64)[:, None]) & np.uint64(1)).astype(bool)
                skipped[t0 + 64 * j:t0 + 64 * j + n] = sk
                c += 1
            t0 += L
        bits[skipped] = 0
        if not inp.hyper.clamp:
            bits[:] = 1
        return torch.from_numpy(bits)


def run_inputs_fwd(inp, device="cuda:0", flags: int = 0) -> dict:
    b = DeviceBundle(inp, device, need_bwd=False, flags=flags)
    b.fwd()
    torch.cuda.synchronize()
    assert b.device_status() == 0
    return dict(out=b.out.float().cpu(), final_state=b.final_state.cpu(), precond_out=b.precond_out.cpu())


def run_inputs_bwd(inp, device="cuda:0", flags: int = 0, reuse_residuals: bool = True) -> dict:
    b = DeviceBundle(inp, device, need_bwd=True, flags=flags)
    b.fwd(save=reuse_residuals)
    b.bwd(residuals_valid=reuse_residuals)
    torch.cuda.synchronize()
    assert b.device_status() == 0
    masks = b.projection_masks() if reuse_residuals else None
    return dict(out=b.out.float().cpu(), final_state=b.final_state.cpu(), precond_out=b.precond_out.cpu(),
                projection_masks=masks, dq=b.dq.float().cpu(), dk=b.dk.float().cpu(), dv=b.dv.float().cpu(), dbeta=b.dbeta.cpu(),
                dgate=b.dgate.cpu(), dlog_ret=b.dlog_ret.cpu(), dinit_state=b.dinit_state.cpu(),
                dprecond_in=b.dprecond_in.cpu())
