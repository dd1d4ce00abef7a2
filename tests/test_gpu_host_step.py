"""osdn_step_host (host buffers, copies inside the call) against the device-resident entry points.

The host step of a dense batch is pipelined sequence by sequence over internal copy streams; a
packed batch goes in one piece.  Either way it must return what osdn_fwd + osdn_bwd return on the
same inputs (the only difference allowed is the summation order of a few atomics).
"""
import pytest
import torch

from paper_2605_13473_b200 import binding
from paper_2605_13473_b200.synth import config, draw

pytestmark = pytest.mark.gpu


def _pinned(t):
    return t.contiguous().pin_memory()


def _run_host(inp, b):
    io_dt = torch.bfloat16 if inp.io_dtype == "bf16" else torch.float32
    T = inp.T_total
    hq, hk, hv = (_pinned(x.to(io_dt)) for x in (inp.q, inp.k, inp.v))
    hb, hg, hdo = _pinned(inp.beta), _pinned(inp.gate), _pinned(inp.dout.to(io_dt))
    hout = torch.empty(T, inp.H, inp.V, dtype=io_dt).pin_memory()
    hdq, hdk = (torch.empty(T, inp.H, inp.K, dtype=io_dt).pin_memory() for _ in range(2))
    hdv = torch.empty(T, inp.H, inp.V, dtype=io_dt).pin_memory()
    hdb, hdg = (torch.empty(T, inp.H, dtype=torch.float32).pin_memory() for _ in range(2))
    staging = torch.empty(binding.osdn_host_staging_bytes(b.params, True), device="cuda:0", dtype=torch.uint8)
    for _ in range(2):   # twice in a row: the internal events and streams are reused
        binding.osdn_step_host(b.params, hq, hk, hv, hb, hg, hdo, hout, hdq, hdk, hdv, hdb, hdg, staging)
    torch.cuda.synchronize()
    return dict(out=hout, dq=hdq, dk=hdk, dv=hdv, dbeta=hdb, dgate=hdg)


def _close(x, y, tol):
    x, y = x.float().cpu(), y.float().cpu()
    scale = max(float(y.abs().max()), 1e-30)
    return float((x - y).abs().max()) / scale <= tol


@pytest.mark.parametrize("case", ["dense_bf16", "dense_fp32", "packed_bf16"])
def test_host_step_matches_device_calls(case):
    if case == "dense_bf16":
        inp = config(2, shrink=dict(B=3, T=320, H=2))
    elif case == "dense_fp32":
        inp = draw("host_fp32", 7, [200, 200], 2, 64, 64, "fp32", dense_B=2, with_dout=True)
    else:
        inp = config(4, shrink=dict(nseq=3, lo=70, hi=300, total=600, H=2))
    b = binding.DeviceBundle(inp, "cuda:0", need_bwd=True)
    b.fwd(save=True)
    b.bwd(residuals_valid=True)
    torch.cuda.synchronize()
    assert b.device_status() == 0
    got = _run_host(inp, b)
    assert b.device_status() == 0
    ref = dict(out=b.out, dq=b.dq, dk=b.dk, dv=b.dv, dbeta=b.dbeta, dgate=b.dgate)
    for key, val in got.items():
        assert _close(val, ref[key], 1e-5), key
