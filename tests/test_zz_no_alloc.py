"""osdn_fwd_static: the forward pass for callers that cannot allocate a workspace.

Some users of the library cannot call cudaMalloc where they need the layer (a serving loop with a
fixed memory pool, a plugin that only receives input and output buffers, code that must not
synchronise the device).  The entry point takes its scratch space from an array built into the
library instead.  This test calls it through the C ABI and checks it against osdn_fwd, twice in a
row, because all calls share the one array and the second call finds the first call's leftovers.

Collected last on purpose: a run that stops at the first failure has then run everything else.
"""
import pytest
import torch

import oracle
import parity
from paper_2605_13473_b200 import binding
from paper_2605_13473_b200.synth import OsdnHyper, config, draw

pytestmark = pytest.mark.gpu


def _reference(inp):
    b = binding.DeviceBundle(inp, "cuda:0", need_bwd=False)
    b.fwd()
    torch.cuda.synchronize()
    assert b.device_status() == 0
    return b, dict(out=b.out.float().cpu(), final_state=b.final_state.cpu(), precond_out=b.precond_out.cpu())


def _static(b):
    out = torch.full_like(b.out, float("nan"))
    fin = torch.full_like(b.final_state, float("nan"))
    dout = torch.full_like(b.precond_out, float("nan"))
    rc = binding.osdn_fwd_static(b.params, b.q, b.k, b.v, b.beta, b.gate, b.log_ret, b.init_state, b.precond_in,
                                 out, fin, dout)
    assert rc == 0, binding.status_string(rc)
    torch.cuda.synchronize()
    assert binding.osdn_read_static_status() == 0     # no device-side error inside the built-in array
    return dict(out=out.float().cpu(), final_state=fin.cpu(), precond_out=dout.cpu())


CASES = [
    ("cfg0_fp32", lambda: config(0)),
    ("bf16_tensor_core", lambda: config(1, shrink=dict(B=1, T=200, H=2))),
    ("varlen_state", lambda: draw("static_varlen", 77, [70, 3, 130], 2, 128, 128, "bf16",
                                  hyper=OsdnHyper(eta=0.3, apf_mode=1), with_state=True)),
]


@pytest.mark.parametrize("name,make", CASES, ids=[c[0] for c in CASES])
def test_static_scratch_forward_matches_workspace_forward(name, make):
    inp = make()
    b, ref = _reference(inp)
    assert binding.osdn_workspace_bytes(b.params, False) <= binding.STATIC_SCRATCH_BYTES
    first = _static(b)
    free_before = torch.cuda.mem_get_info()[0]
    second = _static(b)          # the shared array now holds the first call's contents
    assert torch.cuda.mem_get_info()[0] == free_before      # the call took no device memory
    want = oracle.fwd_inputs(inp)   # the definition itself, so that this test stands without osdn_fwd
    on_tc = inp.io_dtype == "bf16" and inp.K == 128 and inp.V == 128
    for got in (first, second):
        parity.compare(got, ref, inp.io_dtype, parity.FWD_KEYS, f"static_{name}")
        parity.compare(got, want, inp.io_dtype, parity.FWD_KEYS, f"static_{name}_vs_oracle", tensor_core=on_tc)
    # another problem in between, then the first one again
    other = config(1, shrink=dict(B=2, T=128, H=1))
    ob, oref = _reference(other)
    parity.compare(_static(ob), oref, other.io_dtype, parity.FWD_KEYS, "static_other")
    parity.compare(_static(b), ref, inp.io_dtype, parity.FWD_KEYS, f"static_{name}_again")


def test_static_scratch_rejects_problems_that_do_not_fit():
    inp = config(1, shrink=dict(B=1, T=64, H=1))
    b, _ = _reference(inp)
    big = binding.make_params(B=8, T=2048, H=8, K=128, V=128, io_dtype="bf16", hyper=inp.hyper)
    assert binding.osdn_workspace_bytes(big, False) > binding.STATIC_SCRATCH_BYTES
    out = torch.zeros(4, device="cuda:0")
    # rejected during validation: nothing is launched and no buffer is touched
    rc = binding.osdn_fwd_static(big, b.q, b.k, b.v, b.beta, b.gate, None, None, None, b.out, None, None)
    assert rc == -6
    assert "built-in scratch" in binding.status_string(rc)
    torch.cuda.synchronize()
    assert float(out.sum()) == 0.0
