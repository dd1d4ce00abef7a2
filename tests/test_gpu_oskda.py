"""Channel-gate variant of the layer (OSKDA extension) on the GPU, through osdn_kda_fwd / osdn_kda_bwd,
element by element against the fp64 oracle's channel-gate mode on the same seeded inputs."""
import numpy as np
import pytest
import torch

import oracle
import parity
from paper_2605_13473_b200 import binding
from paper_2605_13473_b200.synth import OsdnHyper, draw

pytestmark = pytest.mark.gpu

FWD = ("out", "final_state", "precond_out")
BWD = FWD + ("dq", "dk", "dv", "dbeta", "dgate", "dlog_ret", "dinit_state", "dprecond_in")


def _case(seed, seq_lens, H, K, V, io, apf_mode, dense_B=0, gate_kind="softplus", eta=0.3, **kw):
    hy = OsdnHyper(eta=eta, apf_mode=apf_mode, channel_gate=1)
    return draw("oskda", seed, seq_lens, H, K, V, io, dense_B=dense_B, hyper=hy, with_log_ret=apf_mode >= 2,
                with_state=True, with_dout=True, with_state_cotangents=True, gate_kind=gate_kind, **kw)


CASES = {
    # several chunks and a ragged tail, both widths, both dtypes, every retention mode the extension has
    "fp32_k128_sep": dict(seed=61, seq_lens=[200, 200], H=2, K=128, V=128, io="fp32", apf_mode=2, dense_B=2),
    "fp32_k64_none": dict(seed=62, seq_lens=[150], H=3, K=64, V=64, io="fp32", apf_mode=0, dense_B=1),
    "fp32_k64v128_vec": dict(seed=63, seq_lens=[130], H=2, K=64, V=128, io="fp32", apf_mode=3, dense_B=1),
    "bf16_k128_sep": dict(seed=64, seq_lens=[256, 256], H=2, K=128, V=128, io="bf16", apf_mode=2, dense_B=2),
    "fp32_varlen": dict(seed=65, seq_lens=[1, 64, 0, 129, 63], H=2, K=128, V=64, io="fp32", apf_mode=2),
    "fp32_strong_gates": dict(seed=66, seq_lens=[192], H=2, K=128, V=128, io="fp32", apf_mode=2, dense_B=1,
                              gate_kind="strong"),
    # the paper's setting for this extension: constant retention 0.999, small step
    "bf16_const_retention": dict(seed=67, seq_lens=[320], H=4, K=128, V=128, io="bf16", apf_mode=2, dense_B=1,
                                 eta=0.003),
}


@pytest.mark.parametrize("name", sorted(CASES))
def test_forward_and_backward_match_the_oracle(name):
    c = dict(CASES[name])
    inp = _case(**c)
    if name == "bf16_const_retention":
        inp.log_ret = torch.full_like(inp.log_ret, float(np.log(0.999)))
    got = binding.run_inputs_bwd(inp)
    ref = parity.oracle_all(inp, bwd=True, gpu_masks=got["projection_masks"])
    parity.compare(got, ref, inp.io_dtype, BWD, label="oskda/" + name)


def test_forward_alone_and_recomputed_residuals():
    inp = _case(71, [100, 100], 2, 128, 128, "fp32", 2, dense_B=2)
    f = binding.run_inputs_fwd(inp)
    ref = oracle.fwd_inputs(inp)
    parity.compare(f, ref, "fp32", FWD, label="oskda/fwd_only")
    a = binding.run_inputs_bwd(inp, reuse_residuals=True)
    b = binding.run_inputs_bwd(inp, reuse_residuals=False)
    for k in ("dq", "dk", "dv", "dgate", "dinit_state"):
        # the cross-row sums are atomic additions: equal up to their order
        np.testing.assert_allclose(a[k].numpy(), b[k].numpy(), rtol=1e-4, atol=1e-5)


def test_equal_channels_reproduce_the_scalar_gate_kernels():
    """With the same gate in every channel the extension is the layer itself: compare the two CUDA paths."""
    inp = _case(72, [192], 2, 128, 128, "fp32", 2, dense_B=1)
    g = inp.gate[..., 0].contiguous()
    inp.gate = g.unsqueeze(-1).expand(-1, -1, inp.K).contiguous()
    kda = binding.run_inputs_bwd(inp)
    import copy
    plain = copy.copy(inp)
    plain.hyper = OsdnHyper(eta=0.3, apf_mode=2, channel_gate=0)
    plain.gate = g
    ref = binding.run_inputs_bwd(plain)
    for k in ("out", "final_state", "dq", "dk", "dv", "dbeta", "dinit_state", "dprecond_in"):
        assert parity.err(kda[k].numpy(), ref[k].double().numpy(), "fp32") <= 1e-4, k
    assert parity.err(kda["dgate"].sum(-1).numpy(), ref["dgate"].double().numpy(), "fp32") <= 1e-4


def test_alias_mode_is_rejected():
    hy = OsdnHyper(eta=0.3, apf_mode=1)
    p = binding.make_params(B=1, T=64, H=1, K=64, V=64, io_dtype="fp32", hyper=hy)
    assert binding.osdn_kda_workspace_bytes(p, False) == 0
