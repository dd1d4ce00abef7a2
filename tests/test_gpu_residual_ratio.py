"""osdn_residual_ratio: the mechanism diagnostic q_t as a by-product of the preconditioner sweep,
against the oracle, which forms the ratio from the states themselves (f_t(S_t) / f_t(S_{t-1}))."""
import numpy as np
import pytest
import torch

import oracle
import parity
from paper_2605_13473_b200 import binding
from paper_2605_13473_b200.synth import OsdnHyper, draw

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

CASES = [
    # io, K, lens, dense_B, eta, apf, beta_aware
    ("bf16", 128, [200, 200], 2, 0.003, 1, 1),      # the benchmark setting: d settles on the lower face
    ("bf16", 128, [150, 64, 7, 0, 90], 0, 0.3, 2, 1),
    ("fp32", 64, [130], 1, 0.3, 0, 0),
    ("fp32", 128, [77, 50], 0, 0.0, 0, 1),           # eta = 0: the unscaled delta rule
    ("bf16", 64, [96, 96, 96], 3, 0.2, 3, 1),        # vector retention
]


@pytest.mark.parametrize("io,K,lens,dense_B,eta,apf,ba", CASES)
def test_residual_ratio_matches_definition(io, K, lens, dense_B, eta, apf, ba):
    hy = OsdnHyper(eta=eta, apf_mode=apf, beta_aware=ba)
    inp = draw(f"ratio_{io}_{K}_{apf}", 1200 + K + apf, lens, 2, K, K, io, dense_B=dense_B, hyper=hy,
               with_log_ret=(apf >= 2), with_state=True)
    b = binding.DeviceBundle(inp, DEV, need_bwd=False)
    T, H, S = inp.T_total, inp.H, len(lens)
    ratio = torch.full((T, H), float("nan"), device=DEV)
    lsum = torch.full((S, H), float("nan"), device=DEV)
    dout = torch.empty(S, H, K, device=DEV)
    src = b.log_ret if apf >= 2 else b.gate
    binding.osdn_residual_ratio(b.params, b.k, b.beta, src, b.precond_in, ratio, lsum, dout)
    torch.cuda.synchronize()
    assert binding.osdn_last_launch_count() == 1
    want = oracle.residual_ratio(hy, lens, inp.k, inp.v, inp.beta, inp.gate, inp.log_ret, inp.init_state,
                                 inp.precond_in)
    got = ratio.cpu().numpy()
    assert np.abs(got - want).max() <= 1e-4 * max(1.0, np.abs(want).max())
    # per-chain log sums (tokens whose ratio is far from zero dominate; compare as geometric means)
    cu = np.concatenate([[0], np.cumsum(lens)])
    for s, n in enumerate(lens):
        for h in range(H):
            ref = float(np.log(np.maximum(want[cu[s]:cu[s + 1], h], np.finfo(np.float32).tiny)).sum())
            if n == 0:
                assert lsum[s, h].item() == 0.0
            elif want[cu[s]:cu[s + 1], h].min() > 1e-6:
                assert abs(np.exp(lsum[s, h].item() / n) - np.exp(ref / n)) <= 1e-3 * np.exp(ref / n)
    # the sweep itself is the stand-alone update
    ref_d = oracle.precond_update(hy, lens, inp.k, inp.beta, inp.gate, inp.log_ret, inp.precond_in)["precond_out"]
    assert parity.err(dout.cpu().numpy(), ref_d, "fp32") <= 1e-5


def test_only_one_output_requested():
    hy = OsdnHyper(eta=0.003, apf_mode=1)
    inp = draw("ratio_one", 1300, [64, 64], 1, 128, 128, "bf16", dense_B=2, hyper=hy)
    b = binding.DeviceBundle(inp, DEV, need_bwd=False)
    ratio = torch.empty(128, 1, device=DEV)
    lsum = torch.empty(2, 1, device=DEV)
    binding.osdn_residual_ratio(b.params, b.k, b.beta, b.gate, None, ratio, None)
    binding.osdn_residual_ratio(b.params, b.k, b.beta, b.gate, None, None, lsum)
    torch.cuda.synchronize()
    ref = torch.log(ratio.clamp_min(1.1754944e-38)).reshape(2, 64, 1).sum(1)
    assert torch.allclose(lsum, ref, rtol=1e-5, atol=1e-4)
