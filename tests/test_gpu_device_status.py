"""The device-side error path: errors that only the GPU can see are reported through the status word
at the head of the workspace, and every device-side wait is bounded."""
import pytest
import torch

from paper_2605_13473_b200 import binding
from paper_2605_13473_b200.synth import OsdnHyper, draw

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_bounded_wait_runs_out_and_reports():
    """A wait on a barrier nothing arrives on: the kernel gives up after about a millisecond, leaves
    its code in the status word and returns; the context stays usable."""
    ws = torch.zeros(256, dtype=torch.uint8, device=DEV)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    binding.osdn_selftest_wait_timeout(ws, 1000)
    e1.record()
    torch.cuda.synchronize()
    assert binding.osdn_read_device_status(ws) == 199
    assert 0.2 <= e0.elapsed_time(e1) <= 50.0      # about 1 ms (the bound is counted in clock cycles)
    # the device still works, and a later call clears the word again
    assert float((torch.ones(8, device=DEV) * 2).sum()) == 16.0
    inp = draw("after_timeout", 5, [70], 1, 128, 128, "bf16", dense_B=1, hyper=OsdnHyper())
    b = binding.DeviceBundle(inp, DEV, need_bwd=False)
    b.fwd()
    torch.cuda.synchronize()
    assert b.device_status() == 0


@pytest.mark.parametrize("cu", [[0, 70, 60, 200], [5, 70, 130, 200], [0, 70, 130, 190]],
                         ids=["decreasing", "first_not_zero", "last_not_T"])
def test_malformed_cu_seqlens_is_reported_not_followed(cu):
    """The offsets live on the device, so only the device can check them: a broken contract leaves a
    code in the status word, and because every sequence is clamped into the packed token range no
    access leaves the user tensors."""
    hy = OsdnHyper(eta=0.3, apf_mode=1)
    inp = draw("bad_cu", 31, [70, 60, 70], 2, 128, 128, "bf16", hyper=hy)
    b = binding.DeviceBundle(inp, DEV, need_bwd=False)
    b.cu.copy_(torch.tensor(cu, dtype=torch.int32))
    b.fwd()
    torch.cuda.synchronize()
    assert b.device_status() == 120
    good = binding.DeviceBundle(inp, DEV, need_bwd=False)
    good.fwd()
    torch.cuda.synchronize()
    assert good.device_status() == 0
