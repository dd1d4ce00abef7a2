"""Full-size benchmark configurations on the GPU, checked against the oracle on sampled
chains (every (sequence, head) chain is independent, so the oracle is run on a subset of them,
element by element)."""
import pytest

import parity
from paper_2605_13473_b200 import run_inputs_bwd, run_inputs_fwd
from paper_2605_13473_b200.synth import config

pytestmark = pytest.mark.gpu

REPORT = {}


def teardown_module(module):
    parity.write_report(REPORT, suffix="_fullsize")


def _sampled(inp, bwd, seqs, heads, label):
    got = run_inputs_bwd(inp) if bwd else run_inputs_fwd(inp)
    sub, tok_t, hd = parity.subset(inp, seqs, heads)
    got_sub = parity.subset_result(got, seqs, heads, tok_t, hd)
    ref = parity.oracle_all(sub, bwd, got_sub.get("projection_masks"))
    keys = parity.FWD_KEYS + (parity.BWD_KEYS if bwd else ())
    parity.compare(got_sub, ref, inp.io_dtype, keys, label, report=REPORT, tensor_core=True)


def test_cfg1_full_forward():
    _sampled(config(1), False, [0, 5], [0, 3, 7], "cfg1_full")


def test_cfg2_full_train_step():
    _sampled(config(2), True, [1, 7], [2, 6], "cfg2_full")


def test_cfg3_full_train_step():
    _sampled(config(3), True, [0, 3], [1, 15], "cfg3_full")


def test_cfg4_full_varlen_train_step():
    inp = config(4)
    order = sorted(range(len(inp.seq_lens)), key=lambda i: inp.seq_lens[i])
    _sampled(inp, True, [order[0], order[len(order) // 2]], [0, 7], "cfg4_full_short_mid")
    _sampled(inp, True, [order[-1]], [4], "cfg4_full_longest")
