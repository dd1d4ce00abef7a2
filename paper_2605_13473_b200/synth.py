"""Seeded synthetic inputs for the OSDN layer (no method arithmetic lives here).

The generators only draw random tensors with the value distributions of the
benchmark configurations: unit-norm q/k, standard-normal v, sigmoid-normal
beta, small negative log-gates.  They stand in for the language-model
activations the paper trains on, which are not available offline.  Both the
CPU oracle tests and the CUDA parity tests draw their inputs from here; the
module imports neither of them.

All tensors are CPU torch tensors in the packed layout ``[T_total, H, *]``
(a dense ``[B, T, H, *]`` batch is the same memory with
``cu_seqlens = [0, T, 2T, ...]``).  For bf16 configurations q, k, v and dout
are rounded to bf16-representable values and returned as float32, so that the
oracle (which widens to float64) and the GPU path (which narrows to bf16
without loss) see identical numbers.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional

import torch


@dataclass
class OsdnHyper:
    """Scalar settings of the layer (Section 3.2, Appendix D, Listing 1)."""

    eta: float = 0.003
    d_min: float = 0.5
    d_max: float = 2.0
    eps: float = 1e-6
    scale: float = 0.0  # <= 0 means K ** -0.5
    beta_aware: int = 1
    apf_mode: int = 1  # 0 none, 1 retention aliased to the gate, 2 separate log-retention, 3 one per coordinate
    clamp: int = 1
    chunk: int = 64
    channel_gate: int = 0  # 1: `gate` is [T, H, K], one log-gate per key channel (OSKDA extension)


@dataclass
class OsdnInputs:
    name: str
    H: int
    K: int
    V: int
    io_dtype: str  # "fp32" | "bf16"
    seq_lens: List[int]
    dense_B: int  # >0 when the batch is dense [B, T, H, *]; 0 for var-len
    hyper: OsdnHyper
    q: torch.Tensor
    k: torch.Tensor
    v: torch.Tensor
    beta: torch.Tensor
    gate: torch.Tensor
    log_ret: Optional[torch.Tensor] = None
    dout: Optional[torch.Tensor] = None
    init_state: Optional[torch.Tensor] = None
    precond_in: Optional[torch.Tensor] = None
    dfinal_state: Optional[torch.Tensor] = None
    dprecond_out: Optional[torch.Tensor] = None
    notes: dict = field(default_factory=dict)

    @property
    def T_total(self) -> int:
        return int(sum(self.seq_lens))

    @property
    def nseq(self) -> int:
        return len(self.seq_lens)

    @property
    def cu_seqlens(self) -> torch.Tensor:
        cu = [0]
        for L in self.seq_lens:
            cu.append(cu[-1] + int(L))
        return torch.tensor(cu, dtype=torch.int32)


def _round_io(x: torch.Tensor, io_dtype: str) -> torch.Tensor:
    if io_dtype == "bf16":
        return x.to(torch.bfloat16).to(torch.float32)
    return x.to(torch.float32)


def _unit_rows(x: torch.Tensor) -> torch.Tensor:
    return x / x.norm(dim=-1, keepdim=True).clamp_min(1e-12)


def draw(
    name: str,
    seed: int,
    seq_lens: List[int],
    H: int,
    K: int,
    V: int,
    io_dtype: str,
    *,
    dense_B: int = 0,
    hyper: Optional[OsdnHyper] = None,
    gate_kind: str = "softplus",  # softplus | mixture | strong | zero
    key_kind: str = "gauss",  # gauss | sparse | cyclic16 | raw
    beta_kind: str = "sigmoid",  # sigmoid | uniform39
    with_dout: bool = False,
    with_state: bool = False,
    with_log_ret: bool = False,
    with_state_cotangents: bool = False,
    log_ret_shift: float = 5.0,
) -> OsdnInputs:
    """Draw one input set.  Draw order: q, k, v, beta, gate, then optionals."""
    hyper = hyper or OsdnHyper()
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    T = int(sum(seq_lens))
    nseq = len(seq_lens)

    def randn(*shape):
        return torch.randn(*shape, generator=gen, dtype=torch.float32)

    def rand(*shape):
        return torch.rand(*shape, generator=gen, dtype=torch.float32)

    q = _unit_rows(randn(T, H, K))
    kraw = randn(T, H, K)
    if key_kind == "gauss":
        k = _unit_rows(kraw)
    elif key_kind == "raw":  # un-normalised keys (exercise the 1/n_t normaliser)
        k = kraw * 0.2
    elif key_kind == "sparse":  # 10 % support per key, then unit norm
        mask = (rand(T, H, K) < 0.10).to(torch.float32)
        # guarantee at least one active coordinate per key
        first = torch.zeros(T, H, K)
        idx = torch.randint(0, K, (T, H, 1), generator=gen)
        first.scatter_(-1, idx, 1.0)
        k = _unit_rows(kraw * torch.clamp(mask + first, max=1.0))
    elif key_kind == "cyclic16":  # 16 distinct unit keys per head repeated cyclically
        base = _unit_rows(randn(16, H, K))
        reps = (T + 15) // 16
        k = base.repeat(reps, 1, 1)[:T].contiguous()
    else:
        raise ValueError(key_kind)
    v = randn(T, H, V)
    if beta_kind == "sigmoid":
        beta = torch.sigmoid(randn(T, H))
    elif beta_kind == "uniform39":
        beta = 0.3 + 0.6 * rand(T, H)
    else:
        raise ValueError(beta_kind)
    if gate_kind == "softplus":
        gate = -0.1 * torch.nn.functional.softplus(randn(T, H))
    elif gate_kind == "mixture":  # 90 % near zero, 10 % strong decay in [-3, -1]
        near = -0.005 * randn(T, H).abs()
        strong = -3.0 + 2.0 * rand(T, H)
        pick = rand(T, H) < 0.10
        gate = torch.where(pick, strong, near)
    elif gate_kind == "strong":
        gate = -3.0 + 2.0 * rand(T, H)
    elif gate_kind == "zero":
        gate = torch.zeros(T, H)
    else:
        raise ValueError(gate_kind)

    if hyper.channel_gate:
        # one log-gate per key channel: the token's gate spread over the channels by a factor in [0.25, 1.75]
        gate = gate.unsqueeze(-1) * (0.25 + 1.5 * rand(T, H, K))

    out = OsdnInputs(
        name=name, H=H, K=K, V=V, io_dtype=io_dtype, seq_lens=[int(x) for x in seq_lens],
        dense_B=dense_B, hyper=hyper,
        q=_round_io(q, io_dtype), k=_round_io(k, io_dtype), v=_round_io(v, io_dtype),
        beta=beta.contiguous(), gate=gate.contiguous(),
    )
    if with_dout:
        out.dout = _round_io(randn(T, H, V), io_dtype)
    if with_log_ret:
        # one log-retention per (token, head); per coordinate for the vector-retention mode
        shape = (T, H, K) if hyper.apf_mode == 3 else (T, H)
        out.log_ret = torch.nn.functional.logsigmoid(randn(*shape) + log_ret_shift).contiguous()
    if with_state:
        out.init_state = 0.5 * randn(nseq, H, V, K)
        out.precond_in = hyper.d_min + (hyper.d_max - hyper.d_min) * rand(nseq, H, K)
    if with_state_cotangents:
        out.dfinal_state = 0.1 * randn(nseq, H, V, K)
        out.dprecond_out = randn(nseq, H, K)
    return out


def varlen_lengths(seed: int = 4, nseq: int = 8, lo: int = 512, hi: int = 32768,
                   total: int = 131072) -> List[int]:
    """Log-uniform lengths in [lo, hi], rescaled so that they sum to ``total``.

    The raw draws are scaled by total / sum, clipped back into [lo, hi], and the
    last sequence absorbs the remainder.  Lengths are deliberately not rounded
    to multiples of the chunk size: ragged tails are part of the workload.
    """
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    u = torch.rand(nseq, generator=gen, dtype=torch.float64)
    raw = torch.exp(math.log(lo) + u * (math.log(hi) - math.log(lo)))
    scaled = raw * (total / raw.sum())
    lens = [int(min(max(round(float(x)), lo), hi)) for x in scaled]
    rest = total - sum(lens[:-1])
    # keep the last one inside the range by shaving the longest others if needed
    while rest > hi:
        j = min(range(nseq - 1), key=lambda i: lens[i])
        add = min(hi - lens[j], rest - hi)
        if add <= 0:
            break
        lens[j] += add
        rest -= add
    while rest < lo:
        j = max(range(nseq - 1), key=lambda i: lens[i])
        sub = min(lens[j] - lo, lo - rest)
        if sub <= 0:
            break
        lens[j] -= sub
        rest += sub
    lens[-1] = rest
    return lens


def config(idx: int, *, shrink: Optional[dict] = None) -> OsdnInputs:
    """The five benchmark configurations (index 0..4).

    ``shrink`` may override B / T / H / total for reduced parity-test versions
    that keep the distributions but finish on the CPU oracle in seconds.
    """
    s = shrink or {}
    if idx == 0:
        B, T, H, D = s.get("B", 1), s.get("T", 256), s.get("H", 1), s.get("D", 64)
        return draw("cfg0_tiny_fwd_fp32", 0, [T] * B, H, D, D, "fp32", dense_B=B)
    if idx in (1, 2):
        B, T, H = s.get("B", 8), s.get("T", 2048), s.get("H", 8)
        return draw("cfg1_340m_fwd" if idx == 1 else "cfg2_340m_train", idx, [T] * B, H, 128, 128,
                    "bf16", dense_B=B, with_dout=(idx == 2))
    if idx == 3:
        B, T, H = s.get("B", 4), s.get("T", 4096), s.get("H", 16)
        return draw("cfg3_1p3b_train", 3, [T] * B, H, 128, 128, "bf16", dense_B=B,
                    gate_kind="mixture", with_dout=True)
    if idx == 4:
        lens = varlen_lengths(4, s.get("nseq", 8), s.get("lo", 512), s.get("hi", 32768),
                              s.get("total", 131072))
        return draw("cfg4_varlen_train", 4, lens, s.get("H", 8), 128, 128, "bf16",
                    gate_kind="softplus", with_dout=True)
    raise ValueError(idx)


def lively(idx: int, *, T: int = 200, B: int = 2, H: int = 2, D: int = 128,
           io_dtype: str = "bf16") -> OsdnInputs:
    """Input sets on which the preconditioner really moves (the benchmark
    distributions pin it to the lower bound after a few tokens)."""
    lens = [T] * B
    if idx == 1:  # large step, separate retention near one, sparse keys
        hy = OsdnHyper(eta=0.3, apf_mode=2)
        return draw("lively1_sparse_ret", 101, lens, H, D, D, io_dtype, dense_B=B, hyper=hy,
                    key_kind="sparse", with_dout=True, with_log_ret=True, with_state=True,
                    with_state_cotangents=True)
    if idx == 2:  # repeated keys climb toward 1/beta and reach the upper bound
        hy = OsdnHyper(eta=0.3, apf_mode=0)
        return draw("lively2_cyclic", 102, lens, H, D, D, io_dtype, dense_B=B, hyper=hy,
                    key_kind="cyclic16", beta_kind="uniform39", with_dout=True,
                    with_state_cotangents=True)
    if idx == 3:  # projection switched off
        hy = OsdnHyper(eta=0.05, apf_mode=1, clamp=0)
        return draw("lively3_noclamp", 103, lens, H, D, D, io_dtype, dense_B=B, hyper=hy,
                    with_dout=True, with_state=True)
    if idx == 4:  # strong decay on every token: in-chunk gate products underflow
        hy = OsdnHyper(eta=0.1, apf_mode=0)
        return draw("lively4_strong_decay", 104, lens, H, D, D, io_dtype, dense_B=B, hyper=hy,
                    gate_kind="strong", with_dout=True, with_state=True)
    if idx == 5:  # un-normalised keys, non-beta-aware step
        hy = OsdnHyper(eta=0.2, apf_mode=2, beta_aware=0)
        return draw("lively5_rawkeys", 105, lens, H, D, D, io_dtype, dense_B=B, hyper=hy,
                    key_kind="raw", with_dout=True, with_log_ret=True)
    if idx == 6:  # the ungated 1.3B OSDN setting: g = 0, separate retention near 0.999, non-beta-aware step
        hy = OsdnHyper(eta=0.003, apf_mode=2, beta_aware=0)
        return draw("lively6_ungated_osdn", 106, lens, H, D, D, io_dtype, dense_B=B, hyper=hy,
                    gate_kind="zero", with_dout=True, with_log_ret=True, log_ret_shift=7.0)
    if idx == 7:  # vector retention: one log-retention per coordinate
        hy = OsdnHyper(eta=0.3, apf_mode=3)
        return draw("lively7_vector_ret", 107, lens, H, D, D, io_dtype, dense_B=B, hyper=hy,
                    key_kind="sparse", with_dout=True, with_log_ret=True, with_state=True,
                    with_state_cotangents=True, log_ret_shift=3.0)
    raise ValueError(idx)
