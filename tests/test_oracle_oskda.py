"""Pins of the oracle's channel-gate mode (OSKDA, backbone-extension appendix "Kimi Delta Attention with
Online Scaling") against things that are not the oracle: the scalar-gate oracle, the paper's K x V
left-multiplied recurrence and its chunk equations written out in numpy, and finite differences."""
import numpy as np
import pytest

import oracle
from paper_2605_13473_b200.synth import OsdnHyper, draw


def _inputs(seed, T=70, H=2, K=8, V=6, apf_mode=2, seq_lens=None, **kw):
    hy = OsdnHyper(eta=0.3, apf_mode=apf_mode, channel_gate=1)
    lens = seq_lens or [T]
    return draw("oskda", seed, lens, H, K, V, "fp32", hyper=hy, with_log_ret=apf_mode >= 2, with_state=True,
                with_dout=True, with_state_cotangents=True, gate_kind="strong", log_ret_shift=2.0, **kw)


def _phase1_numpy(inp):
    """d_t and write keys, token by token (Algorithm 1 with the beta-aware step)."""
    hy = inp.hyper
    k = inp.k.double().numpy()
    beta = inp.beta.double().numpy()
    T, H, K = k.shape
    assert inp.nseq == 1
    d = inp.precond_in.double().numpy()[0].copy()
    ktil = np.zeros_like(k)
    for t in range(T):
        for h in range(H):
            kap = k[t, h] ** 2
            ktil[t, h] = d[h] * k[t, h]
            n = max(kap.sum(), hy.eps)
            b = beta[t, h] if hy.beta_aware else 1.0
            c = hy.eta * b * (1.0 - b * (d[h] @ kap)) / n
            if hy.apf_mode == 0:
                r = 1.0
            elif hy.apf_mode == 2:
                r = np.exp(inp.log_ret.double().numpy()[t, h])
            else:
                r = np.exp(inp.log_ret.double().numpy()[t, h])
            d[h] = np.clip(r * d[h] + c * kap, hy.d_min, hy.d_max)
    return ktil, d


def test_equal_channel_gates_are_the_scalar_gate():
    inp = _inputs(11, apf_mode=2)
    g = inp.gate[..., 0].contiguous()
    inp.gate = g.unsqueeze(-1).expand(-1, -1, inp.K).contiguous()
    got = oracle.fwd_inputs(inp)
    gb = oracle.bwd_inputs(inp)
    hy = OsdnHyper(eta=0.3, apf_mode=2, channel_gate=0)
    ref = oracle.fwd(hy, inp.seq_lens, inp.q, inp.k, inp.v, inp.beta, g, inp.log_ret, inp.init_state, inp.precond_in)
    rb = oracle.bwd(hy, inp.seq_lens, inp.q, inp.k, inp.v, inp.beta, g, inp.dout, inp.log_ret, inp.init_state,
                    inp.precond_in, inp.dfinal_state, inp.dprecond_out)
    for name in ("out", "final_state", "precond_out"):
        np.testing.assert_allclose(got[name], ref[name], rtol=1e-12, atol=1e-13)
    for name in ("dq", "dk", "dv", "dbeta", "dlog_ret", "dinit_state", "dprecond_in"):
        np.testing.assert_allclose(gb[name], rb[name], rtol=1e-11, atol=1e-12)
    # a scalar gate is the sum of its channels' gradients
    np.testing.assert_allclose(gb["dgate"].sum(-1), rb["dgate"], rtol=1e-11, atol=1e-12)


@pytest.mark.parametrize("apf_mode", [0, 2, 3])
def test_left_multiplied_k_by_v_recurrence(apf_mode):
    """S'_t = (I - beta ktil k^T) Diag(alpha_t) S'_{t-1} + beta ktil v^T, o_t = S'_t^T q_t, with S' = S^T."""
    inp = _inputs(12 + apf_mode, apf_mode=apf_mode)
    got = oracle.fwd_inputs(inp)
    ktil, d_end = _phase1_numpy(inp)
    q, k, v = (x.double().numpy() for x in (inp.q, inp.k, inp.v))
    beta, gate = inp.beta.double().numpy(), inp.gate.double().numpy()
    T, H, K = k.shape
    scale = K ** -0.5
    for h in range(H):
        Sp = inp.init_state.double().numpy()[0, h].T.copy()   # K x V
        for t in range(T):
            A = np.eye(K) - beta[t, h] * np.outer(ktil[t, h], k[t, h])
            Sp = A @ (np.exp(gate[t, h])[:, None] * Sp) + beta[t, h] * np.outer(ktil[t, h], v[t, h])
            np.testing.assert_allclose(got["out"][t, h], scale * Sp.T @ q[t, h], rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(got["final_state"][0, h], Sp.T, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(got["precond_out"][0], d_end, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("C,T", [(16, 64), (16, 53), (8, 70)])
def test_chunk_equations_with_channel_decays(C, T):
    """The chunk form: cumulative channel decays Gamma_i, decayed keys, the unit-triangular system, the
    state advance with the suffix-gated write key, outputs from the inter- and intra-chunk parts."""
    inp = _inputs(20 + C + T, T=T, apf_mode=2)
    got = oracle.fwd_inputs(inp)
    ktil, _ = _phase1_numpy(inp)
    q, k, v = (x.double().numpy() for x in (inp.q, inp.k, inp.v))
    beta, gate = inp.beta.double().numpy(), inp.gate.double().numpy()
    H, K, V = inp.H, inp.K, inp.V
    scale = K ** -0.5
    for h in range(H):
        S = inp.init_state.double().numpy()[0, h].T.copy()   # K x V
        for c0 in range(0, T, C):
            c1 = min(c0 + C, T)
            L = c1 - c0
            G = np.cumsum(gate[c0:c1, h], axis=0)             # [L, K] log of Gamma_i
            Kd = k[c0:c1, h] * np.exp(G)                      # Gamma_i (.) k_i : reads the chunk-start state
            Kw = ktil[c0:c1, h] * np.exp(-G)                  # ktil_j / Gamma_j
            Qd = q[c0:c1, h] * np.exp(G)
            b = beta[c0:c1, h]
            A_kk = np.tril(Kd @ Kw.T, -1)                     # <Gamma_i/Gamma_j k_i, ktil_j>, j < i
            A_qk = np.tril(Qd @ Kw.T, 0)
            M = np.eye(L) + A_kk * b[None, :]
            # u_i = v_i - k_i^T S_{i-1}; unrolling the in-chunk writes gives M U = V - Kd S
            U = np.linalg.solve(M, v[c0:c1, h] - Kd @ S)
            O = Qd @ S + A_qk @ (b[:, None] * U)
            np.testing.assert_allclose(got["out"][c0:c1, h], scale * O, rtol=1e-9, atol=1e-11)
            GC = G[-1]                                        # log gamma^C
            Ksuf = ktil[c0:c1, h] * np.exp(GC[None, :] - G)   # Gamma^{i->C} (.) ktil_i
            S = np.exp(GC)[:, None] * S + Ksuf.T @ (b[:, None] * U)
        np.testing.assert_allclose(got["final_state"][0, h], S.T, rtol=1e-9, atol=1e-11)


def test_no_write_and_no_gate_special_cases():
    inp = _inputs(31, apf_mode=0)
    inp.beta = inp.beta * 0.0
    got = oracle.fwd_inputs(inp)
    gate = inp.gate.double().numpy()
    S0 = inp.init_state.double().numpy()[0]
    # beta == 0: the state only decays, channel by channel
    expect = S0 * np.exp(gate.sum(0))[:, None, :]
    np.testing.assert_allclose(got["final_state"][0], expect, rtol=1e-12)
    np.testing.assert_allclose(got["precond_out"][0], inp.precond_in.double().numpy()[0], rtol=0, atol=0)
    # zero log-gates: the ungated online-scaled delta rule
    inp2 = _inputs(32, apf_mode=2)
    inp2.gate = inp2.gate * 0.0
    hy = OsdnHyper(eta=0.3, apf_mode=2, channel_gate=0)
    ref = oracle.fwd(hy, inp2.seq_lens, inp2.q, inp2.k, inp2.v, inp2.beta, inp2.gate[..., 0].contiguous(),
                     inp2.log_ret, inp2.init_state, inp2.precond_in)
    got2 = oracle.fwd_inputs(inp2)
    np.testing.assert_allclose(got2["out"], ref["out"], rtol=1e-12, atol=1e-13)


def test_split_sequence_carry():
    inp = _inputs(41, T=90)
    whole = oracle.fwd_inputs(inp)
    cut = 37
    a = oracle.fwd(inp.hyper, [cut], inp.q[:cut], inp.k[:cut], inp.v[:cut], inp.beta[:cut], inp.gate[:cut],
                   inp.log_ret[:cut], inp.init_state, inp.precond_in)
    b = oracle.fwd(inp.hyper, [90 - cut], inp.q[cut:], inp.k[cut:], inp.v[cut:], inp.beta[cut:], inp.gate[cut:],
                   inp.log_ret[cut:], a["final_state"], a["precond_out"])
    np.testing.assert_allclose(np.concatenate([a["out"], b["out"]]), whole["out"], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(b["final_state"], whole["final_state"], rtol=1e-12, atol=1e-13)


def test_gradients_by_central_differences():
    inp = _inputs(51, T=24, H=1, K=5, V=4, apf_mode=2)
    inp.hyper.clamp = 0   # smooth everywhere: the projection has its own pins
    g = oracle.bwd_inputs(inp)
    dout = inp.dout.double().numpy()
    dS, dd = inp.dfinal_state.double().numpy(), inp.dprecond_out.double().numpy()

    def loss(**over):
        args = dict(q=inp.q.double().numpy(), k=inp.k.double().numpy(), v=inp.v.double().numpy(),
                    beta=inp.beta.double().numpy(), gate=inp.gate.double().numpy(),
                    log_ret=inp.log_ret.double().numpy(), init_state=inp.init_state.double().numpy(),
                    precond_in=inp.precond_in.double().numpy())
        args.update(over)
        r = oracle.fwd(inp.hyper, inp.seq_lens, **args)
        return (r["out"] * dout).sum() + (r["final_state"] * dS).sum() + (r["precond_out"] * dd).sum()

    rng = np.random.default_rng(0)
    names = dict(q="dq", k="dk", v="dv", beta="dbeta", gate="dgate", log_ret="dlog_ret", init_state="dinit_state",
                 precond_in="dprecond_in")
    for arg, gname in names.items():
        base = getattr(inp, arg).double().numpy()
        for _ in range(6):
            idx = tuple(rng.integers(0, n) for n in base.shape)
            eps = 1e-6
            hi, lo = base.copy(), base.copy()
            hi[idx] += eps
            lo[idx] -= eps
            fd = (loss(**{arg: hi}) - loss(**{arg: lo})) / (2 * eps)
            assert abs(fd - g[gname][idx]) <= 1e-6 * max(1.0, abs(fd)), (arg, idx, fd, g[gname][idx])
