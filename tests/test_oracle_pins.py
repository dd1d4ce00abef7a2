"""Pins of the fp64 oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA library.  Each pin is chosen so that a
plausible mistake in the oracle (wrong key on the read or write side, gate
applied after the read, update order in phase 1, dropped term or wrong sign in
the adjoint) fails at least one of them.
"""
import os

import numpy as np
import pytest

import oracle
import chunkwise_np as cw
from paper_2605_13473_b200.synth import OsdnHyper, draw

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rng(seed):
    return np.random.default_rng(seed)


def _unit(x):
    return x / np.linalg.norm(x, axis=-1, keepdims=True)


def _small(seed, L=12, H=2, K=6, V=5, unit=True, gate=True):
    r = _rng(seed)
    q = _unit(r.standard_normal((L, H, K)))
    k = r.standard_normal((L, H, K))
    k = _unit(k) if unit else 0.4 * k
    v = r.standard_normal((L, H, V))
    beta = 1.0 / (1.0 + np.exp(-r.standard_normal((L, H))))
    g = -0.3 * np.abs(r.standard_normal((L, H))) if gate else np.zeros((L, H))
    return q, k, v, beta, g


# ---------------------------------------------------------------- P1 / P2
def test_lemma1_residual_identity_and_descent_ratio():
    """After every write S_t k_t - v_t = -(1 - beta <d_t,k_t^2>)(v_t - exp(g_t) S_{t-1} k_t)
    (proof of Lemma 1, post-gate form), hence the loss ratio is (1 - beta<d,k^2>)^2 in (0,1)
    for unit keys and d inside the box (monotone-descent corollary)."""
    hy = OsdnHyper(eta=0.3, apf_mode=1)
    L, H, K, V = 14, 2, 6, 5
    q, k, v, beta, g = _small(1, L, H, K, V)
    full = oracle.fwd(hy, [L], q, k, v, beta, g, want_dtraj=True)
    dtr = full["d_traj"]
    S_prev = np.zeros((1, H, V, K))
    for t in range(L):
        S_t = oracle.fwd(hy, [t + 1], q[:t + 1], k[:t + 1], v[:t + 1], beta[:t + 1], g[:t + 1])["final_state"]
        for h in range(H):
            e = v[t, h] - np.exp(g[t, h]) * S_prev[0, h] @ k[t, h]
            lhs = S_t[0, h] @ k[t, h] - v[t, h]
            fac = 1.0 - beta[t, h] * float(dtr[t, h] @ (k[t, h] ** 2))
            np.testing.assert_allclose(lhs, -fac * e, rtol=0, atol=1e-13)
            ratio = np.sum(lhs ** 2) / np.sum(e ** 2)
            assert 0.0 < ratio < 1.0
            np.testing.assert_allclose(ratio, fac ** 2, rtol=1e-10)
        S_prev = S_t
    # d never leaves the box and does move on this input
    assert dtr.min() >= hy.d_min - 1e-15 and dtr.max() <= hy.d_max + 1e-15
    assert np.abs(dtr[-1] - 1.0).max() > 1e-2


# ---------------------------------------------------------------- P3
def _textbook_gated_delta(q, k, v, beta, g, scale):
    """S_t = S_{t-1} alpha_t (I - beta k k^T) + beta v k^T ; o_t = scale S_t q_t."""
    L, K = k.shape
    V = v.shape[1]
    S = np.zeros((V, K))
    o = np.zeros((L, V))
    for t in range(L):
        S = np.exp(g[t]) * S @ (np.eye(K) - beta[t] * np.outer(k[t], k[t])) + beta[t] * np.outer(v[t], k[t])
        o[t] = scale * S @ q[t]
    return o, S


@pytest.mark.parametrize("gated", [True, False])
def test_reduces_to_gated_delta_rule_when_preconditioner_is_one(gated):
    hy = OsdnHyper(eta=0.0, apf_mode=0)
    L, H, K, V = 20, 2, 8, 4
    q, k, v, beta, g = _small(2, L, H, K, V, unit=False, gate=gated)
    res = oracle.fwd(hy, [L], q, k, v, beta, g)
    for h in range(H):
        o, S = _textbook_gated_delta(q[:, h], k[:, h], v[:, h], beta[:, h], g[:, h], K ** -0.5)
        np.testing.assert_allclose(res["out"][:, h], o, atol=1e-12)
        np.testing.assert_allclose(res["final_state"][0, h], S, atol=1e-12)
    np.testing.assert_allclose(res["precond_out"], 1.0, atol=0)
    # same thing through a degenerate box
    hy2 = OsdnHyper(eta=0.3, apf_mode=1, d_min=1.0, d_max=1.0)
    res2 = oracle.fwd(hy2, [L], q, k, v, beta, g)
    np.testing.assert_allclose(res2["out"], res["out"], atol=1e-12)


# ---------------------------------------------------------------- P4
def test_beta_zero_leaves_state_unwritten():
    hy = OsdnHyper(eta=0.3, apf_mode=1)
    L, H, K, V = 9, 1, 5, 4
    q, k, v, beta, g = _small(3, L, H, K, V)
    beta[:] = 0.0
    r = _rng(30)
    S0 = r.standard_normal((1, H, V, K))
    d0 = 0.5 + 1.5 * r.random((1, H, K))
    res = oracle.fwd(hy, [L], q, k, v, beta, g, init_state=S0, precond_in=d0)
    G = np.cumsum(g[:, 0])
    np.testing.assert_allclose(res["final_state"][0, 0], np.exp(G[-1]) * S0[0, 0], atol=1e-14)
    for t in range(L):
        np.testing.assert_allclose(res["out"][t, 0], K ** -0.5 * np.exp(G[t]) * S0[0, 0] @ q[t, 0], atol=1e-14)
    d = d0[0, 0].copy()
    for t in range(L):
        d = np.clip(np.exp(g[t, 0]) * d, hy.d_min, hy.d_max)
    np.testing.assert_allclose(res["precond_out"][0, 0], d, atol=1e-15)


# ---------------------------------------------------------------- P5
def test_orthonormal_keys_unit_step_overwrite():
    hy = OsdnHyper(eta=0.0, apf_mode=0)
    K, V = 7, 4
    r = _rng(4)
    Qm, _ = np.linalg.qr(r.standard_normal((K, K)))
    k = Qm[:, None, :]                     # K orthonormal keys, H = 1
    v = r.standard_normal((K, 1, V))
    q = k.copy()
    beta = np.ones((K, 1)); g = np.zeros((K, 1))
    res = oracle.fwd(hy, [K], q, k, v, beta, g)
    S = res["final_state"][0, 0]
    for i in range(K):
        np.testing.assert_allclose(S @ k[i, 0], v[i, 0], atol=1e-13)


# ---------------------------------------------------------------- P6 (golden)
def test_onehot_key_closed_form_golden():
    rows = [l for l in open(os.path.join(GOLD, "onehot_precond.txt")) if not l.startswith("#")]
    assert len(rows) == 3
    for line in rows:
        head, vals = line.split(":")
        name, eta, beta, r, dmin, dmax, d0 = head.split()
        eta, beta, r, dmin, dmax, d0 = map(float, (eta, beta, r, dmin, dmax, d0))
        vals = np.array([float(x) for x in vals.split()])
        n = len(vals) - 1
        K = 4
        k = np.zeros((n, 1, K)); k[:, 0, 0] = 1.0
        hy = OsdnHyper(eta=eta, d_min=dmin, d_max=dmax, apf_mode=2)
        lr = np.full((n, 1), np.log(r))
        din = np.full((1, 1, K), d0)
        res = oracle.fwd(hy, [n], k.copy(), k, np.zeros((n, 1, 2)), np.full((n, 1), beta),
                         np.zeros((n, 1)), log_ret=lr, precond_in=din, want_dtraj=True)
        np.testing.assert_allclose(res["d_traj"][:, 0, 0], vals[:-1], rtol=1e-13)
        np.testing.assert_allclose(res["precond_out"][0, 0, 0], vals[-1], rtol=1e-13)
        # other coordinates only see the retention and the box
        other = d0
        for _ in range(n):
            other = min(max(r * other, dmin), dmax)
        np.testing.assert_allclose(res["precond_out"][0, 0, 1:], other, rtol=1e-13)
        pu = oracle.precond_update(hy, [n], k, np.full((n, 1), beta), log_ret=lr, precond_in=din)
        np.testing.assert_allclose(pu["precond_out"], res["precond_out"], atol=0)
    # fixed point beta * d = 1 for r = 1 (first golden row converges towards 1 / 0.8)
    first = np.array([float(x) for x in rows[0].split(":")[1].split()])
    assert abs(first[-1] - 1.25) < 1e-3 and np.all(np.diff(first) > 0)


# ---------------------------------------------------------------- P7 (golden)
def test_alternating_scalar_example_golden():
    rows = [l.split() for l in open(os.path.join(GOLD, "alternating_k1.txt")) if not l.startswith("#")]
    n = len(rows)
    vt = np.array([float(r[1]) for r in rows]).reshape(n, 1, 1)
    St = np.array([float(r[2]) for r in rows])
    hy = OsdnHyper(eta=0.0, apf_mode=0, scale=1.0)
    one = np.ones((n, 1, 1))
    res = oracle.fwd(hy, [n], one, one, vt, np.full((n, 1), 0.5), np.zeros((n, 1)),
                     precond_in=np.full((1, 1, 1), 2.0))
    np.testing.assert_allclose(res["out"][:, 0, 0], St, atol=1e-15)   # o_t = S_t * 1


# ---------------------------------------------------------------- P8
def test_wy_product_identity():
    r = _rng(8)
    C, K = 9, 6
    k = r.standard_normal((C, K)); kt = k * (0.5 + 1.5 * r.random((C, K)))
    beta = r.random(C)
    prod, wy = cw.wy_product(k, kt, beta)
    np.testing.assert_allclose(prod, wy, atol=1e-12)


@pytest.mark.parametrize("C", [4, 64])
@pytest.mark.parametrize("L", [1, 2, 63, 64, 65, 130])
def test_chunkwise_form_equals_recurrence(L, C):
    hy = OsdnHyper(eta=0.3, apf_mode=1)
    H, K, V = 2, 8, 6
    q, k, v, beta, g = _small(80 + L, L, H, K, V)
    r = _rng(81)
    S0 = r.standard_normal((1, H, V, K)); d0 = 0.5 + 1.5 * r.random((1, H, K))
    a = oracle.fwd(hy, [L], q, k, v, beta, g, init_state=S0, precond_in=d0)
    b = cw.layer_fwd(hy, [L], q, k, v, beta, g, init_state=S0, precond_in=d0, C=C)
    for key in ("out", "final_state", "precond_out"):
        np.testing.assert_allclose(a[key], b[key], atol=1e-10, rtol=0)


def test_chunkwise_form_strong_decay_no_division():
    """In-chunk gate products underflow below 1e-6; the recurrence has no such guard."""
    hy = OsdnHyper(eta=0.1, apf_mode=0)
    L, H, K, V = 130, 1, 8, 4
    q, k, v, beta, g = _small(82, L, H, K, V)
    g[:] = -1.0 - 2.0 * _rng(83).random(g.shape)
    a = oracle.fwd(hy, [L], q, k, v, beta, g)
    b = cw.layer_fwd(hy, [L], q, k, v, beta, g)
    np.testing.assert_allclose(a["out"], b["out"], atol=1e-11)
    np.testing.assert_allclose(a["final_state"], b["final_state"], atol=1e-11)


# ---------------------------------------------------------------- P9
def test_apf_with_unit_retention_is_plain_update():
    L, H, K, V = 30, 2, 8, 4
    q, k, v, beta, g = _small(9, L, H, K, V)
    a = oracle.fwd(OsdnHyper(eta=0.3, apf_mode=0), [L], q, k, v, beta, g)
    b = oracle.fwd(OsdnHyper(eta=0.3, apf_mode=2), [L], q, k, v, beta, g, log_ret=np.zeros((L, H)))
    for key in a:
        np.testing.assert_allclose(a[key], b[key], atol=0)
    # aliased retention is mode 2 fed with the gate
    c = oracle.fwd(OsdnHyper(eta=0.3, apf_mode=1), [L], q, k, v, beta, g)
    d = oracle.fwd(OsdnHyper(eta=0.3, apf_mode=2), [L], q, k, v, beta, g, log_ret=g)
    for key in c:
        np.testing.assert_allclose(c[key], d[key], atol=0)
    assert np.abs(a["precond_out"] - c["precond_out"]).max() > 1e-3


# ---------------------------------------------------------------- P10
def test_split_sequence_carry_and_varlen():
    hy = OsdnHyper(eta=0.3, apf_mode=1)
    H, K, V = 2, 8, 4
    lens = [37, 5, 70]
    L = sum(lens)
    q, k, v, beta, g = _small(10, L, H, K, V)
    packed = oracle.fwd(hy, lens, q, k, v, beta, g)
    off = 0
    for s, n in enumerate(lens):
        sl = slice(off, off + n)
        one = oracle.fwd(hy, [n], q[sl], k[sl], v[sl], beta[sl], g[sl])
        np.testing.assert_allclose(packed["out"][sl], one["out"], atol=0)
        np.testing.assert_allclose(packed["final_state"][s], one["final_state"][0], atol=0)
        np.testing.assert_allclose(packed["precond_out"][s], one["precond_out"][0], atol=0)
        off += n
    # carry (S, d) across a split
    n1 = 41
    full = oracle.fwd(hy, [L], q, k, v, beta, g)
    a = oracle.fwd(hy, [n1], q[:n1], k[:n1], v[:n1], beta[:n1], g[:n1])
    b = oracle.fwd(hy, [L - n1], q[n1:], k[n1:], v[n1:], beta[n1:], g[n1:],
                   init_state=a["final_state"], precond_in=a["precond_out"])
    np.testing.assert_allclose(np.concatenate([a["out"], b["out"]]), full["out"], atol=1e-14)
    np.testing.assert_allclose(b["final_state"], full["final_state"], atol=1e-14)
    np.testing.assert_allclose(b["precond_out"], full["precond_out"], atol=0)


def test_phase1_order_write_key_uses_pre_update_d():
    """Algorithm 1: the write key of token t is d_t (.) k_t with d_t BEFORE the step."""
    hy = OsdnHyper(eta=0.4, apf_mode=0)
    L, H, K, V = 6, 1, 5, 3
    q, k, v, beta, g = _small(11, L, H, K, V)
    res = oracle.fwd(hy, [L], q, k, v, beta, g, want_ktil=True, want_dtraj=True)
    np.testing.assert_allclose(res["d_traj"][0], 1.0, atol=0)
    np.testing.assert_allclose(res["ktil"][0], k[0], atol=0)            # d_1 = ones
    np.testing.assert_allclose(res["ktil"], res["d_traj"] * k, atol=0)
    # the step itself, written out for token 1 (Eq. dt_update with beta-aware feedback)
    kap = k[0, 0] ** 2
    d2 = 1.0 + hy.eta * beta[0, 0] * (1 - beta[0, 0] * kap.sum()) / kap.sum() * kap
    np.testing.assert_allclose(res["d_traj"][1, 0], np.clip(d2, 0.5, 2.0), atol=1e-15)
    # un-normalised key: the 1 / max(|k|^2, eps) factor matters
    k2 = 0.3 * k
    res2 = oracle.fwd(hy, [L], q, k2, v, beta, g, want_dtraj=True)
    kap = k2[0, 0] ** 2
    d2 = 1.0 + hy.eta * beta[0, 0] * (1 - beta[0, 0] * kap.sum()) / kap.sum() * kap
    np.testing.assert_allclose(res2["d_traj"][1, 0], np.clip(d2, 0.5, 2.0), atol=1e-15)
    # non-beta-aware form: beta replaced by one inside the feedback
    hy3 = OsdnHyper(eta=0.4, apf_mode=0, beta_aware=0)
    res3 = oracle.fwd(hy3, [L], q, k, v, beta, g, want_dtraj=True)
    kap = k[0, 0] ** 2
    d3 = 1.0 + hy.eta * (1 - kap.sum()) / kap.sum() * kap
    np.testing.assert_allclose(res3["d_traj"][1, 0], np.clip(d3, 0.5, 2.0), atol=1e-15)
    # zero key: normaliser falls back to eps, nothing blows up, d only sees retention
    k0 = k.copy(); k0[2] = 0.0
    res4 = oracle.fwd(OsdnHyper(eta=0.4, apf_mode=1), [L], q, k0, v, beta, g, want_dtraj=True)
    np.testing.assert_allclose(res4["d_traj"][3, 0],
                               np.clip(np.exp(g[2, 0]) * res4["d_traj"][2, 0], 0.5, 2.0), atol=1e-15)
    assert np.isfinite(res4["out"]).all()


# ---------------------------------------------------------------- residual ratio of the mechanism diagnostic
def test_residual_ratio_definition_equals_token_local_closed_form():
    """The oracle forms q_t = f_t(S_t) / f_t(exp(g_t) S_{t-1}) from the states; the proof of the
    token-local theorem gives q_t = (1 - beta_t <d_t, k_t^2>)^2, which involves neither S nor v."""
    hy = OsdnHyper(eta=0.3, apf_mode=1)
    L, H, K, V = 40, 2, 6, 5
    q, k, v, beta, g = _small(4, L, H, K, V, unit=False)
    r = _rng(9)
    S0 = r.standard_normal((2, H, V, K))
    d0 = r.uniform(hy.d_min, hy.d_max, size=(2, H, K))
    lens = [25, 15]
    got = oracle.residual_ratio(hy, lens, k, v, beta, g, None, S0, d0)
    dtr = oracle.fwd(hy, lens, q, k, v, beta, g, None, S0, d0, want_dtraj=True)["d_traj"]
    want = (1.0 - beta * np.einsum("thk,thk->th", dtr, k ** 2)) ** 2
    np.testing.assert_allclose(got, want, rtol=1e-9, atol=1e-12)
    # other values change nothing: the ratio does not depend on v or on the state
    got2 = oracle.residual_ratio(hy, lens, k, 3.0 * v[::-1].copy(), beta, g, None, -S0, d0)
    np.testing.assert_allclose(got2, want, rtol=1e-8, atol=1e-12)


def test_residual_ratio_special_cases():
    L, H, K, V = 9, 1, 4, 3
    q, k, v, beta, g = _small(6, L, H, K, V, unit=True)
    # beta = 0: nothing is written, the loss does not move
    hy = OsdnHyper(eta=0.3, apf_mode=0)
    assert np.array_equal(oracle.residual_ratio(hy, [L], k, v, 0 * beta, g), np.ones((L, H)))
    # plain delta rule (eta = 0, d = 1) with unit keys: q_t = (1 - beta_t)^2, an exact overwrite at beta = 1
    hy0 = OsdnHyper(eta=0.0, apf_mode=0)
    np.testing.assert_allclose(oracle.residual_ratio(hy0, [L], k, v, beta, g), (1 - beta) ** 2, rtol=1e-9, atol=1e-15)
    np.testing.assert_allclose(oracle.residual_ratio(hy0, [L], k, v, np.ones_like(beta), g), 0.0, atol=1e-25)
    # a preconditioner of 2 on unit keys doubles the step: q_t = (1 - 2 beta_t)^2
    d2 = np.full((1, H, K), 2.0)
    np.testing.assert_allclose(oracle.residual_ratio(hy0, [L], k, v, beta, g, None, None, d2), (1 - 2 * beta) ** 2,
                               rtol=1e-9, atol=1e-15)
