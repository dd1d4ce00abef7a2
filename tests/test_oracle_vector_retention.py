"""Pins of the oracle's vector-retention mode (apf_mode 3: diag(r_t) in place of r_t I in the affine
form of the preconditioner update, the paper's "vector-retention extension").

The mode is pinned to things that do not come from its own code path: the scalar mode it must reduce
to, the closed form of pure retention, scalar recurrences written out per coordinate for one-hot
keys, and central finite differences of the forward."""
import numpy as np
import pytest

import oracle
from paper_2605_13473_b200.synth import OsdnHyper


def _unit(x):
    return x / np.linalg.norm(x, axis=-1, keepdims=True)


def _case(seed, hy, lens, H=2, K=5, V=4, unit=False):
    r = np.random.default_rng(seed)
    T, ns = sum(lens), len(lens)
    k = r.standard_normal((T, H, K)) * 0.6
    x = dict(
        q=_unit(r.standard_normal((T, H, K))), k=_unit(k) if unit else k, v=r.standard_normal((T, H, V)),
        beta=1 / (1 + np.exp(-r.standard_normal((T, H)))),
        gate=-0.4 * np.abs(r.standard_normal((T, H))),
        log_ret=-0.3 * np.abs(r.standard_normal((T, H, K))),
        init_state=0.5 * r.standard_normal((ns, H, V, K)),
        precond_in=hy.d_min + (hy.d_max - hy.d_min) * r.random((ns, H, K)),
    )
    cot = dict(out=r.standard_normal((T, H, V)), final_state=r.standard_normal((ns, H, V, K)),
               precond_out=r.standard_normal((ns, H, K)))
    return x, cot


def _fwd(hy, lens, x, **kw):
    return oracle.fwd(hy, lens, x["q"], x["k"], x["v"], x["beta"], x["gate"], x["log_ret"],
                      x["init_state"], x["precond_in"], **kw)


def _bwd(hy, lens, x, cot):
    return oracle.bwd(hy, lens, x["q"], x["k"], x["v"], x["beta"], x["gate"], cot["out"], x["log_ret"],
                      x["init_state"], x["precond_in"], cot["final_state"], cot["precond_out"])


@pytest.mark.parametrize("beta_aware", [1, 0])
def test_equal_coordinates_reduce_to_scalar_retention(beta_aware):
    """diag(r 1) = r I: a vector whose coordinates are all equal gives the scalar mode exactly, and the
    scalar's gradient is the sum of the coordinates' gradients."""
    lens = [9, 14]
    hv = OsdnHyper(eta=0.4, apf_mode=3, beta_aware=beta_aware)
    hs = OsdnHyper(eta=0.4, apf_mode=2, beta_aware=beta_aware)
    x, cot = _case(5, hv, lens)
    scalar = x["log_ret"][:, :, 0].copy()
    xv = dict(x, log_ret=np.repeat(scalar[:, :, None], x["k"].shape[-1], axis=2))
    xs = dict(x, log_ret=scalar)
    fv, fs = _fwd(hv, lens, xv), _fwd(hs, lens, xs)
    for n in ("out", "final_state", "precond_out"):
        assert np.array_equal(fv[n], fs[n]), n
    gv, gs = _bwd(hv, lens, xv, cot), _bwd(hs, lens, xs, cot)
    for n in ("dq", "dk", "dv", "dbeta", "dgate", "dinit_state", "dprecond_in"):
        assert np.allclose(gv[n], gs[n], rtol=1e-13, atol=1e-13), n
    assert gv["dlog_ret"].shape == xv["log_ret"].shape
    assert np.allclose(gv["dlog_ret"].sum(-1), gs["dlog_ret"], rtol=1e-12, atol=1e-13)


def test_pure_retention_closed_form():
    """eta = 0, no projection: d_L = d_0 (.) exp(sum_t l_t), coordinate by coordinate."""
    lens = [17, 6]
    hy = OsdnHyper(eta=0.0, apf_mode=3, clamp=0)
    x, _ = _case(8, hy, lens)
    res = oracle.precond_update(hy, lens, x["k"], x["beta"], x["gate"], x["log_ret"], x["precond_in"])
    off = 0
    for s, n in enumerate(lens):
        want = x["precond_in"][s] * np.exp(x["log_ret"][off:off + n].sum(0))
        assert np.allclose(res["precond_out"][s], want, rtol=1e-13)
        # the write key of token t carries the retention of tokens < t only
        t = off + n - 1
        d_before = x["precond_in"][s] * np.exp(x["log_ret"][off:t].sum(0))
        assert np.allclose(res["ktil"][t], d_before * x["k"][t], rtol=1e-13)
        off += n


def test_onehot_keys_scalar_recurrences_per_coordinate():
    """One-hot keys e_j: coordinate j takes the scalar step r_j d + eta b (1 - b d), every other
    coordinate only decays by its own retention; both projected onto the box."""
    K, L = 4, 40
    hy = OsdnHyper(eta=0.5, apf_mode=3, d_min=0.5, d_max=2.0)
    r = np.random.default_rng(3)
    hot = r.integers(0, K, size=L)
    k = np.zeros((L, 1, K))
    k[np.arange(L), 0, hot] = 1.0
    beta = r.uniform(0.2, 0.95, size=(L, 1))
    lr = -r.uniform(0.0, 0.15, size=(L, 1, K))
    d0 = r.uniform(0.6, 1.8, size=(1, 1, K))
    res = oracle.precond_update(hy, [L], k, beta, np.zeros((L, 1)), lr, d0)
    d = d0[0, 0].copy()
    for t in range(L):
        j, b = hot[t], beta[t, 0]
        assert np.allclose(res["ktil"][t, 0], d * k[t, 0], rtol=1e-14)
        new = np.exp(lr[t, 0]) * d
        new[j] += hy.eta * b * (1.0 - b * d[j])
        d = np.clip(new, hy.d_min, hy.d_max)
    assert np.allclose(res["precond_out"][0, 0], d, rtol=1e-13)
    assert (d == hy.d_min).any() or (d == hy.d_max).any() or L < 10   # the projection was exercised


@pytest.mark.parametrize("clamp", [1, 0])
def test_backward_matches_finite_differences(clamp):
    hy = OsdnHyper(eta=0.5, apf_mode=3, clamp=clamp)
    lens = [7, 5]
    for seed in range(400, 470):
        x, cot = _case(seed, hy, lens)
        f = _fwd(hy, lens, x, want_margin=True)
        frac = 1.0 - f["mask"].mean()
        if not clamp or (f["margin"].min() > 1e-4 and 0.02 < frac < 0.98):
            break
    else:
        pytest.fail("no usable seed")
    g = _bwd(hy, lens, x, cot)
    names = dict(q="dq", k="dk", v="dv", beta="dbeta", gate="dgate", log_ret="dlog_ret",
                 init_state="dinit_state", precond_in="dprecond_in")

    def loss():
        res = _fwd(hy, lens, x)
        return sum(float(np.sum(res[n] * cot[n])) for n in cot)

    h = 1e-6
    r = np.random.default_rng(7)
    for inp, gname in names.items():
        flat = x[inp].reshape(-1)
        for i in r.choice(flat.size, size=min(flat.size, 25), replace=False):
            old = flat[i]
            flat[i] = old + h
            lp = loss()
            flat[i] = old - h
            lm = loss()
            flat[i] = old
            fd, an = (lp - lm) / (2 * h), g[gname].reshape(-1)[i]
            assert abs(fd - an) <= 2e-6 * max(1.0, abs(an)), (inp, i, fd, an)
