"""Chunkwise (UT / WY) statement of the layer in float64 numpy -- a test helper.

A second, independently written program for the same function as the
token-by-token oracle: the gated chunk form of the backbone-extension appendix
(decay-ratio Gram, unit-triangular inverse, W / U, suffix-gated state advance),
written in the division-free ratio form Gamma_ij = exp(G_i - G_j), plus the
reverse-mode derivative of that chunk form.  Tests use it to pin the oracle
(the two must agree to rounding) and as the reference derivation for the
chunk-level backward the CUDA kernels implement.  It imports neither the oracle
nor the CUDA package.
"""
from __future__ import annotations

import numpy as np


def phase1_np(k, beta, gate, log_ret, d0, hy):
    """Sequential preconditioner sweep for one chain.  k [L,K].  Returns
    (ktil [L,K], d_traj [L,K] pre-update, d_final [K], c [L], rho [L], mask [L,K], a, n, above)."""
    L, K = k.shape
    d = np.array(d0, dtype=np.float64).copy()
    ktil = np.zeros((L, K)); dtraj = np.zeros((L, K)); mask = np.ones((L, K), dtype=bool)
    cs = np.zeros(L); rhos = np.ones(L); aa = np.zeros(L); nn = np.zeros(L); above = np.zeros(L, bool)
    for t in range(L):
        dtraj[t] = d
        ktil[t] = d * k[t]
        kap = k[t] * k[t]
        sk = kap.sum()
        n = max(sk, hy.eps)
        a = float(d @ kap)
        b = beta[t] if hy.beta_aware else 1.0
        c = hy.eta * b * (1.0 - b * a) / n
        rho = 1.0
        if hy.apf_mode == 1:
            rho = np.exp(gate[t])
        elif hy.apf_mode == 2:
            rho = np.exp(log_ret[t])
        dbar = rho * d + c * kap
        if hy.clamp:
            mask[t] = (dbar >= hy.d_min) & (dbar <= hy.d_max)
            d = np.clip(dbar, hy.d_min, hy.d_max)
        else:
            d = dbar
        cs[t], rhos[t], aa[t], nn[t], above[t] = c, rho, a, n, sk > hy.eps
    return ktil, dtraj, d, cs, rhos, mask, aa, nn, above


def phase1_adjoint_np(k, beta, dtraj, cs, rhos, mask, aa, nn, above, dktil, dd_final, hy):
    """Reverse sweep over the projected affine recurrence for one chain.
    Returns (dk_add [L,K], dbeta_add [L], drho_log [L] (= rho * drho), dd0 [K])."""
    L, K = k.shape
    lam = np.array(dd_final, dtype=np.float64).copy()
    dk = np.zeros((L, K)); dbeta = np.zeros(L); dlog = np.zeros(L)
    for t in range(L - 1, -1, -1):
        kap = k[t] * k[t]
        lb = np.where(mask[t], lam, 0.0)
        drho = float(lb @ dtraj[t])
        dc = float(lb @ kap)
        b = beta[t] if hy.beta_aware else 1.0
        da = -hy.eta * b * b / nn[t] * dc
        db = hy.eta * (1.0 - 2.0 * b * aa[t]) / nn[t] * dc
        dn = -cs[t] / nn[t] * dc if above[t] else 0.0
        if hy.beta_aware:
            dbeta[t] = db
        dkap = cs[t] * lb + da * dtraj[t] + dn
        dk[t] = dtraj[t] * dktil[t] + 2.0 * k[t] * dkap
        lam = rhos[t] * lb + da * kap + k[t] * dktil[t]
        dlog[t] = rhos[t] * drho
    return dk, dbeta, dlog, lam


def _pad(x, Lp):
    L = x.shape[0]
    if L == Lp:
        return x
    pad = np.zeros((Lp - L,) + x.shape[1:], dtype=x.dtype)
    return np.concatenate([x, pad], axis=0)


def chunk_quantities(q, k, ktil, v, beta, g):
    """All per-chunk matrices of one chunk (C tokens)."""
    C = q.shape[0]
    G = np.cumsum(g)
    gam = np.exp(G)
    Gam = np.exp(np.minimum(G[:, None] - G[None, :], 0.0))  # used only for j <= i
    lower = np.tril(np.ones((C, C), bool), -1)
    lower_eq = np.tril(np.ones((C, C), bool), 0)
    raw_kk = k @ ktil.T
    A = np.where(lower, beta[:, None] * Gam * raw_kk, 0.0)
    Tm = np.linalg.inv(np.eye(C) + A)
    Kb = (beta * gam)[:, None] * k
    Vb = beta[:, None] * v
    W = Tm @ Kb
    U = Tm @ Vb
    raw_qk = q @ ktil.T
    P = np.where(lower_eq, Gam * raw_qk, 0.0)
    rho = np.exp(G[-1] - G)
    return dict(G=G, gam=gam, Gam=Gam, lower=lower, lower_eq=lower_eq, raw_kk=raw_kk, A=A, T=Tm,
                Kb=Kb, Vb=Vb, W=W, U=U, raw_qk=raw_qk, P=P, rho=rho, gC=np.exp(G[-1]))


def chain_fwd(q, k, ktil, v, beta, g, S0, scale, C=64):
    """Chunkwise forward of one chain.  Returns (o [L,V], S_final, saved list)."""
    L = q.shape[0]
    N = (L + C - 1) // C
    Lp = N * C
    qp, kp, ktp, vp, bp, gp = (_pad(x, Lp) for x in (q, k, ktil, v, beta, g))
    S = np.array(S0, dtype=np.float64).copy()
    o = np.zeros((Lp, v.shape[1]))
    saved = []
    for n in range(N):
        sl = slice(n * C, (n + 1) * C)
        cq = chunk_quantities(qp[sl], kp[sl], ktp[sl], vp[sl], bp[sl], gp[sl])
        dU = cq["U"] - cq["W"] @ S.T
        o[sl] = scale * ((cq["gam"][:, None] * qp[sl]) @ S.T + cq["P"] @ dU)
        saved.append((cq, S.copy(), dU))
        S = cq["gC"] * S + dU.T @ (cq["rho"][:, None] * ktp[sl])
    return o[:L], S, saved


def wy_product(k, ktil, beta):
    """prod_i (I - beta_i k_i ktil_i^T) (ungated), and its WY form I - W^T Ktil."""
    C, K = k.shape
    Pm = np.eye(K)
    for i in range(C):
        Pm = Pm @ (np.eye(K) - beta[i] * np.outer(k[i], ktil[i]))
    A = np.tril(beta[:, None] * (k @ ktil.T), -1)
    Tm = np.linalg.inv(np.eye(C) + A)
    W = Tm @ (beta[:, None] * k)
    return Pm, np.eye(K) - W.T @ ktil


def chain_bwd(q, k, ktil, v, beta, g, S0, scale, do, dS_final, C=64):
    """Chunk-level reverse pass of one chain (phase 2 only).
    Returns dq, dk_read, dktil, dv, dbeta, dg, dS0."""
    L, K = q.shape
    V = v.shape[1]
    N = (L + C - 1) // C
    Lp = N * C
    qp, kp, ktp, vp, bp, gp, dop = (_pad(x, Lp) for x in (q, k, ktil, v, beta, g, do))
    _, _, saved = chain_fwd(q, k, ktil, v, beta, g, S0, scale, C)
    dS = np.array(dS_final, dtype=np.float64).copy()  # dL/dS at chunk end
    dq = np.zeros((Lp, K)); dk = np.zeros((Lp, K)); dkt = np.zeros((Lp, K)); dv = np.zeros((Lp, V))
    dbeta = np.zeros(Lp); dg = np.zeros(Lp)
    for n in range(N - 1, -1, -1):
        sl = slice(n * C, (n + 1) * C)
        cq, S, dU = saved[n]
        Q, Kc, Kt, Vc, b, dO = qp[sl], kp[sl], ktp[sl], vp[sl], bp[sl], dop[sl]
        gam, Gam, rho, gC, Tm = cq["gam"], cq["Gam"], cq["rho"], cq["gC"], cq["T"]
        # output and state-advance cotangents
        ddU = scale * cq["P"].T @ dO + (rho[:, None] * Kt) @ dS.T            # [C,V]
        dP = np.where(cq["lower_eq"], scale * dO @ dU.T, 0.0)                  # wrt P entries
        dQg = scale * dO @ S                                                   # wrt gam*Q
        dKtr = dU @ dS                                                         # wrt rho*Ktil  [C,K]
        dW = -ddU @ S                                                          # [C,K]
        dUm = ddU
        dS_prev = gC * dS + scale * dO.T @ (gam[:, None] * Q) - ddU.T @ cq["W"]
        # through W = T Kb, U = T Vb
        dT = dW @ cq["Kb"].T + dUm @ cq["Vb"].T
        dKb = Tm.T @ dW
        dVb = Tm.T @ dUm
        dA = np.where(cq["lower"], -(Tm.T @ dT @ Tm.T), 0.0)
        # leaves
        dq[sl] = gam[:, None] * dQg + (dP * Gam) @ Kt
        dkt[sl] = rho[:, None] * dKtr + (dP * Gam).T @ Q + (dA * b[:, None] * Gam).T @ Kc
        dk[sl] = (b * gam)[:, None] * dKb + (dA * b[:, None] * Gam) @ Kt
        dv[sl] = b[:, None] * dVb
        dbeta[sl] = (np.sum(dKb * (gam[:, None] * Kc), axis=1) + np.sum(dVb * Vc, axis=1)
                     + np.sum(dA * Gam * cq["raw_kk"], axis=1))
        dAA = dA * cq["A"]
        dPP = dP * cq["P"]
        dG = (np.sum(dQg * (gam[:, None] * Q), axis=1) + np.sum(dKb * cq["Kb"], axis=1)
              + dAA.sum(axis=1) - dAA.sum(axis=0) + dPP.sum(axis=1) - dPP.sum(axis=0)
              - np.sum(dKtr * (rho[:, None] * Kt), axis=1))
        dG[-1] += np.sum(dKtr * (rho[:, None] * Kt)) + gC * np.sum(dS * S)
        dg[sl] = np.cumsum(dG[::-1])[::-1]
        dS = dS_prev
    return dq[:L], dk[:L], dkt[:L], dv[:L], dbeta[:L], dg[:L], dS


def layer_fwd(hy, seq_lens, q, k, v, beta, gate, log_ret=None, init_state=None, precond_in=None, C=64):
    T, H, K = q.shape
    V = v.shape[-1]
    scale = hy.scale if hy.scale and hy.scale > 0 else K ** -0.5
    cu = np.concatenate([[0], np.cumsum(seq_lens)]).astype(int)
    out = np.zeros((T, H, V)); Sf = np.zeros((len(seq_lens), H, V, K)); df = np.zeros((len(seq_lens), H, K))
    for s in range(len(seq_lens)):
        sl = slice(cu[s], cu[s + 1])
        for h in range(H):
            d0 = np.ones(K) if precond_in is None else precond_in[s, h]
            S0 = np.zeros((V, K)) if init_state is None else init_state[s, h]
            lr = None if log_ret is None else log_ret[sl, h]
            ktil, _, dfin, *_ = phase1_np(k[sl, h], beta[sl, h], gate[sl, h], lr, d0, hy)
            o, S, _ = chain_fwd(q[sl, h], k[sl, h], ktil, v[sl, h], beta[sl, h], gate[sl, h], S0, scale, C)
            out[sl, h] = o; Sf[s, h] = S; df[s, h] = dfin
    return dict(out=out, final_state=Sf, precond_out=df)


def layer_bwd(hy, seq_lens, q, k, v, beta, gate, dout, log_ret=None, init_state=None, precond_in=None,
              dfinal_state=None, dprecond_out=None, C=64):
    T, H, K = q.shape
    V = v.shape[-1]
    scale = hy.scale if hy.scale and hy.scale > 0 else K ** -0.5
    cu = np.concatenate([[0], np.cumsum(seq_lens)]).astype(int)
    ns = len(seq_lens)
    r = dict(dq=np.zeros((T, H, K)), dk=np.zeros((T, H, K)), dv=np.zeros((T, H, V)),
             dbeta=np.zeros((T, H)), dgate=np.zeros((T, H)), dlog_ret=np.zeros((T, H)),
             dinit_state=np.zeros((ns, H, V, K)), dprecond_in=np.zeros((ns, H, K)))
    for s in range(ns):
        sl = slice(cu[s], cu[s + 1])
        for h in range(H):
            d0 = np.ones(K) if precond_in is None else precond_in[s, h]
            S0 = np.zeros((V, K)) if init_state is None else init_state[s, h]
            dSf = np.zeros((V, K)) if dfinal_state is None else dfinal_state[s, h]
            ddf = np.zeros(K) if dprecond_out is None else dprecond_out[s, h]
            lr = None if log_ret is None else log_ret[sl, h]
            ktil, dtraj, _, cs, rhos, mask, aa, nn, above = phase1_np(
                k[sl, h], beta[sl, h], gate[sl, h], lr, d0, hy)
            dq, dkr, dkt, dv, db, dg, dS0 = chain_bwd(q[sl, h], k[sl, h], ktil, v[sl, h], beta[sl, h],
                                                      gate[sl, h], S0, scale, dout[sl, h], dSf, C)
            dk1, db1, dlog, dd0 = phase1_adjoint_np(k[sl, h], beta[sl, h], dtraj, cs, rhos, mask, aa,
                                                    nn, above, dkt, ddf, hy)
            r["dq"][sl, h] = dq; r["dk"][sl, h] = dkr + dk1; r["dv"][sl, h] = dv
            r["dbeta"][sl, h] = db + db1
            r["dgate"][sl, h] = dg + (dlog if hy.apf_mode == 1 else 0.0)
            if hy.apf_mode == 2:
                r["dlog_ret"][sl, h] = dlog
            r["dinit_state"][s, h] = dS0; r["dprecond_in"][s, h] = dd0
    return r
