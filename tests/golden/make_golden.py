"""Writes the golden text fixtures from closed forms stated in the paper.

Run as ``python tests/golden/make_golden.py``.  It evaluates formulas only; it
calls neither the oracle nor the CUDA library.
"""
import os

HERE = os.path.dirname(os.path.abspath(__file__))


def alternating(n=12):
    # remark after Theorem 2: K=V=1, k=1, v_t=(-1)^t, exact per-token Newton step
    rows = ["# t v_t S_t   (beta=0.5, d=2, eta=0 -> beta*d=1; S_t must equal v_t)"]
    for t in range(1, n + 1):
        v = (-1.0) ** t
        rows.append(f"{t} {v:.1f} {v:.1f}")
    return "\n".join(rows) + "\n"


def onehot(n=40):
    # one coordinate of Eq. dt_update_apf with k = e_0 (kappa = e_0, n_t = 1):
    #   d <- clip((r - eta beta^2) d + eta beta, d_min, d_max)
    rows = ["# case eta beta r d_min d_max d0 : then d_0(t) for t = 0..n"]
    for name, eta, beta, r, dmin, dmax, d0 in [
        ("grow_to_1_over_beta", 0.3, 0.8, 1.0, 0.5, 2.0, 1.0),
        ("hits_dmax", 0.3, 0.4, 1.0, 0.5, 2.0, 1.0),
        ("apf_pulls_down", 0.05, 0.6, 0.9, 0.5, 2.0, 1.5),
    ]:
        d = d0
        vals = [d]
        for _ in range(n):
            d = min(max((r - eta * beta * beta) * d + eta * beta, dmin), dmax)
            vals.append(d)
        rows.append(f"{name} {eta} {beta} {r} {dmin} {dmax} {d0} : " + " ".join(f"{x:.15e}" for x in vals))
    return "\n".join(rows) + "\n"


if __name__ == "__main__":
    open(os.path.join(HERE, "alternating_k1.txt"), "w").write(alternating())
    open(os.path.join(HERE, "onehot_precond.txt"), "w").write(onehot())
