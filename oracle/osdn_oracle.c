/*
 * OSDN oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, double-precision, token-by-token CPU statement of the
 * online-scaled gated delta rule and of its reverse-mode derivative.  It is
 * the definition the CUDA library is checked against; it shares no code with
 * that library and must never be called from it.  Only the tests, the smoke
 * check and the CPU-baseline leg of the benchmark may use it.
 *
 * What is computed, per (sequence, head) chain, for t = 1..L:
 *
 *   phase 1 (Algorithm 1; Eq. "dt_update_apf"; beta-aware form of the
 *   backbone-extension appendix, Eq. "extension_beta_aware_phase1"):
 *       ktil_t = d_t (.) k_t                       write key from PRE-update d
 *       kap    = k_t (.) k_t ,  n = max(sum kap, eps)
 *       a      = <d_t, kap> ,   b = beta_aware ? beta_t : 1
 *       c      = eta * b * (1 - b a) / n
 *       rho    = 1 | exp(g_t) | exp(l_t)           (no APF | aliased | separate)
 *       dbar   = rho d_t + c kap ;  d_{t+1} = clip(dbar, d_min, d_max)
 *   apf_mode 3, the vector-retention extension of the affine form of the update
 *   (diag(r_t) in place of r_t I): dbar = exp(l_t) (.) d_t + c kap with l_t in R^K.
 *
 *   phase 2 (gated, online-scaled delta rule of the backbone-extension
 *   appendix, post-gate residual):
 *       Sbar = exp(g_t) S_{t-1}
 *       u    = v_t - Sbar k_t                      read with the unscaled key
 *       S_t  = Sbar + beta_t u ktil_t^T            write with the scaled key
 *       o_t  = scale * S_t q_t                     read after the write
 *
 *   channel gate (OSKDA, backbone-extension appendix "Kimi Delta Attention with
 *   Online Scaling"): the scalar exp(g_t) becomes one gate per key channel,
 *       Sbar = S_{t-1} Diag(alpha_t),   alpha_t = exp(g_t) in (0,1]^K,
 *   everything else unchanged.  The paper writes the state as K x V with the
 *   gate, the read key and the scaled write key on the left,
 *       S'_t = (I - beta ktil k^T) Diag(alpha_t) S'_{t-1} + beta ktil v^T,  o = S'^T q;
 *   with S' = S^T these are the lines above (S is kept V x K here as well).  The
 *   preconditioner's retention stays separate from the channel gate, so the
 *   aliased mode (apf_mode 1) is not defined for it.
 *
 * The backward pass is the hand-derived adjoint of exactly these lines
 * (Section 3.5 only states its factorisation); it is validated against
 * central finite differences in the tests.
 *
 * Pins (tests/test_oracle_pins.py): Lemma 1 residual identity, the monotone
 * descent corollary, reduction to the gated delta rule / DeltaNet for d == 1,
 * beta == 0 no-op, exact overwrite for orthonormal keys, the one-hot closed
 * form of the preconditioner recurrence, the K=V=1 alternating example, the
 * WY product identity and the chunkwise form (an independent numpy program),
 * APF with unit retention, split-sequence carry, finite differences.
 * Channel gate (tests/test_oracle_oskda.py): equal gates in every channel give
 * the scalar-gate result, an independent numpy program of the paper's chunk
 * equations (cumulative channel decays, suffix-gated write key) gives the same
 * outputs and state, the K x V left-multiplied form written out in numpy gives
 * the transpose, finite differences for the gradients.
 * Absolute output values for random inputs have no printed example in the
 * paper: beyond those pins they are "parity unpinned".
 *
 * Layout: packed tokens [T_total, H, *]; sequences given by cu_seqlens
 * (nseq + 1 entries).  States S are [nseq, H, V, K], preconditioners
 * [nseq, H, K].  Everything is double.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    double eta, d_min, d_max, eps, scale;
    int beta_aware, apf_mode, clamp;
    int channel_gate;   /* gate is [T,H,K]: one log-gate per key channel (OSKDA) */
} oracle_hyper;

int osdn_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Retention inputs of token-head th: apf_mode 2 reads one log-retention per
 * token-head, apf_mode 3 (vector retention, diag(r_t) in place of r_t I in the
 * affine form of the update) one per coordinate. */
#define LRET_S(hp, lr, th) (((lr) && (hp)->apf_mode != 3) ? (lr)[th] : 0.0)
#define LRET_V(hp, lr, th, K) (((lr) && (hp)->apf_mode == 3) ? (lr) + (th) * (size_t)(K) : (const double *)0)
/* Gate inputs of token-head th: one log-gate, or K of them with a channel gate. */
#define GATE_S(hp, g, th) ((hp)->channel_gate ? 0.0 : (g)[th])
#define GATE_V(hp, g, th, K) ((hp)->channel_gate ? (g) + (th) * (size_t)(K) : (const double *)0)

/* One phase-1 step.  Reads d (length K) and overwrites it with d_{t+1}.
 * Optionally reports ktil, the scalar c and the pass-through mask.
 * lret_vec (apf_mode 3 only): K log-retentions, one per coordinate. */
static void phase1_step(const oracle_hyper *hp, int K, const double *k, double beta,
                        double g, double lret, const double *lret_vec, double *d, double *ktil,
                        double *c_out, double *rho_out, double *a_out, double *n_out,
                        int *raw_norm_above_eps, unsigned char *mask, double *margin)
{
    double sumk = 0.0, a = 0.0;
    for (int i = 0; i < K; ++i) {
        double kap = k[i] * k[i];
        if (ktil) ktil[i] = d[i] * k[i];
        sumk += kap;
        a += d[i] * kap;
    }
    double n = sumk > hp->eps ? sumk : hp->eps;
    double b = hp->beta_aware ? beta : 1.0;
    double c = hp->eta * b * (1.0 - b * a) / n;
    double rho = 1.0;
    if (hp->apf_mode == 1) rho = exp(g);
    else if (hp->apf_mode == 2) rho = exp(lret);
    for (int i = 0; i < K; ++i) {
        double ri = (hp->apf_mode == 3 && lret_vec) ? exp(lret_vec[i]) : rho;
        double dbar = ri * d[i] + c * k[i] * k[i];
        unsigned char m = 1;
        if (margin) {
            double lo = fabs(dbar - hp->d_min), hi = fabs(dbar - hp->d_max);
            margin[i] = hp->clamp ? (lo < hi ? lo : hi) : 1e300;
        }
        if (hp->clamp) {
            if (dbar < hp->d_min) { dbar = hp->d_min; m = 0; }
            else if (dbar > hp->d_max) { dbar = hp->d_max; m = 0; }
        }
        d[i] = dbar;
        if (mask) mask[i] = m;
    }
    if (c_out) *c_out = c;
    if (rho_out) *rho_out = rho;
    if (a_out) *a_out = a;
    if (n_out) *n_out = n;
    if (raw_norm_above_eps) *raw_norm_above_eps = sumk > hp->eps;
}

/* One phase-2 step on S (V x K, row-major); gvec (nullable): K channel log-gates in place of g.  u_out (length V) receives the
 * post-gate residual v - Sbar k; S is overwritten by S_t. */
static void phase2_step(int K, int V, const double *k, const double *ktil, const double *v,
                        double beta, double g, const double *gvec, double *S, double *u_out)
{
    for (int r = 0; r < V; ++r) {
        double *row = S + (size_t)r * K;
        double acc = 0.0;
        for (int i = 0; i < K; ++i) {
            row[i] *= exp(gvec ? gvec[i] : g);
            acc += row[i] * k[i];
        }
        double u = v[r] - acc;
        if (u_out) u_out[r] = u;
        double bu = beta * u;
        for (int i = 0; i < K; ++i) row[i] += bu * ktil[i];
    }
}

/*
 * Forward.  Nullable: log_ret (needed for apf_mode 2: [T,H]; 3: [T,H,K]), S0 (zeros), d0 (ones),
 * ktil_out, d_traj_out ([T_total, H, K], the PRE-update d_t of every token).
 */
void osdn_oracle_fwd(int nseq, const int *cu, int H, int K, int V, const oracle_hyper *hp,
                     const double *q, const double *k, const double *v,
                     const double *beta, const double *gate, const double *log_ret,
                     const double *S0, const double *d0,
                     double *out, double *S_final, double *d_final,
                     double *ktil_out, double *d_traj_out, double *margin_out, unsigned char *mask_out)
{
    int nchain = nseq * H;
#pragma omp parallel for schedule(dynamic, 1)
    for (int ch = 0; ch < nchain; ++ch) {
        int s = ch / H, h = ch % H;
        int t0 = cu[s], t1 = cu[s + 1];
        double *S = (double *)malloc(sizeof(double) * V * K);
        double *d = (double *)malloc(sizeof(double) * K);
        double *ktil = (double *)malloc(sizeof(double) * K);
        if (S0) memcpy(S, S0 + ((size_t)s * H + h) * V * K, sizeof(double) * V * K);
        else memset(S, 0, sizeof(double) * V * K);
        for (int i = 0; i < K; ++i) d[i] = d0 ? d0[((size_t)s * H + h) * K + i] : 1.0;
        for (int t = t0; t < t1; ++t) {
            size_t th = (size_t)t * H + h;
            const double *kt = k + th * K, *qt = q + th * K, *vt = v + th * V;
            if (d_traj_out) memcpy(d_traj_out + th * K, d, sizeof(double) * K);
            phase1_step(hp, K, kt, beta[th], GATE_S(hp, gate, th), LRET_S(hp, log_ret, th), LRET_V(hp, log_ret, th, K), d, ktil,
                        0, 0, 0, 0, 0, mask_out ? mask_out + th * K : 0, margin_out ? margin_out + th * K : 0);
            if (ktil_out) memcpy(ktil_out + th * K, ktil, sizeof(double) * K);
            phase2_step(K, V, kt, ktil, vt, beta[th], GATE_S(hp, gate, th), GATE_V(hp, gate, th, K), S, 0);
            for (int r = 0; r < V; ++r) {
                double acc = 0.0;
                for (int i = 0; i < K; ++i) acc += S[(size_t)r * K + i] * qt[i];
                out[th * V + r] = hp->scale * acc;
            }
        }
        if (S_final) memcpy(S_final + ((size_t)s * H + h) * V * K, S, sizeof(double) * V * K);
        if (d_final) memcpy(d_final + ((size_t)s * H + h) * K, d, sizeof(double) * K);
        free(S); free(d); free(ktil);
    }
}

/*
 * Residual ratio of the mechanism diagnostic, by its definition: with the
 * per-token loss f_t(S) = 1/2 |S k_t - v_t|^2,
 *     q_t = f_t(S_t) / f_t(Sbar_{t-1}),      Sbar_{t-1} = exp(g_t) S_{t-1},
 * the loss after the write over the loss before it (the state the write starts
 * from is the gated one).  0/0 is read as 1 (no residual, nothing to reduce).
 * The closed form (1 - beta_t <d_t, k_t^2>)^2 of the token-local theorem is NOT
 * used here; it is what the tests and the CUDA path are compared with.
 * ratio_out [T_total, H].
 */
void osdn_oracle_residual_ratio(int nseq, const int *cu, int H, int K, int V, const oracle_hyper *hp,
                                const double *k, const double *v, const double *beta, const double *gate,
                                const double *log_ret, const double *S0, const double *d0, double *ratio_out)
{
    int nchain = nseq * H;
#pragma omp parallel for schedule(dynamic, 1)
    for (int ch = 0; ch < nchain; ++ch) {
        int s = ch / H, h = ch % H;
        double *S = (double *)malloc(sizeof(double) * V * K);
        double *d = (double *)malloc(sizeof(double) * K);
        double *ktil = (double *)malloc(sizeof(double) * K);
        double *u = (double *)malloc(sizeof(double) * V);
        if (S0) memcpy(S, S0 + ((size_t)s * H + h) * V * K, sizeof(double) * V * K);
        else memset(S, 0, sizeof(double) * V * K);
        for (int i = 0; i < K; ++i) d[i] = d0 ? d0[((size_t)s * H + h) * K + i] : 1.0;
        for (int t = cu[s]; t < cu[s + 1]; ++t) {
            size_t th = (size_t)t * H + h;
            const double *kt = k + th * K, *vt = v + th * V;
            phase1_step(hp, K, kt, beta[th], gate[th], LRET_S(hp, log_ret, th), LRET_V(hp, log_ret, th, K), d, ktil,
                        0, 0, 0, 0, 0, 0, 0);
            phase2_step(K, V, kt, ktil, vt, beta[th], gate[th], 0, S, u);   /* u = v - Sbar k */
            double before = 0.0, after = 0.0;
            for (int r = 0; r < V; ++r) {
                double acc = 0.0;
                for (int i = 0; i < K; ++i) acc += S[(size_t)r * K + i] * kt[i];
                after += (acc - vt[r]) * (acc - vt[r]);
                before += u[r] * u[r];
            }
            ratio_out[th] = before > 0.0 ? after / before : 1.0;
        }
        free(S); free(d); free(ktil); free(u);
    }
}

/* Phase 1 alone (the stand-alone preconditioner update). */
void osdn_oracle_precond_update(int nseq, const int *cu, int H, int K, const oracle_hyper *hp,
                                const double *k, const double *beta, const double *gate,
                                const double *log_ret, const double *d0,
                                double *ktil_out, double *d_final)
{
    int nchain = nseq * H;
#pragma omp parallel for schedule(dynamic, 1)
    for (int ch = 0; ch < nchain; ++ch) {
        int s = ch / H, h = ch % H;
        double *d = (double *)malloc(sizeof(double) * K);
        double *ktil = (double *)malloc(sizeof(double) * K);
        for (int i = 0; i < K; ++i) d[i] = d0 ? d0[((size_t)s * H + h) * K + i] : 1.0;
        for (int t = cu[s]; t < cu[s + 1]; ++t) {
            size_t th = (size_t)t * H + h;
            phase1_step(hp, K, k + th * K, beta[th], gate ? gate[th] : 0.0,
                        LRET_S(hp, log_ret, th), LRET_V(hp, log_ret, th, K), d, ktil, 0, 0, 0, 0, 0, 0, 0);
            if (ktil_out) memcpy(ktil_out + th * K, ktil, sizeof(double) * K);
        }
        memcpy(d_final + ((size_t)s * H + h) * K, d, sizeof(double) * K);
        free(d); free(ktil);
    }
}

/*
 * Backward: reverse sweep over the same recurrence.
 *
 * Cotangents in: dout [T,H,V]; dS_final, dd_final nullable (zeros).
 * Gradients out: dq, dk [T,H,K], dv [T,H,V], dbeta, dgate [T,H],
 * dlog_ret [T,H] for apf_mode 2, [T,H,K] for apf_mode 3 (nullable), dS0, dd0 (nullable).
 *
 * S_{t-1} and d_t are needed in reverse order.  Each chain keeps S and d at
 * every SEG-token boundary during a forward sweep, then walks the segments
 * backwards, re-running each segment forward with a full per-token history.
 *
 * Conventions where the paper is silent: the box projection passes gradient
 * iff d_min <= dbar <= d_max; max(|k|^2, eps) passes gradient iff |k|^2 > eps.
 *
 * mask_override ([T_total, H, K], nullable): 0 / 1 force the pass decision of
 * one coordinate of one step, 255 leaves it to the rule above.  The gradient is
 * discontinuous where dbar touches a face; a caller comparing against an fp32
 * implementation uses this to take near-tie decisions (|dbar - face| within
 * fp32 rounding) in that implementation's precision, and only those.
 */
#define SEG 64

void osdn_oracle_bwd(int nseq, const int *cu, int H, int K, int V, const oracle_hyper *hp,
                     const double *q, const double *k, const double *v,
                     const double *beta, const double *gate, const double *log_ret,
                     const double *S0, const double *d0,
                     const double *dout, const double *dS_final, const double *dd_final,
                     const unsigned char *mask_override,
                     double *dq, double *dk, double *dv, double *dbeta, double *dgate,
                     double *dlog_ret, double *dS0, double *dd0)
{
    int nchain = nseq * H;
    size_t VK = (size_t)V * K;
#pragma omp parallel for schedule(dynamic, 1)
    for (int ch = 0; ch < nchain; ++ch) {
        int s = ch / H, h = ch % H;
        int t0 = cu[s], t1 = cu[s + 1];
        int L = t1 - t0;
        int nseg = (L + SEG - 1) / SEG;
        double *Sck = (double *)malloc(sizeof(double) * VK * (nseg > 0 ? nseg : 1));
        double *dck = (double *)malloc(sizeof(double) * K * (nseg > 0 ? nseg : 1));
        double *Shist = (double *)malloc(sizeof(double) * VK * (SEG + 1)); /* S before each token */
        double *dhist = (double *)malloc(sizeof(double) * K * (SEG + 1));  /* d before each token */
        double *S = (double *)malloc(sizeof(double) * VK);
        double *d = (double *)malloc(sizeof(double) * K);
        double *ktil = (double *)malloc(sizeof(double) * K);
        double *Shat = (double *)malloc(sizeof(double) * VK);   /* dL/dS_t */
        double *lam = (double *)malloc(sizeof(double) * K);     /* dL/dd_{t+1} */
        double *Sbar = (double *)malloc(sizeof(double) * VK);
        double *u = (double *)malloc(sizeof(double) * V);
        double *w = (double *)malloc(sizeof(double) * V);
        double *du = (double *)malloc(sizeof(double) * V);
        double *dktil = (double *)malloc(sizeof(double) * K);
        double *dnew = (double *)malloc(sizeof(double) * K);
        unsigned char *mask = (unsigned char *)malloc(K);

        if (S0) memcpy(S, S0 + ((size_t)s * H + h) * VK, sizeof(double) * VK);
        else memset(S, 0, sizeof(double) * VK);
        for (int i = 0; i < K; ++i) d[i] = d0 ? d0[((size_t)s * H + h) * K + i] : 1.0;

        /* forward sweep keeping segment-boundary checkpoints */
        for (int sg = 0; sg < nseg; ++sg) {
            memcpy(Sck + (size_t)sg * VK, S, sizeof(double) * VK);
            memcpy(dck + (size_t)sg * K, d, sizeof(double) * K);
            int a0 = t0 + sg * SEG, a1 = a0 + SEG < t1 ? a0 + SEG : t1;
            for (int t = a0; t < a1; ++t) {
                size_t th = (size_t)t * H + h;
                phase1_step(hp, K, k + th * K, beta[th], GATE_S(hp, gate, th), LRET_S(hp, log_ret, th),
                            LRET_V(hp, log_ret, th, K), d, ktil, 0, 0, 0, 0, 0, 0, 0);
                phase2_step(K, V, k + th * K, ktil, v + th * V, beta[th], GATE_S(hp, gate, th),
                            GATE_V(hp, gate, th, K), S, 0);
            }
        }

        if (dS_final) memcpy(Shat, dS_final + ((size_t)s * H + h) * VK, sizeof(double) * VK);
        else memset(Shat, 0, sizeof(double) * VK);
        for (int i = 0; i < K; ++i) lam[i] = dd_final ? dd_final[((size_t)s * H + h) * K + i] : 0.0;

        for (int sg = nseg - 1; sg >= 0; --sg) {
            int a0 = t0 + sg * SEG, a1 = a0 + SEG < t1 ? a0 + SEG : t1;
            /* replay the segment, recording S_{t-1} and d_t for every token */
            memcpy(S, Sck + (size_t)sg * VK, sizeof(double) * VK);
            memcpy(d, dck + (size_t)sg * K, sizeof(double) * K);
            for (int t = a0; t < a1; ++t) {
                size_t th = (size_t)t * H + h;
                memcpy(Shist + (size_t)(t - a0) * VK, S, sizeof(double) * VK);
                memcpy(dhist + (size_t)(t - a0) * K, d, sizeof(double) * K);
                phase1_step(hp, K, k + th * K, beta[th], GATE_S(hp, gate, th), LRET_S(hp, log_ret, th),
                            LRET_V(hp, log_ret, th, K), d, ktil, 0, 0, 0, 0, 0, 0, 0);
                phase2_step(K, V, k + th * K, ktil, v + th * V, beta[th], GATE_S(hp, gate, th),
                            GATE_V(hp, gate, th, K), S, 0);
            }
            for (int t = a1 - 1; t >= a0; --t) {
                size_t th = (size_t)t * H + h;
                const double *kt = k + th * K, *qt = q + th * K, *vt = v + th * V;
                const double *dot = dout + th * V;
                const double *Sprev = Shist + (size_t)(t - a0) * VK;
                const double *dt = dhist + (size_t)(t - a0) * K;
                double bt = beta[th], gt = GATE_S(hp, gate, th), lt = LRET_S(hp, log_ret, th);
                const double *lv = LRET_V(hp, log_ret, th, K);
                const double *gv = GATE_V(hp, gate, th, K);
#define ALPHA(i) exp(gv ? gv[i] : gt)

                /* recompute this token's forward quantities */
                double c, rho, a, n; int above;
                memcpy(dnew, dt, sizeof(double) * K);
                phase1_step(hp, K, kt, bt, gt, lt, lv, dnew, ktil, &c, &rho, &a, &n, &above, mask, 0);
                if (mask_override)
                    for (int i = 0; i < K; ++i)
                        if (mask_override[th * K + i] != 255) mask[i] = mask_override[th * K + i];
                for (int r = 0; r < V; ++r) {
                    double acc = 0.0;
                    for (int i = 0; i < K; ++i) {
                        Sbar[(size_t)r * K + i] = ALPHA(i) * Sprev[(size_t)r * K + i];
                        acc += Sbar[(size_t)r * K + i] * kt[i];
                    }
                    u[r] = vt[r] - acc;
                }
                /* o_t = scale S_t q_t with S_t = Sbar + beta u ktil^T */
                {
                    for (int i = 0; i < K; ++i) dq[th * K + i] = 0.0;
                    for (int r = 0; r < V; ++r) {
                        double sdo = hp->scale * dot[r];
                        for (int i = 0; i < K; ++i) {
                            double St = Sbar[(size_t)r * K + i] + bt * u[r] * ktil[i];
                            dq[th * K + i] += sdo * St;
                            Shat[(size_t)r * K + i] += sdo * qt[i];
                        }
                    }
                }
                /* S_t = Sbar + beta u ktil^T */
                double dbeta_t = 0.0;
                for (int i = 0; i < K; ++i) dktil[i] = 0.0;
                for (int r = 0; r < V; ++r) {
                    double acc = 0.0;
                    for (int i = 0; i < K; ++i) acc += Shat[(size_t)r * K + i] * ktil[i];
                    w[r] = acc;
                    dbeta_t += u[r] * acc;
                    du[r] = bt * acc;
                    for (int i = 0; i < K; ++i) dktil[i] += bt * u[r] * Shat[(size_t)r * K + i];
                }
                /* u = v - Sbar k ; Sbar = alpha S_{t-1} */
                double dg_t = 0.0;
                for (int i = 0; i < K; ++i) dk[th * K + i] = 0.0;
                if (gv)
                    for (int i = 0; i < K; ++i) dgate[th * K + i] = 0.0;
                for (int r = 0; r < V; ++r) {
                    dv[th * V + r] = du[r];
                    for (int i = 0; i < K; ++i) {
                        size_t id = (size_t)r * K + i;
                        dk[th * K + i] -= Sbar[id] * du[r];
                        double dSbar = Shat[id] - du[r] * kt[i];
                        if (gv) dgate[th * K + i] += dSbar * Sbar[id];   /* d/dg_i of exp(g_i) S[:, i] */
                        else dg_t += dSbar * Sbar[id];
                        Shat[id] = ALPHA(i) * dSbar;       /* now dL/dS_{t-1} */
                    }
                }
                /* phase-1 adjoint of this step; lam holds dL/dd_{t+1} */
                double drho = 0.0, dc = 0.0;
                for (int i = 0; i < K; ++i) {
                    double lb = mask[i] ? lam[i] : 0.0;
                    lam[i] = lb;
                    drho += lb * dt[i];
                    dc += lb * kt[i] * kt[i];
                }
                double b = hp->beta_aware ? bt : 1.0;
                double da = -hp->eta * b * b / n * dc;
                double db = hp->eta * (1.0 - 2.0 * b * a) / n * dc;
                double dn = above ? -c / n * dc : 0.0;
                if (hp->beta_aware) dbeta_t += db;
                for (int i = 0; i < K; ++i) {
                    double kap = kt[i] * kt[i];
                    double dkap = c * lam[i] + da * dt[i] + dn;
                    dk[th * K + i] += dt[i] * dktil[i] + 2.0 * kt[i] * dkap;
                    double ri = lv ? exp(lv[i]) : rho;
                    /* vector retention: d(dbar_i)/d(l_i) = r_i d_i, one gradient per coordinate */
                    if (lv && dlog_ret) dlog_ret[th * K + i] = ri * lam[i] * dt[i];
                    lam[i] = ri * lam[i] + da * kap + kt[i] * dktil[i];   /* dL/dd_t */
                }
                if (hp->apf_mode == 1) dg_t += rho * drho;
                if (dlog_ret && !lv) dlog_ret[th] = hp->apf_mode == 2 ? rho * drho : 0.0;
                dbeta[th] = dbeta_t;
                if (!gv) dgate[th] = dg_t;
#undef ALPHA
            }
        }
        if (dS0) memcpy(dS0 + ((size_t)s * H + h) * VK, Shat, sizeof(double) * VK);
        if (dd0) memcpy(dd0 + ((size_t)s * H + h) * K, lam, sizeof(double) * K);

        free(Sck); free(dck); free(Shist); free(dhist); free(S); free(d); free(ktil);
        free(Shat); free(lam); free(Sbar); free(u); free(w); free(du); free(dktil);
        free(dnew); free(mask);
    }
}
