/*
 * Q-Delta fp64 CPU oracle.  TEST INFRASTRUCTURE ONLY: nothing on the product
 * (CUDA) path may include, link or call this file; only the test-suite, the
 * smoke check and the benchmark's CPU-baseline leg use it.  It shares no code
 * with the CUDA library.
 *
 * What it computes is the plain definition of the method: the token-by-token
 * gated Q-Delta recurrence (paper Section 3.3.1, final update rule with forget
 * gate, and the read-out o_t = S_t q_t), with x_t = k_t + lambda_t q_t
 * (Section 3.3.2, first display).  The state is held transposed with respect
 * to the paper: h_t = S_t^T, a d_k x d_v matrix, row-major.
 *
 *   hbar  = alpha_t * h_{t-1}
 *   p_t   = hbar^T x_t                  (= alpha (S_{t-1} k + lambda S_{t-1} q))
 *   e_t   = v_t - p_t                   (mixed key-query prediction error)
 *   delta = beta_t * e_t
 *   h_t   = hbar + k_t delta^T          (rank-one write along k_t)
 *   o_t   = h_t^T q_t                   (read-out uses the post-update state)
 *
 * The forget gate multiplies S_{t-1} in front of the whole bracket of the
 * final rule, hence it also scales the prediction inside the error (the
 * Q-Delta row of Table 1 says the same).
 *
 * The paper never writes a backward pass; the reverse pass below is the exact
 * gradient of the forward above for the scalar
 *   L = sum_t <o_t, dO_t> + <h_T, dh_T>_F,
 * walked from t = T down to 1.  It keeps one state checkpoint every `ckpt`
 * tokens and recomputes the states inside a segment.
 *
 * All tensors are token-major: q,k [B,T,H,dk], v,o [B,T,H,dv],
 * beta,alpha,lambda [B,T,H], states [B,H,dk,dv]; everything double.
 * Parallelism: one OpenMP iteration per (b,h) sequence, nothing else.
 */
#include <stdlib.h>
#include <string.h>
#include <stddef.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int qd_oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* One step of the recurrence on one (b,h) state, in place.
 * h: [dk*dv] (becomes h_t), scratch e: [dv] receives e_t, o: [dv] or NULL. */
static void step_fwd(int dk, int dv, double *h, const double *q, const double *k,
                     const double *v, double beta, double alpha, double lam,
                     double *e, double *o) {
    /* p = (alpha h)^T x, accumulated into e as v - p */
    for (int j = 0; j < dv; ++j) e[j] = 0.0;
    for (int i = 0; i < dk; ++i) {
        const double xi = k[i] + lam * q[i];
        double *hi = h + (size_t)i * dv;
        for (int j = 0; j < dv; ++j) {
            hi[j] *= alpha;            /* hbar */
            e[j] += hi[j] * xi;        /* p_j */
        }
    }
    for (int j = 0; j < dv; ++j) e[j] = v[j] - e[j];
    for (int i = 0; i < dk; ++i) {
        double *hi = h + (size_t)i * dv;
        const double bk = beta * k[i];
        for (int j = 0; j < dv; ++j) hi[j] += bk * e[j];
    }
    if (o) {
        for (int j = 0; j < dv; ++j) o[j] = 0.0;
        for (int i = 0; i < dk; ++i) {
            const double *hi = h + (size_t)i * dv;
            const double qi = q[i];
            for (int j = 0; j < dv; ++j) o[j] += hi[j] * qi;
        }
    }
}

/* Forward recurrence.  h0 may be NULL (zero state); hT may be NULL. */
int qd_oracle_fwd(int B, int T, int H, int dk, int dv,
                  const double *q, const double *k, const double *v,
                  const double *beta, const double *alpha, const double *lam,
                  const double *h0, double *o, double *hT) {
    if (B <= 0 || T < 0 || H <= 0 || dk <= 0 || dv <= 0) return 1;
    int fail = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < B * H; ++bh) {
        const int b = bh / H, hh = bh % H;
        double *h = (double *)malloc(sizeof(double) * (size_t)dk * dv);
        double *e = (double *)malloc(sizeof(double) * (size_t)dv);
        if (!h || !e) { fail = 1; free(h); free(e); continue; }
        if (h0) memcpy(h, h0 + (size_t)bh * dk * dv, sizeof(double) * (size_t)dk * dv);
        else memset(h, 0, sizeof(double) * (size_t)dk * dv);
        for (int t = 0; t < T; ++t) {
            const size_t r = ((size_t)b * T + t) * H + hh;
            step_fwd(dk, dv, h, q + r * dk, k + r * dk, v + r * dv,
                     beta[r], alpha ? alpha[r] : 1.0, lam ? lam[r] : 0.0,
                     e, o ? o + r * dv : NULL);
        }
        if (hT) memcpy(hT + (size_t)bh * dk * dv, h, sizeof(double) * (size_t)dk * dv);
        free(h); free(e);
    }
    return fail;
}

/* Reverse pass.  Outputs dq,dk_,dv_ [B,T,H,d], dbeta,dalpha,dlam [B,T,H],
 * dh0 [B,H,dk,dv] (may be NULL).  dhT may be NULL (zero).  dalpha is the
 * derivative with respect to alpha itself.  ckpt >= 1 is the checkpoint
 * spacing (memory/time trade only; the result does not depend on it). */
int qd_oracle_bwd(int B, int T, int H, int dk, int dv, int ckpt,
                  const double *q, const double *k, const double *v,
                  const double *beta, const double *alpha, const double *lam,
                  const double *h0, const double *dO, const double *dhT,
                  double *dq, double *dk_, double *dv_,
                  double *dbeta, double *dalpha, double *dlam, double *dh0) {
    if (B <= 0 || T < 0 || H <= 0 || dk <= 0 || dv <= 0 || ckpt <= 0) return 1;
    const size_t S = (size_t)dk * dv;
    const int nseg = (T + ckpt - 1) / ckpt;
    int fail = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < B * H; ++bh) {
        const int b = bh / H, hh = bh % H;
        /* checkpoints: state at the entry of every segment */
        double *cp = (double *)malloc(sizeof(double) * S * (size_t)(nseg > 0 ? nseg : 1));
        /* states inside one segment: hs[0] = entry, hs[s] = after s steps */
        double *hs = (double *)malloc(sizeof(double) * S * (size_t)(ckpt + 1));
        double *dh = (double *)malloc(sizeof(double) * S);
        double *e = (double *)malloc(sizeof(double) * (size_t)dv);
        double *ddl = (double *)malloc(sizeof(double) * (size_t)dv);
        double *dp = (double *)malloc(sizeof(double) * (size_t)dv);
        double *dx = (double *)malloc(sizeof(double) * (size_t)dk);
        if (!cp || !hs || !dh || !e || !ddl || !dp || !dx) {
            fail = 1;
            free(cp); free(hs); free(dh); free(e); free(ddl); free(dp); free(dx);
            continue;
        }
        /* forward sweep, storing checkpoints */
        double *h = hs; /* reuse hs[0] as the running state */
        if (h0) memcpy(h, h0 + (size_t)bh * S, sizeof(double) * S);
        else memset(h, 0, sizeof(double) * S);
        for (int t = 0; t < T; ++t) {
            if (t % ckpt == 0) memcpy(cp + (size_t)(t / ckpt) * S, h, sizeof(double) * S);
            const size_t r = ((size_t)b * T + t) * H + hh;
            step_fwd(dk, dv, h, q + r * dk, k + r * dk, v + r * dv,
                     beta[r], alpha ? alpha[r] : 1.0, lam ? lam[r] : 0.0, e, NULL);
        }
        if (dhT) memcpy(dh, dhT + (size_t)bh * S, sizeof(double) * S);
        else memset(dh, 0, sizeof(double) * S);

        for (int seg = nseg - 1; seg >= 0; --seg) {
            const int t0 = seg * ckpt;
            const int len = (t0 + ckpt <= T) ? ckpt : (T - t0);
            memcpy(hs, cp + (size_t)seg * S, sizeof(double) * S);
            for (int s = 0; s < len; ++s) {
                const size_t r = ((size_t)b * T + (t0 + s)) * H + hh;
                memcpy(hs + (size_t)(s + 1) * S, hs + (size_t)s * S, sizeof(double) * S);
                step_fwd(dk, dv, hs + (size_t)(s + 1) * S, q + r * dk, k + r * dk, v + r * dv,
                         beta[r], alpha ? alpha[r] : 1.0, lam ? lam[r] : 0.0, e, NULL);
            }
            for (int s = len - 1; s >= 0; --s) {
                const size_t r = ((size_t)b * T + (t0 + s)) * H + hh;
                const double *qt = q + r * dk, *kt = k + r * dk, *vt = v + r * dv;
                const double *dOt = dO + r * dv;
                const double bt = beta[r];
                const double at = alpha ? alpha[r] : 1.0;
                const double lt = lam ? lam[r] : 0.0;
                const double *hp = hs + (size_t)s * S;        /* h_{t-1} */
                const double *hn = hs + (size_t)(s + 1) * S;  /* h_t     */
                double *dqt = dq + r * dk, *dkt = dk_ + r * dk, *dvt = dv_ + r * dv;

                /* recompute e_t = v - alpha h_{t-1}^T x */
                for (int j = 0; j < dv; ++j) e[j] = 0.0;
                for (int i = 0; i < dk; ++i) {
                    const double xi = kt[i] + lt * qt[i];
                    const double *hpi = hp + (size_t)i * dv;
                    for (int j = 0; j < dv; ++j) e[j] += at * hpi[j] * xi;
                }
                for (int j = 0; j < dv; ++j) e[j] = vt[j] - e[j];

                /* o_t = h_t^T q_t */
                for (int i = 0; i < dk; ++i) {
                    double acc = 0.0;
                    const double *hni = hn + (size_t)i * dv;
                    double *dhi = dh + (size_t)i * dv;
                    for (int j = 0; j < dv; ++j) {
                        acc += hni[j] * dOt[j];
                        dhi[j] += qt[i] * dOt[j];
                    }
                    dqt[i] = acc;
                }
                /* h_t = hbar + k delta^T,  delta = beta e */
                for (int j = 0; j < dv; ++j) ddl[j] = 0.0;
                for (int i = 0; i < dk; ++i) {
                    const double *dhi = dh + (size_t)i * dv;
                    double acc = 0.0;
                    for (int j = 0; j < dv; ++j) {
                        acc += dhi[j] * bt * e[j];
                        ddl[j] += dhi[j] * kt[i];
                    }
                    dkt[i] = acc;
                }
                double db = 0.0;
                for (int j = 0; j < dv; ++j) {
                    db += ddl[j] * e[j];
                    dvt[j] = bt * ddl[j];      /* de = beta ddelta; dv = de */
                    dp[j] = -bt * ddl[j];      /* dp = -de */
                }
                dbeta[r] = db;
                /* p = hbar^T x, hbar = alpha h_{t-1} */
                double da = 0.0;
                for (int i = 0; i < dk; ++i) {
                    const double xi = kt[i] + lt * qt[i];
                    const double *hpi = hp + (size_t)i * dv;
                    double *dhi = dh + (size_t)i * dv;
                    double acc = 0.0;
                    for (int j = 0; j < dv; ++j) {
                        acc += at * hpi[j] * dp[j];
                        dhi[j] += xi * dp[j];          /* dhbar */
                        da += dhi[j] * hpi[j];
                        dhi[j] *= at;                  /* now d h_{t-1} */
                    }
                    dx[i] = acc;
                }
                dalpha[r] = da;
                /* x = k + lambda q */
                double dl = 0.0;
                for (int i = 0; i < dk; ++i) {
                    dkt[i] += dx[i];
                    dl += dx[i] * qt[i];
                    dqt[i] += lt * dx[i];
                }
                dlam[r] = dl;
            }
        }
        if (dh0) memcpy(dh0 + (size_t)bh * S, dh, sizeof(double) * S);
        free(cp); free(hs); free(dh); free(e); free(ddl); free(dp); free(dx);
    }
    return fail;
}
