/*
 * fp64 CPU oracle for tree-structured linear attention with a PER-CHANNEL decay.  TEST INFRASTRUCTURE ONLY:
 * nothing on the product path may call, link or import this file.
 *
 * The recurrence is the first term of the paper's Eq. 1 (Section 2.2), the diagonal decay Diag(gamma_t) acting on
 * the key dimension of the state, with the plain outer-product update (U = V, W = 0; the paper defines neither U
 * nor W, so the delta-rule part of Eq. 1 has no oracle):
 *
 *     S_0 = 0,   S_t = Diag(exp(g_t)) S_{t-1} + k_t^T v_t,   o_t = q_t S_t,     g_t in R^{dk}, g_t <= 0   (per head)
 *
 * As in la_oracle.c it is the plain definition: one trajectory at a time, token by token, no chunks.  Reverse
 * recurrence (dS_t is the gradient of L = sum_t <dO_t, o_t> w.r.t. S_t):
 *     dS_t = q_t^T dO_t + Diag(exp(g_{t+1})) dS_{t+1},   dS_{T+1} = 0
 *     dq_t = S_t dO_t^T,   dk_t = dS_t v_t^T,   dv_t = dS_t^T k_t,
 *     dg_t[i] = exp(g_t[i]) * sum_j S_{t-1}[i][j] dS_t[i][j]
 * The backward sweep re-runs the forward over windows of WIN tokens from saved window-start states.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>

#define WIN 100

/* S <- Diag(exp(g)) S + k^T v */
static void state_step(int dk, int dv, double *S, const double *g, const double *k, const double *v) {
    for (int i = 0; i < dk; i++) {
        double a = exp(g[i]);
        for (int j = 0; j < dv; j++) S[i * dv + j] = a * S[i * dv + j] + k[i] * v[j];
    }
}

static void read_out(int dk, int dv, const double *S, const double *q, double *o) {
    for (int j = 0; j < dv; j++) o[j] = 0.0;
    for (int i = 0; i < dk; i++)
        for (int j = 0; j < dv; j++) o[j] += q[i] * S[i * dv + j];
}

/* Forward of one trajectory, one head: q,k [T,dk], v [T,dv], g [T,dk] -> o [T,dv]. */
void harts_gk_oracle_traj_fwd(int T, int dk, int dv, const double *q, const double *k, const double *v,
                              const double *g, double *o) {
    double *S = (double *)calloc((size_t)dk * dv, sizeof(double));
    for (int t = 0; t < T; t++) {
        state_step(dk, dv, S, g + (size_t)t * dk, k + (size_t)t * dk, v + (size_t)t * dv);
        read_out(dk, dv, S, q + (size_t)t * dk, o + (size_t)t * dv);
    }
    free(S);
}

/* Backward of one trajectory, one head; dg is [T,dk]. */
void harts_gk_oracle_traj_bwd(int T, int dk, int dv, const double *q, const double *k, const double *v,
                              const double *g, const double *dO, double *dq, double *dk_, double *dv_, double *dg) {
    size_t n = (size_t)dk * dv;
    int nwin = (T + WIN - 1) / WIN;
    double *start = (double *)calloc((size_t)(nwin + 1) * n, sizeof(double));
    double *hist = (double *)calloc((size_t)(WIN + 1) * n, sizeof(double));
    double *dS = (double *)calloc(n, sizeof(double));      /* Diag(exp(g_{t+1})) dS_{t+1} on entry to token t */
    double *S = (double *)calloc(n, sizeof(double));
    for (int t = 0; t < T; t++) {
        if (t % WIN == 0) memcpy(start + (size_t)(t / WIN) * n, S, n * sizeof(double));
        state_step(dk, dv, S, g + (size_t)t * dk, k + (size_t)t * dk, v + (size_t)t * dv);
    }
    for (int w = nwin - 1; w >= 0; w--) {
        int t0 = w * WIN, t1 = t0 + WIN < T ? t0 + WIN : T;
        memcpy(hist, start + (size_t)w * n, n * sizeof(double));
        for (int t = t0; t < t1; t++) {
            memcpy(hist + (size_t)(t - t0 + 1) * n, hist + (size_t)(t - t0) * n, n * sizeof(double));
            state_step(dk, dv, hist + (size_t)(t - t0 + 1) * n, g + (size_t)t * dk, k + (size_t)t * dk, v + (size_t)t * dv);
        }
        for (int t = t1 - 1; t >= t0; t--) {
            const double *St = hist + (size_t)(t - t0 + 1) * n, *Sp = hist + (size_t)(t - t0) * n;
            const double *qt = q + (size_t)t * dk, *kt = k + (size_t)t * dk, *vt = v + (size_t)t * dv;
            const double *dOt = dO + (size_t)t * dv, *gt = g + (size_t)t * dk;
            for (int i = 0; i < dk; i++)
                for (int j = 0; j < dv; j++) dS[i * dv + j] += qt[i] * dOt[j];
            for (int i = 0; i < dk; i++) {
                double aq = 0.0, ak = 0.0, ag = 0.0;
                for (int j = 0; j < dv; j++) {
                    aq += St[i * dv + j] * dOt[j];
                    ak += dS[i * dv + j] * vt[j];
                    ag += Sp[i * dv + j] * dS[i * dv + j];
                }
                dq[(size_t)t * dk + i] = aq;
                dk_[(size_t)t * dk + i] = ak;
                dg[(size_t)t * dk + i] = exp(gt[i]) * ag;
            }
            for (int j = 0; j < dv; j++) {
                double av = 0.0;
                for (int i = 0; i < dk; i++) av += dS[i * dv + j] * kt[i];
                dv_[(size_t)t * dv + j] = av;
            }
            /* hand Diag(exp(g_t)) dS_t to token t-1 */
            for (int i = 0; i < dk; i++) {
                double a = exp(gt[i]);
                for (int j = 0; j < dv; j++) dS[i * dv + j] *= a;
            }
        }
    }
    free(start); free(hist); free(dS); free(S);
}
