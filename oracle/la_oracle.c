/*
 * fp64 CPU oracle for tree-structured linear attention.  TEST INFRASTRUCTURE ONLY:
 * nothing on the product path may call, link or import this file.
 *
 * What it computes is the plain definition, not the method: every root-to-leaf
 * trajectory of the rollout tree is evaluated on its own, token by token, from a
 * zero state (the conventional trajectory-wise training the paper's Section 1 and
 * Section 4.3 take as the baseline):
 *
 *     S_0 = 0,   S_t = exp(g_t) * S_{t-1} + k_t^T v_t,   o_t = q_t S_t        (per head)
 *
 * which is the paper's Eq. 1 with U = V, W = 0 and a scalar decay per head and token.
 * Semantic positions reach compact rows through the map m of Eq. 3: the output of a
 * compact row is the output of any semantic position mapped to it (all copies must
 * agree; the largest disagreement is reported), and gradients of
 * L = sum_c <dO_c, o_c> are accumulated over all copies, each copy carrying
 * dO_c / multiplicity (Eq. 20 defines the multiplicity), the same accumulate-over-m
 * pattern as Eq. 19.
 *
 * Reverse recurrence per trajectory (dS_t is the gradient of L w.r.t. S_t):
 *     dS_t = q_t^T dO_t + exp(g_{t+1}) dS_{t+1},  dS_{T+1} = 0
 *     dq_t = S_t dO_t^T,  dk_t = dS_t v_t^T,  dv_t = dS_t^T k_t,
 *     dg_t = exp(g_t) * <S_{t-1}, dS_t>
 *
 * No chunking, no blocking of the arithmetic, no reordering.  The only concession to
 * memory is that the backward sweep re-runs the forward recurrence over windows of
 * WIN tokens from saved window-start states instead of keeping every S_t.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define WIN 100 /* deliberately not a multiple of any chunk length */

/* S <- exp(g) S + k^T v */
static void state_step(int dk, int dv, double *S, double g, const double *k, const double *v) {
    double a = exp(g);
    for (int i = 0; i < dk; i++)
        for (int j = 0; j < dv; j++) S[i * dv + j] = a * S[i * dv + j] + k[i] * v[j];
}

/* o = q S */
static void read_out(int dk, int dv, const double *S, const double *q, double *o) {
    for (int j = 0; j < dv; j++) o[j] = 0.0;
    for (int i = 0; i < dk; i++)
        for (int j = 0; j < dv; j++) o[j] += q[i] * S[i * dv + j];
}

/* Forward of one trajectory, one head.  Inputs are row-major [T,dk], [T,dv], [T]. */
void harts_oracle_traj_fwd(int T, int dk, int dv, const double *q, const double *k, const double *v,
                           const double *g, double *o) {
    double *S = (double *)calloc((size_t)dk * dv, sizeof(double));
    for (int t = 0; t < T; t++) {
        state_step(dk, dv, S, g[t], k + (size_t)t * dk, v + (size_t)t * dv);
        read_out(dk, dv, S, q + (size_t)t * dk, o + (size_t)t * dv);
    }
    free(S);
}

/* Backward of one trajectory, one head.  o_chk (may be NULL) receives the recomputed outputs. */
void harts_oracle_traj_bwd(int T, int dk, int dv, const double *q, const double *k, const double *v,
                           const double *g, const double *dO, double *dq, double *dk_, double *dv_,
                           double *dg, double *o_chk) {
    size_t n = (size_t)dk * dv;
    int nwin = (T + WIN - 1) / WIN;
    double *start = (double *)calloc((size_t)(nwin + 1) * n, sizeof(double)); /* S before each window */
    double *hist = (double *)calloc((size_t)(WIN + 1) * n, sizeof(double));   /* S_{t-1}..S_t inside a window */
    double *dS = (double *)calloc(n, sizeof(double));                          /* exp(g_{t+1}) dS_{t+1} on entry */
    double *S = (double *)calloc(n, sizeof(double));
    /* forward sweep: remember the state at every window start */
    for (int t = 0; t < T; t++) {
        if (t % WIN == 0) memcpy(start + (size_t)(t / WIN) * n, S, n * sizeof(double));
        state_step(dk, dv, S, g[t], k + (size_t)t * dk, v + (size_t)t * dv);
        if (o_chk) read_out(dk, dv, S, q + (size_t)t * dk, o_chk + (size_t)t * dv);
    }
    for (int w = nwin - 1; w >= 0; w--) {
        int t0 = w * WIN, t1 = t0 + WIN < T ? t0 + WIN : T;
        /* hist[0] = S_{t0-1} (state before token t0), hist[i+1] = S_{t0+i} */
        memcpy(hist, start + (size_t)w * n, n * sizeof(double));
        for (int t = t0; t < t1; t++) {
            memcpy(hist + (size_t)(t - t0 + 1) * n, hist + (size_t)(t - t0) * n, n * sizeof(double));
            state_step(dk, dv, hist + (size_t)(t - t0 + 1) * n, g[t], k + (size_t)t * dk, v + (size_t)t * dv);
        }
        for (int t = t1 - 1; t >= t0; t--) {
            const double *St = hist + (size_t)(t - t0 + 1) * n, *Sp = hist + (size_t)(t - t0) * n;
            const double *qt = q + (size_t)t * dk, *kt = k + (size_t)t * dk, *vt = v + (size_t)t * dv;
            const double *dOt = dO + (size_t)t * dv;
            /* dS_t = q_t^T dO_t + (decayed gradient from t+1) */
            for (int i = 0; i < dk; i++)
                for (int j = 0; j < dv; j++) dS[i * dv + j] += qt[i] * dOt[j];
            double acc_g = 0.0;
            for (int i = 0; i < dk; i++) {
                double aq = 0.0, ak = 0.0;
                for (int j = 0; j < dv; j++) {
                    aq += St[i * dv + j] * dOt[j];
                    ak += dS[i * dv + j] * vt[j];
                    acc_g += Sp[i * dv + j] * dS[i * dv + j];
                }
                dq[(size_t)t * dk + i] = aq;
                dk_[(size_t)t * dk + i] = ak;
            }
            for (int j = 0; j < dv; j++) {
                double av = 0.0;
                for (int i = 0; i < dk; i++) av += dS[i * dv + j] * kt[i];
                dv_[(size_t)t * dv + j] = av;
            }
            double a = exp(g[t]);
            dg[t] = a * acc_g;
            /* hand exp(g_t) dS_t to token t-1 */
            for (size_t e = 0; e < n; e++) dS[e] *= a;
        }
    }
    free(start); free(hist); free(dS); free(S);
}

static void atomic_add(double *p, double x) {
#pragma omp atomic
    *p += x;
}

/*
 * All trajectories of a forest.  Compact tensors are row-major [C,H,dk] / [C,H,dv] / [C,H].
 * traj_ptr[n_traj+1], traj_rows[...]: compact row of every semantic position (the map m).
 * Outputs: o [C,H,dv]; if dO != NULL also dq,dk_,dv_ [C,H,d] and dg [C,H] (must be zeroed by
 * the caller; contributions of all copies are added).  *copy_gap receives the largest absolute
 * difference between the outputs of two semantic positions mapped to the same compact row.
 * Returns the number of threads used.
 */
int harts_oracle_forest(int n_traj, const long long *traj_ptr, const long long *traj_rows, long long C,
                        int H, int dk, int dv, const double *q, const double *k, const double *v,
                        const double *g, const double *dO, double *o, double *dq, double *dk_,
                        double *dv_, double *dg, double *copy_gap) {
    /* multiplicity of every compact row and the first trajectory that visits it */
    long long *mult = (long long *)calloc((size_t)C, sizeof(long long));
    int *owner = (int *)malloc((size_t)C * sizeof(int));
    for (long long c = 0; c < C; c++) owner[c] = -1;
    for (int x = 0; x < n_traj; x++)
        for (long long s = traj_ptr[x]; s < traj_ptr[x + 1]; s++) {
            long long c = traj_rows[s];
            mult[c]++;
            if (owner[c] < 0) owner[c] = x;
        }
    int nthreads = 1;
    double gap = 0.0;
    for (int pass = 0; pass < 2; pass++) {
        /* pass 0: forward, the first visitor of a row writes its output;
           pass 1: every copy is compared with that output and, if asked, back-propagated */
#pragma omp parallel
        {
#ifdef _OPENMP
#pragma omp single
            nthreads = omp_get_num_threads();
#endif
            double local_gap = 0.0;
#pragma omp for schedule(dynamic, 1) collapse(2)
            for (int x = 0; x < n_traj; x++)
                for (int h = 0; h < H; h++) {
                    int T = (int)(traj_ptr[x + 1] - traj_ptr[x]);
                    const long long *rows = traj_rows + traj_ptr[x];
                    double *tq = (double *)malloc((size_t)T * dk * sizeof(double));
                    double *tk = (double *)malloc((size_t)T * dk * sizeof(double));
                    double *tv = (double *)malloc((size_t)T * dv * sizeof(double));
                    double *tg = (double *)malloc((size_t)T * sizeof(double));
                    double *to = (double *)malloc((size_t)T * dv * sizeof(double));
                    for (int t = 0; t < T; t++) {
                        size_t r = (size_t)rows[t] * H + h;
                        memcpy(tq + (size_t)t * dk, q + r * dk, dk * sizeof(double));
                        memcpy(tk + (size_t)t * dk, k + r * dk, dk * sizeof(double));
                        memcpy(tv + (size_t)t * dv, v + r * dv, dv * sizeof(double));
                        tg[t] = g[r];
                    }
                    if (pass == 0) {
                        harts_oracle_traj_fwd(T, dk, dv, tq, tk, tv, tg, to);
                        for (int t = 0; t < T; t++)
                            if (owner[rows[t]] == x)
                                memcpy(o + ((size_t)rows[t] * H + h) * dv, to + (size_t)t * dv, dv * sizeof(double));
                    } else if (dO == NULL) {
                        harts_oracle_traj_fwd(T, dk, dv, tq, tk, tv, tg, to);
                    } else {
                        double *tdO = (double *)malloc((size_t)T * dv * sizeof(double));
                        double *tdq = (double *)malloc((size_t)T * dk * sizeof(double));
                        double *tdk = (double *)malloc((size_t)T * dk * sizeof(double));
                        double *tdv = (double *)malloc((size_t)T * dv * sizeof(double));
                        double *tdg = (double *)malloc((size_t)T * sizeof(double));
                        for (int t = 0; t < T; t++) {
                            size_t r = (size_t)rows[t] * H + h;
                            for (int j = 0; j < dv; j++)
                                tdO[(size_t)t * dv + j] = dO[r * dv + j] / (double)mult[rows[t]];
                        }
                        harts_oracle_traj_bwd(T, dk, dv, tq, tk, tv, tg, tdO, tdq, tdk, tdv, tdg, to);
                        for (int t = 0; t < T; t++) {
                            size_t r = (size_t)rows[t] * H + h;
                            for (int i = 0; i < dk; i++) {
                                atomic_add(dq + r * dk + i, tdq[(size_t)t * dk + i]);
                                atomic_add(dk_ + r * dk + i, tdk[(size_t)t * dk + i]);
                            }
                            for (int j = 0; j < dv; j++) atomic_add(dv_ + r * dv + j, tdv[(size_t)t * dv + j]);
                            atomic_add(dg + r, tdg[t]);
                        }
                        free(tdO); free(tdq); free(tdk); free(tdv); free(tdg);
                    }
                    if (pass == 1)
                        for (int t = 0; t < T; t++)
                            for (int j = 0; j < dv; j++) {
                                double d = fabs(to[(size_t)t * dv + j] - o[((size_t)rows[t] * H + h) * dv + j]);
                                if (d > local_gap) local_gap = d;
                            }
                    free(tq); free(tk); free(tv); free(tg); free(to);
                }
#pragma omp critical
            if (local_gap > gap) gap = local_gap;
        }
    }
    if (copy_gap) *copy_gap = gap;
    free(mult); free(owner);
    return nthreads;
}
