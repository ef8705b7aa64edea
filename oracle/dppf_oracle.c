/*
 * CPU oracle for the DPPF communication-round consensus step.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA path is checked against.  It shares no code, header, table or helper
 * with the CUDA library, and nothing in the product path may call it.
 *
 * Everything is evaluated in fp64 on widened fp32 inputs.  The scalars
 * (alpha, lambda, lr, momentum, weight decay) arrive as the same fp32 values
 * the GPU receives and are widened here, never re-parsed from decimals.
 *
 * What is computed (paper notation):
 *   x_A      = (1/M) sum_i x_i                      Algorithm 1 (last line), Sec. 4
 *   r_m      = || x_m - x_A ||_2                    Eq. (single-line update), Sec. 5
 *   x_m^+    = x_m + (x_A - x_m)(alpha - lambda/r_m)   Eq. (single-line update);
 *              same form with Delta = x_A - x_m in the proof of Theorem 1
 *   all workers use the same pre-round x_A          proof of Theorem 1, first display
 *
 * Readings where the paper is silent:
 *   - r_m == 0: the push direction is 0/0; no push is applied and the pull
 *     acts on a zero vector, so x_m is left exactly as it is (a plain copy,
 *     which also keeps the sign of zeros) and r_m = 0 is reported.  No
 *     epsilon is added anywhere.
 *   - local optimiser between rounds: Algorithm 1 prints plain SGD; the
 *     experiments use momentum 0.9 and weight decay without writing the
 *     recurrence.  The reading used is the standard coupled form
 *        g~ = g + wd*x ;  v <- mu*v + g~ ;  x <- x - lr*v ,  v_0 = 0.
 *
 * Parity status: every function below is pinned by tests/test_oracle_*.py
 * (hand cases, closed forms, exact rational brute force, invariants from the
 * proof of Theorem 1).  Inputs with 0 < r_m < 1e-15 are "parity unpinned".
 *
 * Layout: row-major [M, ld] with ld >= d; columns d..ld-1 are never read or
 * written.  Return value 0 = ok, 1 = bad argument, 2 = out of memory.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ---- core on an fp64 state -------------------------------------------- */

/* x_A[i] = (sum_{m ascending} x[m][i]) / M   (Algorithm 1, definition of x_A) */
static void average_f64(const double *x, int M, int64_t d, int64_t ld, double *A)
{
    for (int64_t i = 0; i < d; ++i) {
        double s = 0.0;
        for (int m = 0; m < M; ++m) s += x[(int64_t)m * ld + i];
        A[i] = s / (double)M;
    }
}

/* r[m] = sqrt(sum_{i ascending} (x[m][i] - A[i])^2)   (norm in Eq. single-line) */
static void distances_f64(const double *x, int M, int64_t d, int64_t ld,
                          const double *A, double *r)
{
    for (int m = 0; m < M; ++m) {
        double S = 0.0;
        const double *xm = x + (int64_t)m * ld;
        for (int64_t i = 0; i < d; ++i) {
            double diff = xm[i] - A[i];
            S += diff * diff;
        }
        r[m] = sqrt(S);
    }
}

/*
 * One pull-push round on an fp64 state; result rounded to fp32 once.
 * x_out may not alias x (different element types).
 */
int dppf_oracle_consensus_f64(const double *x, int M, int64_t d, int64_t ld,
                              float alpha, float lambda,
                              float *x_out, int64_t ld_out, double *r_out)
{
    if (!x || !x_out || !r_out || M < 1 || d < 1 || ld < d || ld_out < d) return 1;
    double *A = (double *)malloc((size_t)d * sizeof(double));
    if (!A) return 2;
    const double a = (double)alpha, lam = (double)lambda;

    average_f64(x, M, d, ld, A);
    distances_f64(x, M, d, ld, A, r_out);
    for (int m = 0; m < M; ++m) {
        /* c_m = alpha - lambda / r_m ; zero distance: replica unchanged (see header) */
        const double *xm = x + (int64_t)m * ld;
        float *om = x_out + (int64_t)m * ld_out;
        if (!(r_out[m] > 0.0)) {
            for (int64_t i = 0; i < d; ++i) om[i] = (float)xm[i];
            continue;
        }
        double c = a - lam / r_out[m];
        for (int64_t i = 0; i < d; ++i)
            om[i] = (float)(xm[i] + (A[i] - xm[i]) * c);
    }
    free(A);
    return 0;
}

/* Same round on fp32 replicas (each element widened first).  x_out may be x. */
int dppf_oracle_consensus(const float *x, int M, int64_t d, int64_t ld,
                          float alpha, float lambda,
                          float *x_out, int64_t ld_out, double *r_out)
{
    if (!x || !x_out || !r_out || M < 1 || d < 1 || ld < d || ld_out < d) return 1;
    double *A = (double *)malloc((size_t)d * sizeof(double));
    if (!A) return 2;
    const double a = (double)alpha, lam = (double)lambda;

    for (int64_t i = 0; i < d; ++i) {
        double s = 0.0;
        for (int m = 0; m < M; ++m) s += (double)x[(int64_t)m * ld + i];
        A[i] = s / (double)M;
    }
    for (int m = 0; m < M; ++m) {
        double S = 0.0;
        const float *xm = x + (int64_t)m * ld;
        for (int64_t i = 0; i < d; ++i) {
            double diff = (double)xm[i] - A[i];
            S += diff * diff;
        }
        r_out[m] = sqrt(S);
    }
    for (int m = 0; m < M; ++m) {
        const float *xm = x + (int64_t)m * ld;
        float *om = x_out + (int64_t)m * ld_out;
        if (!(r_out[m] > 0.0)) {                 /* zero distance: replica unchanged */
            for (int64_t i = 0; i < d; ++i) om[i] = xm[i];
            continue;
        }
        double c = a - lam / r_out[m];
        for (int64_t i = 0; i < d; ++i) {
            double xi = (double)xm[i];
            om[i] = (float)(xi + (A[i] - xi) * c);
        }
    }
    free(A);
    return 0;
}

/*
 * The two-step form printed in Algorithm 1: pull toward x_C = x_A, then push
 * along the direction of the pulled point from x_A.  Kept as a separate
 * transcription so that the single-line form can be checked against it
 * (they agree whenever alpha < 1; at alpha = 1 this form divides 0 by 0 and
 * the zero-distance reading leaves the pulled point where it is).
 */
int dppf_oracle_consensus_two_step(const float *x, int M, int64_t d, int64_t ld,
                                   float alpha, float lambda,
                                   float *x_out, int64_t ld_out, double *r_out)
{
    if (!x || !x_out || !r_out || M < 1 || d < 1 || ld < d || ld_out < d) return 1;
    double *A = (double *)malloc((size_t)d * sizeof(double));
    double *y = (double *)malloc((size_t)d * sizeof(double));
    if (!A || !y) { free(A); free(y); return 2; }
    const double a = (double)alpha, lam = (double)lambda;

    for (int64_t i = 0; i < d; ++i) {
        double s = 0.0;
        for (int m = 0; m < M; ++m) s += (double)x[(int64_t)m * ld + i];
        A[i] = s / (double)M;
    }
    for (int m = 0; m < M; ++m) {
        const float *xm = x + (int64_t)m * ld;
        float *om = x_out + (int64_t)m * ld_out;
        double S0 = 0.0, S1 = 0.0;
        for (int64_t i = 0; i < d; ++i) {
            double xi = (double)xm[i];
            double diff0 = xi - A[i];
            S0 += diff0 * diff0;
            y[i] = (1.0 - a) * xi + a * A[i];            /* pull */
            double diff1 = y[i] - A[i];
            S1 += diff1 * diff1;
        }
        r_out[m] = sqrt(S0);                              /* pre-round distance */
        if (!(r_out[m] > 0.0)) {                          /* zero distance: replica unchanged */
            for (int64_t i = 0; i < d; ++i) om[i] = xm[i];
            continue;
        }
        double n1 = sqrt(S1);
        for (int64_t i = 0; i < d; ++i) {
            double push = (n1 > 0.0) ? lam * (y[i] - A[i]) / n1 : 0.0;
            om[i] = (float)(y[i] + push);                 /* push */
        }
    }
    free(A); free(y);
    return 0;
}

/*
 * One local optimiser step on an fp64 state, in place (reading stated in the
 * header): g~ = g + wd*x ; v <- mu*v + g~ ; x <- x - lr*v.
 */
int dppf_oracle_local_step_f64(double *x, double *v, const float *g,
                               int M, int64_t d, int64_t ld, int64_t ld_g,
                               float lr, float momentum, float weight_decay)
{
    if (!x || !v || !g || M < 1 || d < 1 || ld < d || ld_g < d) return 1;
    const double eta = (double)lr, mu = (double)momentum, wd = (double)weight_decay;
    for (int m = 0; m < M; ++m) {
        double *xm = x + (int64_t)m * ld, *vm = v + (int64_t)m * ld;
        const float *gm = g + (int64_t)m * ld_g;
        for (int64_t i = 0; i < d; ++i) {
            double gt = (double)gm[i] + wd * xm[i];
            vm[i] = mu * vm[i] + gt;
            xm[i] = xm[i] - eta * vm[i];
        }
    }
    return 0;
}

/*
 * Column-block parallel copy of dppf_oracle_consensus for timing and for
 * full-size parity cases: thread t owns a contiguous column block, keeps its
 * own partial sums of squares, and the partials are combined in thread order.
 * Differs from the plain function only in the grouping of the sum over i.
 * threads <= 0 means "all available".  Returns the thread count used in
 * *threads_used.
 */
int dppf_oracle_consensus_blocked(const float *x, int M, int64_t d, int64_t ld,
                                  float alpha, float lambda,
                                  float *x_out, int64_t ld_out, double *r_out,
                                  int threads, int *threads_used)
{
    if (!x || !x_out || !r_out || M < 1 || d < 1 || ld < d || ld_out < d) return 1;
    int T = 1;
#ifdef _OPENMP
    T = threads > 0 ? threads : omp_get_max_threads();
#else
    (void)threads;
#endif
    if ((int64_t)T > d) T = (int)d;
    if (threads_used) *threads_used = T;
    double *A = (double *)malloc((size_t)d * sizeof(double));
    double *part = (double *)calloc((size_t)T * (size_t)M, sizeof(double));
    if (!A || !part) { free(A); free(part); return 2; }
    const double a = (double)alpha, lam = (double)lambda;

#pragma omp parallel for num_threads(T) schedule(static, 1)
    for (int t = 0; t < T; ++t) {
        int64_t lo = d * t / T, hi = d * (t + 1) / T;
        for (int64_t i = lo; i < hi; ++i) {
            double s = 0.0;
            for (int m = 0; m < M; ++m) s += (double)x[(int64_t)m * ld + i];
            A[i] = s / (double)M;
        }
        for (int m = 0; m < M; ++m) {
            double S = 0.0;
            const float *xm = x + (int64_t)m * ld;
            for (int64_t i = lo; i < hi; ++i) {
                double diff = (double)xm[i] - A[i];
                S += diff * diff;
            }
            part[(size_t)t * M + m] = S;
        }
    }
    for (int m = 0; m < M; ++m) {
        double S = 0.0;
        for (int t = 0; t < T; ++t) S += part[(size_t)t * M + m];
        r_out[m] = sqrt(S);
    }
#pragma omp parallel for num_threads(T) schedule(static, 1)
    for (int t = 0; t < T; ++t) {
        int64_t lo = d * t / T, hi = d * (t + 1) / T;
        for (int m = 0; m < M; ++m) {
            const float *xm = x + (int64_t)m * ld;
            float *om = x_out + (int64_t)m * ld_out;
            if (!(r_out[m] > 0.0)) {             /* zero distance: replica unchanged */
                for (int64_t i = lo; i < hi; ++i) om[i] = xm[i];
                continue;
            }
            double c = a - lam / r_out[m];
            for (int64_t i = lo; i < hi; ++i) {
                double xi = (double)xm[i];
                om[i] = (float)(xi + (A[i] - xi) * c);
            }
        }
    }
    free(A); free(part);
    return 0;
}

/*
 * General consensus round: Algorithm 1 with an arbitrary consensus variable and the
 * optional second term of the regulariser's gradient.
 *
 *   x_A = (1/M) sum_i x_i                        (Algorithm 1, last line)
 *   x_C = sum_i w_i x_i / sum_i w_i              ("any combination of worker parameters",
 *                                                 Sec. 3; w = one-hot gives a leader, as in
 *                                                 LSGD; w = NULL means x_C = x_A)
 *   P   = x_A, or x_C when push_from_c != 0      (the remark on LSGD: the push may be
 *                                                 redefined to oppose the leader)
 *   pull    y_m = (1 - alpha) x_m + alpha x_C    (Algorithm 1, pull line)
 *   u_m     = (y_m - P) / ||y_m - P||            (Algorithm 1, push line: direction of the
 *                                                 pulled point from the reference point)
 *   push    x_m+ = y_m + lambda u_m                            one term (Algorithm 1), or
 *           x_m+ = y_m + lambda (u_m - (1/M) sum_j u_j)        both terms of step (a) of
 *                                                 the regulariser-gradient equation in
 *                                                 Sec. 5 with lambda = lambda_r / M
 *
 * Readings: x_A, x_C and P are the pre-round values for every worker (Jacobi, as in the
 * proof of Theorem 1).  A worker whose pulled point coincides with P has no direction:
 * u_m = 0 (no push for it, and it adds nothing to the mean direction).
 * r_out[m]  = ||x_m - x_A||  before the round (the logged consensus distance),
 * n_out[m]  = ||y_m - P||    (may be NULL).
 * If every r_m is zero (identical replicas) x is copied unchanged.
 */
int dppf_oracle_consensus_general(const float *x, int M, int64_t d, int64_t ld,
                                  float alpha, float lambda, const float *w,
                                  int push_from_c, int two_term,
                                  float *x_out, int64_t ld_out, double *r_out, double *n_out)
{
    if (!x || !x_out || !r_out || M < 1 || d < 1 || ld < d || ld_out < d) return 1;
    double *A = (double *)malloc((size_t)d * sizeof(double));
    double *C = (double *)malloc((size_t)d * sizeof(double));
    double *ubar = (double *)calloc((size_t)d, sizeof(double));
    double *nrm = (double *)malloc((size_t)M * sizeof(double));
    if (!A || !C || !ubar || !nrm) { free(A); free(C); free(ubar); free(nrm); return 2; }
    const double a = (double)alpha, lam = (double)lambda;
    double wsum = 0.0;
    for (int m = 0; m < M; ++m) wsum += w ? (double)w[m] : 1.0;
    if (!(wsum != 0.0)) { free(A); free(C); free(ubar); free(nrm); return 1; }

    for (int64_t i = 0; i < d; ++i) {
        double s = 0.0, c = 0.0;
        for (int m = 0; m < M; ++m) {
            double xi = (double)x[(int64_t)m * ld + i];
            s += xi;
            c += (w ? (double)w[m] : 1.0) * xi;
        }
        A[i] = s / (double)M;
        C[i] = c / wsum;
    }
    const double *P = push_from_c ? C : A;
    int all_zero = 1;
    for (int m = 0; m < M; ++m) {
        const float *xm = x + (int64_t)m * ld;
        double S = 0.0, N = 0.0;
        for (int64_t i = 0; i < d; ++i) {
            double xi = (double)xm[i];
            double dr = xi - A[i];
            S += dr * dr;
            double y = (1.0 - a) * xi + a * C[i];
            double dn = y - P[i];
            N += dn * dn;
        }
        r_out[m] = sqrt(S);
        nrm[m] = sqrt(N);
        if (n_out) n_out[m] = nrm[m];
        if (r_out[m] > 0.0) all_zero = 0;
    }
    if (all_zero) {
        for (int m = 0; m < M; ++m)
            for (int64_t i = 0; i < d; ++i) x_out[(int64_t)m * ld_out + i] = x[(int64_t)m * ld + i];
        free(A); free(C); free(ubar); free(nrm);
        return 0;
    }
    if (two_term) {
        for (int m = 0; m < M; ++m) {
            if (!(nrm[m] > 0.0)) continue;
            const float *xm = x + (int64_t)m * ld;
            for (int64_t i = 0; i < d; ++i) {
                double y = (1.0 - a) * (double)xm[i] + a * C[i];
                ubar[i] += (y - P[i]) / nrm[m];
            }
        }
        for (int64_t i = 0; i < d; ++i) ubar[i] /= (double)M;
    }
    for (int m = 0; m < M; ++m) {
        const float *xm = x + (int64_t)m * ld;
        float *om = x_out + (int64_t)m * ld_out;
        for (int64_t i = 0; i < d; ++i) {
            double y = (1.0 - a) * (double)xm[i] + a * C[i];
            double u = (nrm[m] > 0.0) ? (y - P[i]) / nrm[m] : 0.0;
            om[i] = (float)(y + lam * (u - ubar[i]));      /* ubar is 0 unless two_term */
        }
    }
    free(A); free(C); free(ubar); free(nrm);
    return 0;
}

/*
 * One AdamW local step on an fp64 state, in place.  The ViT experiments (appendix,
 * "Experiments with ViT") train with AdamW, lr 5e-4, weight decay 0.01; the recurrence is
 * not printed in the paper.  The reading used is the standard decoupled form:
 *   x   <- x (1 - lr wd)
 *   m   <- beta1 m + (1 - beta1) g
 *   v   <- beta2 v + (1 - beta2) g^2
 *   x   <- x - lr (m / (1 - beta1^t)) / ( sqrt(v / (1 - beta2^t)) + eps ),   t = step >= 1
 */
int dppf_oracle_adamw_step_f64(double *x, double *m1, double *m2, const float *g,
                               int M, int64_t d, int64_t ld, int64_t ld_g,
                               float lr, float beta1, float beta2, float eps, float weight_decay,
                               int step)
{
    if (!x || !m1 || !m2 || !g || M < 1 || d < 1 || ld < d || ld_g < d || step < 1) return 1;
    const double eta = (double)lr, b1 = (double)beta1, b2 = (double)beta2, e = (double)eps,
                 wd = (double)weight_decay;
    const double bc1 = 1.0 - pow(b1, (double)step), bc2 = 1.0 - pow(b2, (double)step);
    for (int w = 0; w < M; ++w) {
        double *xw = x + (int64_t)w * ld, *aw = m1 + (int64_t)w * ld, *bw = m2 + (int64_t)w * ld;
        const float *gw = g + (int64_t)w * ld_g;
        for (int64_t i = 0; i < d; ++i) {
            double gi = (double)gw[i];
            xw[i] = xw[i] * (1.0 - eta * wd);
            aw[i] = b1 * aw[i] + (1.0 - b1) * gi;
            bw[i] = b2 * bw[i] + (1.0 - b2) * gi * gi;
            xw[i] = xw[i] - eta * (aw[i] / bc1) / (sqrt(bw[i] / bc2) + e);
        }
    }
    return 0;
}
