/*
 * Float64 CPU oracle for the Egeria plasticity-evaluation path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the CUDA
 * library is checked against.  It shares no code with the CUDA path, is never
 * linked into it, and must only be used by the tests, the smoke check and the
 * benchmark's CPU-baseline leg.
 *
 * What it computes (paper sections in brackets):
 *   - SP loss between the training and the reference activations of one layer
 *     module, the paper's plasticity P_i^(l) [Sec. 4.2.1, Eq. 1]: each
 *     activation tensor is flattened per sample to b x d, mapped to its b x b
 *     pair-wise similarity matrix G = A A^T, every row of G is scaled to unit
 *     L2 norm, and the loss is the squared Frobenius distance of the two
 *     normalised matrices divided by b^2.  (Eq. 1 only names the SP loss; the
 *     formula is the similarity-preserving loss the paper cites for it.)
 *   - the moving average of the raw plasticity readings [Sec. 4.2.2, Eq. 2],
 *     read as the mean of the last min(i+1, W) readings;
 *   - the least-squares straight-line fit of the last min(len, W) smoothed
 *     values against the evaluation index, and its slope [Sec. 4.2.2,
 *     Algorithm 1 "windowLinearFit"];
 *   - the stale counter and the convergence decision [Algorithm 1].
 *
 * Everything is written out as the definition: no symmetry shortcut, no
 * tiling, no split sums.  Sums run in ascending index order in float64.
 * OpenMP, where enabled, only distributes independent (row) iterations; it
 * never splits a sum.
 *
 * Pins (see tests): closed forms for b = 2 and for one-hot / identical-row
 * inputs, exact rational arithmetic on tiny inputs, a BLAS route, invariants
 * and a negative control, closed-form and pair-wise brute-force slopes, and
 * hand-replayed Algorithm 1 traces.  Nothing numerical is printed in the paper
 * for this path, so no value here is pinned to a number of the paper's own.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* bfloat16 bits -> double (exact): bf16 is the upper half of an IEEE float. */
static double bf16_to_f64(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int egeria_oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void egeria_oracle_set_num_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* Step 1: widen a b x d bf16 matrix (row-major) to float64. */
void egeria_oracle_widen(const uint16_t *A, int64_t b, int64_t d, double *X) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < b; ++i)
        for (int64_t k = 0; k < d; ++k) X[i * d + k] = bf16_to_f64(A[i * d + k]);
}

/* Pair-wise similarity matrix [Sec. 4.2.1]: G[i][j] = sum_k X[i][k] X[j][k],
 * all b*b entries, k ascending. */
void egeria_oracle_gram_f64(const double *X, int64_t b, int64_t d, double *G) {
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t i = 0; i < b; ++i) {
        for (int64_t j = 0; j < b; ++j) {
            const double *xi = X + i * d, *xj = X + j * d;
            double acc = 0.0;
            for (int64_t k = 0; k < d; ++k) acc += xi[k] * xj[k];
            G[i * b + j] = acc;
        }
    }
}

/* Same, from bf16 bits. Returns 0, or -1 if the scratch could not be had. */
int egeria_oracle_gram(const uint16_t *A, int64_t b, int64_t d, double *G) {
    double *X = (double *)malloc(sizeof(double) * (size_t)(b * d > 0 ? b * d : 1));
    if (!X) return -1;
    egeria_oracle_widen(A, b, d, X);
    egeria_oracle_gram_f64(X, b, d, G);
    free(X);
    return 0;
}

/* One row of G only (for sampled checks at sizes where b*b dots are too slow). */
int egeria_oracle_gram_row(const uint16_t *A, int64_t b, int64_t d, int64_t i, double *Grow) {
    if (i < 0 || i >= b) return -2;
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < b; ++j) {
        double acc = 0.0;
        for (int64_t k = 0; k < d; ++k)
            acc += bf16_to_f64(A[i * d + k]) * bf16_to_f64(A[j * d + k]);
        Grow[j] = acc;
    }
    return 0;
}

/* Row L2 normalisation: Gn[i][:] = G[i][:] / max(||G[i][:]||_2, eps). */
void egeria_oracle_row_normalise(const double *G, int64_t b, double eps, double *Gn) {
    for (int64_t i = 0; i < b; ++i) {
        double ss = 0.0;
        for (int64_t j = 0; j < b; ++j) ss += G[i * b + j] * G[i * b + j];
        double n = sqrt(ss);
        if (n < eps) n = eps;
        for (int64_t j = 0; j < b; ++j) Gn[i * b + j] = G[i * b + j] / n;
    }
}

/* SP loss from two normalised b x b matrices [Eq. 1]:
 * (1/b^2) sum_ij (Gt[i][j] - Gr[i][j])^2, row-major order. */
double egeria_oracle_frobenius_loss(const double *Gtn, const double *Grn, int64_t b) {
    double s = 0.0;
    for (int64_t i = 0; i < b; ++i)
        for (int64_t j = 0; j < b; ++j) {
            double diff = Gtn[i * b + j] - Grn[i * b + j];
            s += diff * diff;
        }
    return s / ((double)b * (double)b);
}

/* Plasticity of one module [Eq. 1]. Optionally returns the two normalised
 * similarity matrices (b*b doubles each; pass NULL to skip).
 * Returns 0 on success, -1 on allocation failure, -2 on bad sizes. */
int egeria_oracle_sp_loss(const uint16_t *At, const uint16_t *Ar, int64_t b, int64_t d,
                          double eps, double *loss, double *Gtn_out, double *Grn_out) {
    if (b < 1 || d < 0 || !loss) return -2;
    size_t bb = (size_t)(b * b);
    double *G = (double *)malloc(sizeof(double) * bb);
    double *Gtn = Gtn_out ? Gtn_out : (double *)malloc(sizeof(double) * bb);
    double *Grn = Grn_out ? Grn_out : (double *)malloc(sizeof(double) * bb);
    int rc = 0;
    if (!G || !Gtn || !Grn) { rc = -1; goto done; }
    if (egeria_oracle_gram(At, b, d, G)) { rc = -1; goto done; }
    egeria_oracle_row_normalise(G, b, eps, Gtn);
    if (egeria_oracle_gram(Ar, b, d, G)) { rc = -1; goto done; }
    egeria_oracle_row_normalise(G, b, eps, Grn);
    *loss = egeria_oracle_frobenius_loss(Gtn, Grn, b);
done:
    free(G);
    if (!Gtn_out) free(Gtn);
    if (!Grn_out) free(Grn);
    return rc;
}

/* All monitored modules of one evaluation, one after another. */
int egeria_oracle_sp_loss_batch(int M, const uint16_t *const *At, const uint16_t *const *Ar,
                                int64_t b, const int64_t *d, double eps, double *losses) {
    for (int m = 0; m < M; ++m) {
        int rc = egeria_oracle_sp_loss(At[m], Ar[m], b, d[m], eps, &losses[m], NULL, NULL);
        if (rc) return rc;
    }
    return 0;
}

/* Moving average [Eq. 2]: mean of the last min(i+1, W) raw readings P[0..i]. */
double egeria_oracle_smooth(const double *P, int64_t i, int64_t W) {
    int64_t n = (i + 1 < W) ? i + 1 : W;
    double s = 0.0;
    for (int64_t k = i - n + 1; k <= i; ++k) s += P[k];
    return s / (double)n;
}

/* Ordinary least squares slope of y[0..n-1] against x = 0..n-1
 * [Sec. 4.2.2 "linear least-squares regression"]. n < 2 has no line: +inf. */
double egeria_oracle_ols_slope(const double *y, int64_t n) {
    if (n < 2) return INFINITY;
    double xm = 0.0, ym = 0.0;
    for (int64_t k = 0; k < n; ++k) { xm += (double)k; ym += y[k]; }
    xm /= (double)n;
    ym /= (double)n;
    double sxy = 0.0, sxx = 0.0;
    for (int64_t k = 0; k < n; ++k) {
        sxy += ((double)k - xm) * (y[k] - ym);
        sxx += ((double)k - xm) * ((double)k - xm);
    }
    return sxy / sxx;
}

/* Algorithm 1 for one module over a whole history of H raw readings.
 *
 *   for i = 0..H-1, while staleCounter < W:
 *       Pbar_i = smooth(P, i, W); pList += Pbar_i
 *       s_i = slope of the last min(len(pList), W) entries of pList
 *       stale = signed_test ? (s_i < T) : (|s_i| < T)   (NaN is never stale)
 *       staleCounter = stale ? staleCounter + 1 : 0
 *       if staleCounter reaches W: converged, freeze_eval = i, state stops.
 *
 * Outputs (any may be NULL): smoothed[H], slopes[H] (entries after convergence
 * are NaN), final counter, freeze_eval (-1 if never).  Returns 1 if the module
 * converged within the history, 0 if not, negative on error. */
int egeria_oracle_plasticity_replay(const float *hist, int64_t H, int64_t W, double T,
                                    int signed_test, double *smoothed, double *slopes,
                                    int32_t *counter_out, int32_t *freeze_eval_out) {
    if (H < 0 || W < 1) return -2;
    double *P = (double *)malloc(sizeof(double) * (size_t)(H > 0 ? H : 1));
    double *pl = (double *)malloc(sizeof(double) * (size_t)(H > 0 ? H : 1));
    if (!P || !pl) { free(P); free(pl); return -1; }
    int64_t counter = 0, len = 0;
    int32_t freeze_eval = -1;
    for (int64_t i = 0; i < H; ++i) {
        if (smoothed) smoothed[i] = NAN;
        if (slopes) slopes[i] = NAN;
    }
    for (int64_t i = 0; i < H; ++i) {
        if (counter >= W) break;
        P[i] = (double)hist[i];
        double pbar = egeria_oracle_smooth(P, i, W);
        pl[len++] = pbar;
        int64_t n = (len < W) ? len : W;
        double s = egeria_oracle_ols_slope(pl + (len - n), n);
        int stale = signed_test ? (s < T) : (fabs(s) < T);
        counter = stale ? counter + 1 : 0;
        if (smoothed) smoothed[i] = pbar;
        if (slopes) slopes[i] = s;
        if (counter >= W) freeze_eval = (int32_t)i;
    }
    if (counter_out) *counter_out = (int32_t)counter;
    if (freeze_eval_out) *freeze_eval_out = freeze_eval;
    free(P);
    free(pl);
    return counter >= W ? 1 : 0;
}
