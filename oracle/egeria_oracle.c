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
 *   - the stale counter and the convergence decision [Algorithm 1];
 *   - the policies stated around Algorithm 1: per-module automatic tolerance,
 *     frontmost-active module, end of the bootstrapping stage [Sec. 3,
 *     Sec. 4.2.2], and unfreezing on learning-rate annealing with the halved
 *     window [Sec. 4.2.2 "Unfreezing"; Algorithm 1, second half].
 *
 * Everything is written out as the definition: no symmetry shortcut, no
 * tiling, no split sums.  Sums run in ascending index order in float64.
 * OpenMP, where enabled, only distributes independent (row) iterations; it
 * never splits a sum.
 *
 * Pins (see tests): closed forms for b = 2 and for one-hot / identical-row
 * inputs, exact rational arithmetic on tiny inputs, a BLAS route, invariants
 * and a negative control, closed-form and pair-wise brute-force slopes,
 * hand-replayed Algorithm 1 traces, and for the policies hand-worked traces
 * plus their reduction to chained runs of the plain rule.  Nothing numerical is printed in the paper
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
 * [Sec. 4.2.2: the smoothed plasticity is fitted with a least-squares line]. n < 2 has no line: +inf. */
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

/* ------------------------------------------------------------------------------------------
 * Policies around Algorithm 1 that the paper states in prose.
 * ------------------------------------------------------------------------------------------ */

/* State of Algorithm 1 for one monitored module, advanced one reading at a time. */
typedef struct {
    double *P;        /* raw readings taken so far */
    double *pl;       /* pList: smoothed readings */
    int64_t len;      /* readings taken */
    int64_t counter;  /* staleCounter */
    double T;         /* tolerance in use (NaN while the automatic one is not set yet) */
    double smax;      /* automatic tolerance: largest |slope| seen in the initial readings */
} module_state;

/* One call of checkPlasticity for a new raw reading [Algorithm 1], with the optional
 * per-module tolerance of Sec. 4.2.2 ("Hyperparameters guideline"): T = 20% of the maximal
 * |slope| in the module's initial 3 readings.  A slope exists from the 2nd reading on, so
 * these are the slopes of evaluations 1 and 2; up to and including evaluation 2 no tolerance
 * is known and the evaluation is never stale.  Returns the slope of this evaluation. */
static double module_advance(module_state *st, double reading, int64_t W, int signed_test, int auto_T) {
    int64_t i = st->len;
    st->P[i] = reading;
    double pbar = egeria_oracle_smooth(st->P, i, W);
    st->pl[i] = pbar;
    st->len = i + 1;
    int64_t n = (st->len < W) ? st->len : W;
    double s = egeria_oracle_ols_slope(st->pl + (st->len - n), n);
    int stale;
    if (auto_T && i <= 2) {
        if (i >= 1 && fabs(s) > st->smax) st->smax = fabs(s);
        if (i == 2) st->T = 0.2 * st->smax;
        stale = 0;
    } else {
        stale = signed_test ? (s < st->T) : (fabs(s) < st->T);
    }
    st->counter = stale ? st->counter + 1 : 0;
    return s;
}

/* Algorithm 1 for one module with the automatic tolerance.  Same outputs as
 * egeria_oracle_plasticity_replay plus the tolerance that was derived (NaN if the history
 * has fewer than 3 readings). */
int egeria_oracle_plasticity_replay_auto(const float *hist, int64_t H, int64_t W, int signed_test,
                                         double *slopes, int32_t *freeze_eval_out, double *T_out) {
    if (H < 0 || W < 1) return -2;
    module_state st;
    st.P = (double *)malloc(sizeof(double) * (size_t)(H > 0 ? H : 1));
    st.pl = (double *)malloc(sizeof(double) * (size_t)(H > 0 ? H : 1));
    if (!st.P || !st.pl) { free(st.P); free(st.pl); return -1; }
    st.len = 0; st.counter = 0; st.T = NAN; st.smax = 0.0;
    int32_t freeze_eval = -1;
    for (int64_t i = 0; i < H; ++i) if (slopes) slopes[i] = NAN;
    for (int64_t i = 0; i < H && st.counter < W; ++i) {
        double s = module_advance(&st, (double)hist[i], W, signed_test, 1);
        if (slopes) slopes[i] = s;
        if (st.counter >= W) freeze_eval = (int32_t)i;
    }
    if (freeze_eval_out) *freeze_eval_out = freeze_eval;
    if (T_out) *T_out = st.T;
    int conv = st.counter >= W;
    free(st.P); free(st.pl);
    return conv;
}

/* The frontmost-active policy [Sec. 4.2.2: only the frontmost module that is still active is
 * monitored, so that the frozen modules always form a prefix; Algorithm 1: freeze, then
 * l <- l + 1].  Modules are ordered front to back.  Only module l = (number of frozen modules) is monitored: evaluation i feeds
 * it hist[l][i]; when its counter reaches W it is frozen at that evaluation and the next
 * evaluation starts module l + 1 from a cleared state.  hist is [M][H] row-major.
 * Outputs: freeze_eval[M] (-1 = not frozen within the history), monitored[H] (module fed at
 * evaluation i, or M when all are frozen), slopes[H] (its slope, NaN when none was fed).
 * T is [M] (ignored when auto_T).  Returns the number of frozen modules, negative on error. */
int egeria_oracle_frontmost_replay(const float *hist, int64_t M, int64_t H, int64_t W, const double *T,
                                   int signed_test, int auto_T, int32_t *freeze_eval,
                                   int32_t *monitored, double *slopes) {
    if (M < 1 || H < 0 || W < 1) return -2;
    module_state st;
    st.P = (double *)malloc(sizeof(double) * (size_t)(H > 0 ? H : 1));
    st.pl = (double *)malloc(sizeof(double) * (size_t)(H > 0 ? H : 1));
    if (!st.P || !st.pl) { free(st.P); free(st.pl); return -1; }
    for (int64_t m = 0; m < M; ++m) freeze_eval[m] = -1;
    int64_t l = 0;
    st.len = 0; st.counter = 0; st.smax = 0.0;
    st.T = auto_T ? NAN : T[0];
    for (int64_t i = 0; i < H; ++i) {
        if (monitored) monitored[i] = (int32_t)l;
        if (slopes) slopes[i] = NAN;
        if (l >= M) continue;
        double s = module_advance(&st, (double)hist[l * H + i], W, signed_test, auto_T);
        if (slopes) slopes[i] = s;
        if (st.counter >= W) {
            freeze_eval[l] = (int32_t)i;
            ++l;
            st.len = 0; st.counter = 0; st.smax = 0.0;
            st.T = (auto_T || l >= M) ? NAN : T[l];
        }
    }
    free(st.P); free(st.pl);
    return (int)l;
}

/* End of the bootstrapping stage [Sec. 3 "Bootstrapping stage": the changing rate of the
 * training loss is watched with the same machinery as the plasticity later on; Sec. 4.2.2: the
 * changing rate that ends the stage is 10%].  The training-loss readings are smoothed [Eq. 2]
 * and fitted like the plasticity; with a full window of W smoothed values, slope s and window
 * mean ybar, the changing rate is |s| (W - 1) / |ybar|: the relative change of the fitted line
 * across the window.  The stage ends at the first evaluation with a full window whose rate is
 * below rate_tol.  rates[H] gets the rate (NaN before the window is full and after the end).
 * Returns the evaluation index at which the stage ended, -1 if it did not, -2 on bad sizes. */
int64_t egeria_oracle_bootstrap_replay(const float *loss, int64_t H, int64_t W, double rate_tol,
                                       double *rates) {
    if (H < 0 || W < 2) return -2;
    double *P = (double *)malloc(sizeof(double) * (size_t)(H > 0 ? H : 1));
    double *pl = (double *)malloc(sizeof(double) * (size_t)(H > 0 ? H : 1));
    if (!P || !pl) { free(P); free(pl); return -2; }
    int64_t end = -1;
    for (int64_t i = 0; i < H; ++i) if (rates) rates[i] = NAN;
    for (int64_t i = 0; i < H && end < 0; ++i) {
        P[i] = (double)loss[i];
        pl[i] = egeria_oracle_smooth(P, i, W);
        if (i + 1 < W) continue;
        const double *y = pl + (i + 1 - W);
        double s = egeria_oracle_ols_slope(y, W);
        double ybar = 0.0;
        for (int64_t k = 0; k < W; ++k) ybar += y[k];
        ybar /= (double)W;
        double rate = fabs(s) * (double)(W - 1) / fabs(ybar);
        if (rates) rates[i] = rate;
        if (rate < rate_tol) end = i;
    }
    free(P); free(pl);
    return end;
}

/* ------------------------------------------------------------------------------------------
 * Unfreezing on learning-rate annealing [Sec. 4.2.2 "Unfreezing"; Algorithm 1, the branch that
 * follows the freeze step: unfreezeAllLayers, l <- l_0].
 *
 * The rule as the paper states it: once the learning rate has fallen by a factor of ten or
 * more since the frontmost layers were frozen, every frozen module is trained again, the
 * monitored module goes back to the first one, and the counter / history-buffer length W is
 * halved for the refreezing.
 *
 * Readings taken where the text leaves room:
 *   - which freeze the drop is counted from: the learning rate in force at the first freeze
 *     after the start or after the last restart is remembered (lr_ref);
 *   - the test runs at the end of every evaluation, after the freeze step, as in Algorithm 1:
 *     restart iff lr_i <= lr_ref / 10 * (1 + 1e-6).  The slack of one part in a million lets a
 *     step decay by exactly 10x count ("decreased by 90%") even when the schedule was computed
 *     in single precision.  A learning rate that is not positive carries no information: it
 *     neither sets lr_ref nor triggers a restart;
 *   - a restart clears every module's raw history, pList and staleCounter (with the automatic
 *     tolerance also the derived T: the initial readings are those after the restart), forgets
 *     lr_ref (nothing is frozen any more) and sets W <- max(2, floor(W / 2)) (a line needs two
 *     points; W = 1 stays 1).  The reading of the evaluation that triggered the restart has
 *     been consumed by the old state; the next evaluation is the first of the new one.
 *
 * hist is [M][H] row-major raw readings, lr is [H] (the learning rate at each evaluation),
 * T is [M] (ignored with auto_T).  frontmost != 0 monitors only the frontmost module that is
 * not frozen (as egeria_oracle_frontmost_replay), else every module runs Algorithm 1 on its own.
 * Outputs (any may be NULL):
 *   slopes[M][H]   slope of module m at evaluation i, NaN where the module was not advanced
 *   frozen[H][M]   1 where module m is frozen after evaluation i (after the unfreezing test)
 *   window[H]      W in force during evaluation i
 *   restarted[H]   1 if the unfreezing fired at the end of evaluation i
 * Returns the number of restarts, negative on error. */
static int64_t halve_window(int64_t W) {
    if (W < 2) return W;
    int64_t h = W / 2;
    return h < 2 ? 2 : h;
}

int egeria_oracle_unfreeze_replay(const float *hist, const double *lr, int64_t M, int64_t H, int64_t W0,
                                  const double *T, int signed_test, int auto_T, int frontmost,
                                  double *slopes, uint8_t *frozen, int32_t *window, int32_t *restarted) {
    if (M < 1 || H < 0 || W0 < 1 || !hist || !lr) return -2;
    module_state *st = (module_state *)calloc((size_t)M, sizeof(module_state));
    uint8_t *is_frozen = (uint8_t *)calloc((size_t)M, 1);
    if (!st || !is_frozen) { free(st); free(is_frozen); return -1; }
    int rc = 0;
    for (int64_t m = 0; m < M; ++m) {
        st[m].P = (double *)malloc(sizeof(double) * (size_t)(H > 0 ? H : 1));
        st[m].pl = (double *)malloc(sizeof(double) * (size_t)(H > 0 ? H : 1));
        if (!st[m].P || !st[m].pl) rc = -1;
    }
    if (rc == 0) {
        int64_t W = W0, l = 0;
        double lr_ref = NAN;
        for (int64_t m = 0; m < M; ++m) {
            st[m].len = 0; st[m].counter = 0; st[m].smax = 0.0;
            st[m].T = auto_T ? NAN : T[m];
        }
        for (int64_t i = 0; i < H; ++i) {
            if (window) window[i] = (int32_t)W;
            if (slopes) for (int64_t m = 0; m < M; ++m) slopes[m * H + i] = NAN;
            int froze_now = 0;
            /* checkPlasticity for the monitored module(s) */
            for (int64_t m = 0; m < M; ++m) {
                if (is_frozen[m]) continue;
                if (frontmost && m != l) continue;
                double s = module_advance(&st[m], (double)hist[m * H + i], W, signed_test, auto_T);
                if (slopes) slopes[m * H + i] = s;
                if (st[m].counter >= W) { is_frozen[m] = 1; froze_now = 1; }
            }
            if (frontmost && l < M && is_frozen[l]) ++l;   /* freezeLayer(l); l <- l + 1 */
            if (froze_now && isnan(lr_ref) && lr[i] > 0.0) lr_ref = lr[i];
            /* learning-rate-based unfreezing */
            int fire = (!isnan(lr_ref) && lr[i] > 0.0 && lr[i] <= lr_ref / 10.0 * (1.0 + 1e-6));
            if (fire) {
                for (int64_t m = 0; m < M; ++m) {          /* unfreezeAllLayers() */
                    is_frozen[m] = 0;
                    st[m].len = 0; st[m].counter = 0; st[m].smax = 0.0;
                    st[m].T = auto_T ? NAN : T[m];
                }
                l = 0;                                      /* l <- l_0 */
                W = halve_window(W);
                lr_ref = NAN;
                ++rc;
            }
            if (restarted) restarted[i] = fire;
            if (frozen) for (int64_t m = 0; m < M; ++m) frozen[i * M + m] = is_frozen[m];
        }
    }
    for (int64_t m = 0; m < M; ++m) { free(st[m].P); free(st[m].pl); }
    free(st); free(is_frozen);
    return rc;
}
