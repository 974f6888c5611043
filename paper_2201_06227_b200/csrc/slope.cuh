// The freezing rule (Sec. 4.2.2, Eq. 2, Algorithm 1) for all modules: moving average
// of the raw plasticity readings, least-squares slope of the last W smoothed values,
// tolerance test, consecutive-stale counter; and the policies the paper states around it:
// the per-module automatic tolerance (Sec. 4.2.2 "Hyperparameters guideline"), the
// frontmost-active policy (Sec. 4.2.2; Algorithm 1 "l <- l + 1"), the learning-rate-based
// unfreezing with the halved window (Sec. 4.2.2 "Unfreezing"; Algorithm 1, second half) and the
// end of the bootstrapping stage (Sec. 3).  One warp per module, float64 throughout.
#pragma once
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

namespace egeria {

enum RuleFlags : int {
    kRuleSigned = 1,     // the literal test of Algorithm 1, slope < T, instead of |slope| < T
    kRuleAutoT = 2,      // T = 20 % of the largest |slope| in the module's initial 3 readings
    kRuleFrontmost = 4,  // only the frontmost module that is not frozen is monitored
};

struct SlopeState {     // per-module arrays (device)
    double *raw;        // [M][W_cap] the last min(n_evals, W) raw readings P_i, oldest first
    double *plist;      // [M][W_cap] the last min(n_evals, W) smoothed readings (tail of pList), oldest first
    int32_t *n_evals;   // [M] readings taken so far (== len(pList))
    int32_t *counter;   // [M] consecutive stale evaluations
    int32_t *freeze_eval;  // [M] evaluation index at which the counter reached W, or -1
    double *last_slope; // [M]
    double *Tauto;      // [M] automatic tolerance (NaN until the third reading)
    double *smax;       // [M] largest |slope| of the initial readings
    unsigned long long *front;  // [1] frontmost policy: (serial of the evaluation that last moved the front) << 32
                                //     | number of frozen modules; one 8-byte word, read and written whole
    const float *T;     // [M] tolerance given at creation
    int32_t W_cap;      // window pitch (the W given at creation)
    // Unfreezing on learning-rate annealing: the window in force lives on the device, because the
    // device halves it when it restarts the modules.
    int32_t *W_cur;     // [1] window in force (<= W_cap)
    unsigned long long *lr_ref;  // [1] bits of the learning rate (double) at the first freeze since the start
                                 //     or the last restart; kLrUnset while nothing has frozen
    int32_t *restarts;  // [1] restarts so far
};

constexpr unsigned long long kLrUnset = 0x7ff8000000000000ull;  // a quiet NaN: "no reference rate"

// W <- max(2, floor(W / 2)): a line needs two points (W = 1 stays 1).
__host__ __device__ inline int halve_window(int W) {
    if (W < 2) return W;
    const int h = W / 2;
    return h < 2 ? 2 : h;
}

__device__ __forceinline__ double warp_sum_f64(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// windowLinearFit: least-squares slope of y(0..n2-1) against x = 0..n2-1; `val(k)` returns
// element k for the k this lane owns (k = lane, lane + 32, ...).  Fewer than 2 points: +inf.
template <class F>
__device__ __forceinline__ double window_slope(int n2, int lane, F val) {
    if (n2 < 2) return INFINITY;
    const double xm = 0.5 * (double)(n2 - 1);
    double sy = 0.0;
    for (int k = lane; k < n2; k += 32) sy += val(k);
    const double ym = warp_sum_f64(sy) / (double)n2;
    double sxy = 0.0, sxx = 0.0;
    for (int k = lane; k < n2; k += 32) {
        const double dx = (double)k - xm;
        sxy += dx * (val(k) - ym);
        sxx += dx * dx;
    }
    sxy = warp_sum_f64(sxy);
    sxx = warp_sum_f64(sxx);
    return sxy / sxx;
}

constexpr int kStepRegs = 4;  // window elements a lane keeps in registers: W <= 128 takes the fast path

// The same fit with the window in registers: this lane holds elements lane + 32 j in y[j].
__device__ __forceinline__ double window_slope_regs(int n2, int lane, const double (&y)[kStepRegs]) {
    if (n2 < 2) return INFINITY;
    const double xm = 0.5 * (double)(n2 - 1);
    double sy = 0.0;
#pragma unroll
    for (int j = 0; j < kStepRegs; ++j)
        if (lane + 32 * j < n2) sy += y[j];
    const double ym = warp_sum_f64(sy) / (double)n2;
    double sxy = 0.0, sxx = 0.0;
#pragma unroll
    for (int j = 0; j < kStepRegs; ++j)
        if (lane + 32 * j < n2) {
            const double dx = (double)(lane + 32 * j) - xm;
            sxy += dx * (y[j] - ym);
            sxx += dx * dx;
        }
    sxy = warp_sum_f64(sxy);
    sxx = warp_sum_f64(sxx);
    return sxy / sxx;
}

// One warp: append reading P to a pair of windows kept oldest-first in memory (global or
// shared), `len` entries each before the call, capacity W.  Eq. 2: the smoothed value is the
// mean of the raw window after the append.  Returns the number of entries after the call and
// the smoothed value and slope of this evaluation.
__device__ __forceinline__ int window_push(double *raw, double *plist, int len, int W, double P, int lane,
                                           double &pbar, double &slope) {
    const bool drop = (len >= W);
    const int n = drop ? W : len + 1;
    if (drop) {  // the oldest entry leaves: shift both windows left by one, 32 entries at a time
        for (int k0 = 0; k0 < W - 1; k0 += 32) {
            const int k = k0 + lane;
            double r = 0.0, q = 0.0;
            if (k < W - 1) {
                r = raw[k + 1];
                q = plist[k + 1];
            }
            __syncwarp();
            if (k < W - 1) {
                raw[k] = r;
                plist[k] = q;
            }
            __syncwarp();
        }
    }
    if (lane == 0) raw[n - 1] = P;
    __syncwarp();
    double s = 0.0;
    for (int k = lane; k < n; k += 32) s += raw[k];
    pbar = warp_sum_f64(s) / (double)n;
    if (lane == 0) plist[n - 1] = pbar;
    __syncwarp();
    slope = window_slope(n, lane, [&](int k) { return plist[k]; });
    return n;
}

// Is evaluation i with this slope stale?  With the automatic tolerance the module's initial 3
// readings (evaluations 0..2) only set it and are never stale.  NaN compares false: never stale.
__device__ __forceinline__ bool rule_is_stale(double slope, int i, int flags, double T_fixed, double &Tauto,
                                              double &smax) {
    double T = T_fixed;
    if (flags & kRuleAutoT) {
        if (i <= 2) {
            if (i >= 1 && fabs(slope) > smax) smax = fabs(slope);
            if (i == 2) Tauto = 0.2 * smax;
            return false;
        }
        T = Tauto;
    }
    return (flags & kRuleSigned) ? (slope < T) : (fabs(slope) < T);
}

// The two windows are kept oldest-first at fixed addresses, so for W <= 128 every load of the
// step (counters, both windows, and both windows shifted by one for the case that the oldest
// entry drops out) is issued at once: one memory round trip, then arithmetic in registers.
struct StepLoaded {
    double ra[kStepRegs], rb[kStepRegs], pa[kStepRegs], pb[kStepRegs];
    double slope, T, Tauto, smax;
    int i, counter, freeze_eval;
    int W;  // window in force
};

// Issue every load of one step of module m (nothing here depends on the new reading).
__device__ __forceinline__ StepLoaded plasticity_step_load(const SlopeState &st, int m, int lane) {
    StepLoaded L;
    const double *raw = st.raw + (int64_t)m * st.W_cap, *plist = st.plist + (int64_t)m * st.W_cap;
    const int Wc = st.W_cap;  // the window in force is at most this; what lies beyond it is never used
    if (Wc <= 32 * kStepRegs) {
#pragma unroll
        for (int j = 0; j < kStepRegs; ++j) {
            const int k = lane + 32 * j;
            L.ra[j] = (k < Wc) ? raw[k] : 0.0;
            L.pa[j] = (k < Wc) ? plist[k] : 0.0;
            L.rb[j] = (k + 1 < Wc) ? raw[k + 1] : 0.0;
            L.pb[j] = (k + 1 < Wc) ? plist[k + 1] : 0.0;
        }
    }
    L.W = *st.W_cur;
    L.i = st.n_evals[m];  // readings taken before this one == index of this evaluation
    L.counter = st.counter[m];
    L.freeze_eval = st.freeze_eval[m];
    L.slope = st.last_slope[m];
    L.Tauto = st.Tauto[m];
    L.smax = st.smax[m];
    L.T = (double)st.T[m];
    return L;
}

// One new reading for module m, by one warp: Algorithm 1 on the context's state.  Returns
// whether the module is converged after this evaluation; `slope_out` is the slope of this
// evaluation (the last one if the module had converged before).  `lr` is the learning rate in
// force (not positive or NaN: unknown): the first module to freeze records it as the reference
// rate of the unfreezing rule.
__device__ __forceinline__ bool plasticity_step_apply(const SlopeState &st, StepLoaded &L, int m, int flags,
                                                      float reading, double lr, int lane, double &slope_out) {
    double *raw = st.raw + (int64_t)m * st.W_cap, *plist = st.plist + (int64_t)m * st.W_cap;
    const int W = L.W;
    const bool fast = (st.W_cap <= 32 * kStepRegs);
    double(&ra)[kStepRegs] = L.ra, (&rb)[kStepRegs] = L.rb, (&pa)[kStepRegs] = L.pa, (&pb)[kStepRegs] = L.pb;
    const int i = L.i;
    int counter = L.counter, freeze_eval = L.freeze_eval;
    double slope = L.slope;
    __syncwarp();
    if (counter < W) {
        const int len = (i < W) ? i : W;       // entries in the windows now
        const double P = (double)reading;
        if (fast) {
            const bool drop = (len == W);      // the oldest entry leaves
            const int n = drop ? W : len + 1;  // entries after this reading: min(i + 1, W)
            // windows after the update, in registers: element k = lane + 32 j
#pragma unroll
            for (int j = 0; j < kStepRegs; ++j) {
                const int k = lane + 32 * j;
                ra[j] = (k == n - 1) ? P : (drop ? rb[j] : ra[j]);
                pa[j] = drop ? pb[j] : pa[j];
            }
            double s = 0.0;  // Eq. 2: mean of the last min(i + 1, W) raw readings
#pragma unroll
            for (int j = 0; j < kStepRegs; ++j)
                if (lane + 32 * j < n) s += ra[j];
            const double pbar = warp_sum_f64(s) / (double)n;
#pragma unroll
            for (int j = 0; j < kStepRegs; ++j)
                if (lane + 32 * j == n - 1) pa[j] = pbar;
            slope = window_slope_regs(n, lane, pa);
#pragma unroll
            for (int j = 0; j < kStepRegs; ++j) {
                const int k = lane + 32 * j;
                if (k < n && (drop || k == n - 1)) {
                    raw[k] = ra[j];
                    plist[k] = pa[j];
                }
            }
        } else {
            double pbar;
            window_push(raw, plist, len, W, P, lane, pbar, slope);
        }
        const bool stale = rule_is_stale(slope, i, flags, L.T, L.Tauto, L.smax);
        counter = stale ? counter + 1 : 0;
        if (counter >= W && freeze_eval < 0) {
            freeze_eval = i;
            // every freeze of one evaluation carries the same rate, so who wins does not matter
            if (lane == 0 && lr > 0.0) atomicCAS(st.lr_ref, kLrUnset, (unsigned long long)__double_as_longlong(lr));
        }
        if (lane == 0) {
            st.n_evals[m] = i + 1;
            st.counter[m] = counter;
            st.freeze_eval[m] = freeze_eval;
            st.last_slope[m] = slope;
            if (flags & kRuleAutoT) {
                st.Tauto[m] = L.Tauto;
                st.smax[m] = L.smax;
            }
        }
    }
    slope_out = slope;
    return counter >= W;
}

// One evaluation of the rule as module m's warp sees it (all modules' warps call this, each
// with its own new reading).  Without the frontmost policy every module advances and reports
// for itself.  With it, only the frontmost module that is not frozen advances; its warp (the
// last module's when all are frozen) also reports for everybody: mask[j] = j is frozen,
// slopes[j] = the slope of this evaluation for the monitored module, the final slope of a
// frozen one, +inf for one that has not been monitored yet.  `serial` numbers the evaluations
// (from 1): a front that moved during evaluation `serial` is left alone for the rest of it,
// so the module that becomes the front starts with the next evaluation.
__device__ __forceinline__ void plasticity_rule_step(const SlopeState &st, StepLoaded &L, int m, int M, int flags,
                                                     uint32_t serial, float reading, double lr, double *out_slopes,
                                                     uint8_t *out_mask, int lane) {
    if (!(flags & kRuleFrontmost)) {
        double slope;
        const bool conv = plasticity_step_apply(st, L, m, flags, reading, lr, lane, slope);
        if (lane == 0) {
            if (out_slopes) out_slopes[m] = slope;
            if (out_mask) out_mask[m] = conv ? 1 : 0;
        }
        return;
    }
    const unsigned long long word = *reinterpret_cast<volatile unsigned long long *>(st.front);
    if ((uint32_t)(word >> 32) == serial) return;  // the front moved in this evaluation: it has been dealt with
    const int front = (int)(uint32_t)word;
    const int reporter = front < M ? front : M - 1;
    if (m != reporter) return;
    int front_new = front;
    double slope = INFINITY;
    if (front < M) {
        const bool conv = plasticity_step_apply(st, L, m, flags, reading, lr, lane, slope);
        if (conv) front_new = front + 1;
    }
    if (lane == 0 && front_new != front)
        *reinterpret_cast<volatile unsigned long long *>(st.front) =
            ((unsigned long long)serial << 32) | (unsigned long long)(uint32_t)front_new;
    for (int j = lane; j < M; j += 32) {
        if (out_mask) out_mask[j] = (j < front_new) ? 1 : 0;
        if (out_slopes) out_slopes[j] = (j == m && front < M) ? slope : (j < front ? st.last_slope[j] : INFINITY);
    }
}

// One new reading per module.  grid = M warps (one 32-thread block each).
__global__ void __launch_bounds__(32) plasticity_step_kernel(SlopeState st, int M, int flags, uint32_t serial,
                                                             double lr, const float *losses, double *out_slopes,
                                                             uint8_t *out_mask) {
    const int m = blockIdx.x, lane = threadIdx.x;
    if (m >= M) return;
    StepLoaded L = plasticity_step_load(st, m, lane);
    plasticity_rule_step(st, L, m, M, flags, serial, losses[m], lr, out_slopes, out_mask, lane);
}

// The unfreezing test of Algorithm 1 [Sec. 4.2.2 "Unfreezing"], run after the evaluation whose
// learning rate `lr` differs from the previous one's (the test cannot change its mind while the
// rate stands still).  If the rate has fallen to a tenth, or less, of the rate at the first freeze
// (one part in a million of slack, so that a step decay by exactly 10x counts even when it was
// computed in single precision): every module starts afresh, the front goes back to module 0,
// the window is halved and the reference rate is forgotten; the mask of the evaluation that
// just ran is cleared.  One block.
__global__ void unfreeze_check_kernel(SlopeState st, int M, double lr, uint8_t *out_mask) {
    __shared__ int fire;
    if (threadIdx.x == 0) {
        const unsigned long long bits = *st.lr_ref;
        const double ref = __longlong_as_double((long long)bits);
        fire = (bits != kLrUnset && lr > 0.0 && lr <= ref / 10.0 * (1.0 + 1e-6)) ? 1 : 0;
    }
    __syncthreads();
    if (!fire) return;
    for (int m = threadIdx.x; m < M; m += blockDim.x) {
        st.n_evals[m] = 0;
        st.counter[m] = 0;
        st.freeze_eval[m] = -1;
        st.last_slope[m] = INFINITY;
        st.Tauto[m] = NAN;
        st.smax[m] = 0.0;
        if (out_mask) out_mask[m] = 0;
    }
    if (threadIdx.x == 0) {
        *st.front = 0ull;
        *st.lr_ref = kLrUnset;
        *st.W_cur = halve_window(*st.W_cur);
        *st.restarts += 1;
    }
}

// Whole histories from a cleared private state (windows in shared memory: 2 * W doubles).
// Without the frontmost policy: one warp per module (grid = M).  With it: one warp in all
// (grid = 1) walks the modules front to back.  out_slopes[m][i] is NaN where module m was
// not advanced at evaluation i.
__global__ void __launch_bounds__(32) plasticity_replay_kernel(const float *T, int M, const int32_t *W_cur, int W_cap,
                                                               int flags, const float *hist, int H,
                                                               double *out_slopes, uint8_t *out_mask,
                                                               int32_t *out_freeze_eval) {
    extern __shared__ double windows[];
    const int W = *W_cur;  // the window in force (<= W_cap, which sizes the shared memory)
    double *raw = windows, *plist = windows + W_cap;
    const int lane = threadIdx.x;
    const bool frontmost = (flags & kRuleFrontmost) != 0;
    int m = frontmost ? 0 : (int)blockIdx.x;
    if (m >= M) return;
    if (frontmost) {
        for (int64_t k = lane; k < (int64_t)M * H; k += 32)
            if (out_slopes) out_slopes[k] = NAN;
        for (int j = lane; j < M; j += 32) {
            if (out_mask) out_mask[j] = 0;
            if (out_freeze_eval) out_freeze_eval[j] = -1;
        }
        __syncwarp();
    }
    int len = 0, n_evals = 0, counter = 0, freeze_eval = -1;
    double Tauto = NAN, smax = 0.0;
    for (int i = 0; i < H && m < M; ++i) {
        double slope = NAN;
        if (counter < W) {
            double pbar;
            len = window_push(raw, plist, len, W, (double)hist[(int64_t)m * H + i], lane, pbar, slope);
            const bool stale = rule_is_stale(slope, n_evals, flags, (double)T[m], Tauto, smax);
            counter = stale ? counter + 1 : 0;
            if (counter >= W) freeze_eval = i;
            ++n_evals;
        }
        if (out_slopes && lane == 0) out_slopes[(int64_t)m * H + i] = slope;
        if (frontmost && counter >= W) {  // frozen: the next evaluation starts the next module afresh
            if (lane == 0) {
                if (out_mask) out_mask[m] = 1;
                if (out_freeze_eval) out_freeze_eval[m] = freeze_eval;
            }
            ++m;
            len = n_evals = counter = 0;
            freeze_eval = -1;
            Tauto = NAN;
            smax = 0.0;
            __syncwarp();
        }
    }
    if (!frontmost && lane == 0) {
        if (out_mask) out_mask[m] = (counter >= W) ? 1 : 0;
        if (out_freeze_eval) out_freeze_eval[m] = freeze_eval;
    }
}

// Whole histories with the learning-rate-based unfreezing [Sec. 4.2.2 "Unfreezing"; Algorithm 1,
// second half], from a cleared state private to the call.  A restart couples the modules (any
// freeze arms it, every module is cleared by it), so one block runs all of them: warp w takes
// modules w, w + warps, ...; after every evaluation thread 0 moves the front, remembers the rate
// of the first freeze and takes the unfreezing decision for everybody.  The windows are in global
// scratch ([M][W_cap] each), the per-module scalars in shared memory (M * sizeof(ReplayModule)).
struct ReplayModule {
    int32_t len, n_evals, counter, frozen;
    double Tauto, smax;
};

__global__ void __launch_bounds__(1024) plasticity_replay_lr_kernel(
    const float *T, double *raw_all, double *plist_all, int W_cap, const int32_t *W_start, int M, int flags,
    const float *hist, const double *lr, int H, double *out_slopes, uint8_t *out_frozen, int32_t *out_window,
    uint8_t *out_restarted, uint8_t *out_mask, int32_t *out_freeze_eval) {
    extern __shared__ double replay_smem[];
    ReplayModule *mod = reinterpret_cast<ReplayModule *>(replay_smem);
    __shared__ int s_W, s_front, s_froze_now, s_fire;
    __shared__ unsigned long long s_lr_ref;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    const bool frontmost = (flags & kRuleFrontmost) != 0;
    for (int m = threadIdx.x; m < M; m += blockDim.x) {
        mod[m] = ReplayModule{0, 0, 0, 0, NAN, 0.0};
        if (out_freeze_eval) out_freeze_eval[m] = -1;
    }
    if (threadIdx.x == 0) {
        s_W = *W_start;
        s_front = 0;
        s_lr_ref = kLrUnset;
    }
    __syncthreads();
    for (int i = 0; i < H; ++i) {
        if (threadIdx.x == 0) {
            s_froze_now = 0;
            s_fire = 0;
            if (out_window) out_window[i] = s_W;
        }
        __syncthreads();
        const int W = s_W, front = s_front;
        for (int m = warp; m < M; m += n_warps) {
            ReplayModule &st = mod[m];
            double slope = NAN;
            if (!st.frozen && (!frontmost || m == front)) {
                double pbar;
                st.len = window_push(raw_all + (int64_t)m * W_cap, plist_all + (int64_t)m * W_cap, st.len, W,
                                     (double)hist[(int64_t)m * H + i], lane, pbar, slope);
                double Tauto = st.Tauto, smax = st.smax;
                const bool stale = rule_is_stale(slope, st.n_evals, flags, (double)T[m], Tauto, smax);
                __syncwarp();
                if (lane == 0) {
                    st.Tauto = Tauto;
                    st.smax = smax;
                    st.counter = stale ? st.counter + 1 : 0;
                    st.n_evals += 1;
                    if (st.counter >= W) {
                        st.frozen = 1;
                        s_froze_now = 1;
                        if (out_freeze_eval) out_freeze_eval[m] = i;
                    }
                }
                __syncwarp();
            }
            if (out_slopes && lane == 0) out_slopes[(int64_t)m * H + i] = slope;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            if (frontmost && s_front < M && mod[s_front].frozen) s_front += 1;  // freezeLayer(l); l <- l + 1
            const double rate = lr ? lr[i] : NAN;
            if (s_froze_now && s_lr_ref == kLrUnset && rate > 0.0)
                s_lr_ref = (unsigned long long)__double_as_longlong(rate);
            const double ref = __longlong_as_double((long long)s_lr_ref);
            if (s_lr_ref != kLrUnset && rate > 0.0 && rate <= ref / 10.0 * (1.0 + 1e-6)) {
                s_fire = 1;
                s_front = 0;
                s_W = halve_window(s_W);
                s_lr_ref = kLrUnset;
            }
            if (out_restarted) out_restarted[i] = (uint8_t)s_fire;
        }
        __syncthreads();
        for (int m = threadIdx.x; m < M; m += blockDim.x) {
            if (s_fire) {
                mod[m] = ReplayModule{0, 0, 0, 0, NAN, 0.0};
                if (out_freeze_eval) out_freeze_eval[m] = -1;
            }
            if (out_frozen) out_frozen[(int64_t)i * M + m] = (uint8_t)mod[m].frozen;
        }
        __syncthreads();
    }
    for (int m = threadIdx.x; m < M; m += blockDim.x)
        if (out_mask) out_mask[m] = (uint8_t)mod[m].frozen;
}

// Clear the rule state of every module.  set_W > 0: the window in force becomes set_W (context
// creation); else, if halve != 0, it is halved.
__global__ void plasticity_clear_kernel(SlopeState st, int M, int set_W, int halve) {
    const int m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m == 0) {
        *st.front = 0ull;
        *st.lr_ref = kLrUnset;
        if (set_W > 0) {
            *st.W_cur = set_W;
            *st.restarts = 0;
        } else if (halve) {
            *st.W_cur = halve_window(*st.W_cur);
        }
    }
    if (m >= M) return;
    st.n_evals[m] = 0;
    st.counter[m] = 0;
    st.freeze_eval[m] = -1;
    st.last_slope[m] = INFINITY;
    st.Tauto[m] = NAN;
    st.smax[m] = 0.0;
}

// ------------------------------------------------------------------------------------------
// End of the bootstrapping stage (Sec. 3; the 10 % of Sec. 4.2.2): the training loss is
// smoothed and fitted like the plasticity; with a full window of W smoothed values, slope s
// and window mean ybar, the changing rate is |s| (W - 1) / |ybar|, and the stage ends at the
// first evaluation whose rate is below the tolerance.
// ------------------------------------------------------------------------------------------
struct BootState {
    double *raw;       // [W_cap] raw training losses, oldest first
    double *plist;     // [W_cap] smoothed ones
    int32_t *n_evals;  // [1]
    int32_t *end;      // [1] evaluation at which the stage ended, -1 while it lasts
};

// One warp: one more training loss.  Returns the changing rate of this evaluation (NaN before
// the window is full and after the end); `end` is updated.
__device__ __forceinline__ double bootstrap_advance(double *raw, double *plist, int &n_evals, int &end, double loss,
                                                    int W, double rate_tol, int lane) {
    if (end >= 0) return NAN;
    const int len = n_evals < W ? n_evals : W;
    double pbar, slope;
    const int n = window_push(raw, plist, len, W, loss, lane, pbar, slope);
    const int i = n_evals++;
    if (n < W) return NAN;
    double sy = 0.0;
    for (int k = lane; k < W; k += 32) sy += plist[k];
    const double ybar = warp_sum_f64(sy) / (double)W;
    const double rate = fabs(slope) * (double)(W - 1) / fabs(ybar);
    if (rate < rate_tol) end = i;
    return rate;
}

__global__ void __launch_bounds__(32) bootstrap_step_kernel(BootState bs, int W, double rate_tol, const float *loss,
                                                            double *out_rate, uint8_t *out_done) {
    const int lane = threadIdx.x;
    int n_evals = *bs.n_evals, end = *bs.end;
    __syncwarp();
    const double rate = bootstrap_advance(bs.raw, bs.plist, n_evals, end, (double)*loss, W, rate_tol, lane);
    if (lane == 0) {
        *bs.n_evals = n_evals;
        *bs.end = end;
        if (out_rate) *out_rate = rate;
        if (out_done) *out_done = end >= 0 ? 1 : 0;
    }
}

// A whole training-loss history from a cleared private state (2 * W doubles of shared memory).
__global__ void __launch_bounds__(32) bootstrap_replay_kernel(int W, double rate_tol, const float *hist, int H,
                                                              double *out_rates, int32_t *out_end) {
    extern __shared__ double windows[];
    const int lane = threadIdx.x;
    int n_evals = 0, end = -1;
    for (int i = 0; i < H; ++i) {
        const double rate = bootstrap_advance(windows, windows + W, n_evals, end, (double)hist[i], W, rate_tol, lane);
        if (out_rates && lane == 0) out_rates[i] = rate;
    }
    if (out_end && lane == 0) *out_end = end;
}

__global__ void bootstrap_clear_kernel(BootState bs) {
    *bs.n_evals = 0;
    *bs.end = -1;
}

}  // namespace egeria
