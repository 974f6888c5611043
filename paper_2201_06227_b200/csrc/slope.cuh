// The freezing rule (Sec. 4.2.2, Eq. 2, Algorithm 1) for all modules: moving average
// of the raw plasticity readings, least-squares slope of the last W smoothed values,
// tolerance test, consecutive-stale counter.  One warp per module, float64 throughout.
#pragma once
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

namespace egeria {

struct SlopeState {     // per-module arrays (device)
    double *raw;        // [M][W_cap] the last min(n_evals, W) raw readings P_i, oldest first
    double *plist;      // [M][W_cap] the last min(n_evals, W) smoothed readings (tail of pList), oldest first
    int32_t *n_evals;   // [M] readings taken so far (== len(pList))
    int32_t *counter;   // [M] consecutive stale evaluations
    int32_t *freeze_eval;  // [M] evaluation index at which the counter reached W, or -1
    double *last_slope; // [M]
    const float *T;     // [M] tolerance
    int32_t W_cap;      // ring pitch
};

__device__ __forceinline__ double warp_sum_f64(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// One evaluation of one module by one warp.  raw/plist are this module's rings of pitch
// >= W (global or shared memory).  Returns the slope of this evaluation (all lanes).
__device__ __forceinline__ double plasticity_advance(double *raw, double *plist, int &n_evals, int &counter,
                                                     int &freeze_eval, double reading, int W, double T,
                                                     bool signed_test, int lane) {
    const int i = n_evals;
    if (lane == 0) raw[i % W] = reading;
    __syncwarp();
    // Eq. 2: mean of the last min(i + 1, W) raw readings
    const int n = (i + 1 < W) ? i + 1 : W;
    double s = 0.0;
    for (int k = lane; k < n; k += 32) s += raw[(i - n + 1 + k) % W];
    const double pbar = warp_sum_f64(s) / (double)n;
    if (lane == 0) plist[i % W] = pbar;
    __syncwarp();
    // windowLinearFit: least squares over the last min(len, W) entries of pList, x = 0..n2-1
    const int len = i + 1;
    const int n2 = (len < W) ? len : W;
    double slope;
    if (n2 < 2) {
        slope = INFINITY;
    } else {
        const double xm = 0.5 * (double)(n2 - 1);
        double sy = 0.0;
        for (int k = lane; k < n2; k += 32) sy += plist[(len - n2 + k) % W];
        const double ym = warp_sum_f64(sy) / (double)n2;
        double sxy = 0.0, sxx = 0.0;
        for (int k = lane; k < n2; k += 32) {
            const double dx = (double)k - xm;
            sxy += dx * (plist[(len - n2 + k) % W] - ym);
            sxx += dx * dx;
        }
        sxy = warp_sum_f64(sxy);
        sxx = warp_sum_f64(sxx);
        slope = sxy / sxx;
    }
    const bool stale = signed_test ? (slope < T) : (fabs(slope) < T);  // NaN compares false
    counter = stale ? counter + 1 : 0;
    if (counter >= W && freeze_eval < 0) freeze_eval = i;
    n_evals = i + 1;
    return slope;
}

// Smoothing (Eq. 2), window fit and counter update of Algorithm 1 for one new reading, given
// the module's two windows AFTER the new values are in place.  `val(k)` returns element k of
// the smoothed window (k = 0 oldest) for the k this lane owns (k = lane, lane + 32, ...).
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

// One new reading for module m, by one warp: Algorithm 1 on the context's state.
// The two windows are kept oldest-first at fixed addresses, so for W <= 128 every load of the
// step (counters, both windows, and both windows shifted by one for the case that the oldest
// entry drops out) is issued at once: one memory round trip, then arithmetic in registers.
struct StepLoaded {
    double ra[kStepRegs], rb[kStepRegs], pa[kStepRegs], pb[kStepRegs];
    double slope, T;
    int i, counter, freeze_eval;
};

// Issue every load of one step of module m (nothing here depends on the new reading).
__device__ __forceinline__ StepLoaded plasticity_step_load(const SlopeState &st, int m, int W, int lane) {
    StepLoaded L;
    const double *raw = st.raw + (int64_t)m * st.W_cap, *plist = st.plist + (int64_t)m * st.W_cap;
    if (W <= 32 * kStepRegs) {
#pragma unroll
        for (int j = 0; j < kStepRegs; ++j) {
            const int k = lane + 32 * j;
            L.ra[j] = (k < W) ? raw[k] : 0.0;
            L.pa[j] = (k < W) ? plist[k] : 0.0;
            L.rb[j] = (k + 1 < W) ? raw[k + 1] : 0.0;
            L.pb[j] = (k + 1 < W) ? plist[k + 1] : 0.0;
        }
    }
    L.i = st.n_evals[m];  // readings taken before this one == index of this evaluation
    L.counter = st.counter[m];
    L.freeze_eval = st.freeze_eval[m];
    L.slope = st.last_slope[m];
    L.T = (double)st.T[m];
    return L;
}

__device__ __forceinline__ void plasticity_step_apply(const SlopeState &st, StepLoaded &L, int m, int W,
                                                      int signed_test, float reading, double *out_slopes,
                                                      uint8_t *out_mask, int lane) {
    double *raw = st.raw + (int64_t)m * st.W_cap, *plist = st.plist + (int64_t)m * st.W_cap;
    const bool fast = (W <= 32 * kStepRegs);
    double(&ra)[kStepRegs] = L.ra, (&rb)[kStepRegs] = L.rb, (&pa)[kStepRegs] = L.pa, (&pb)[kStepRegs] = L.pb;
    const int i = L.i;
    int counter = L.counter, freeze_eval = L.freeze_eval;
    double slope = L.slope;
    const double T = L.T;
    __syncwarp();
    if (counter < W) {
        const int len = (i < W) ? i : W;       // entries in the windows now
        const bool drop = (len == W);          // the oldest entry leaves
        const int n = drop ? W : len + 1;      // entries after this reading: min(i + 1, W)
        const double P = (double)reading;
        if (fast) {
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
            if (drop) {  // shift both windows left by one, 32 entries at a time
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
            const double pbar = warp_sum_f64(s) / (double)n;
            if (lane == 0) plist[n - 1] = pbar;
            __syncwarp();
            slope = window_slope(n, lane, [&](int k) { return plist[k]; });
        }
        const bool stale = signed_test ? (slope < T) : (fabs(slope) < T);  // NaN compares false
        counter = stale ? counter + 1 : 0;
        if (counter >= W && freeze_eval < 0) freeze_eval = i;
        if (lane == 0) {
            st.n_evals[m] = i + 1;
            st.counter[m] = counter;
            st.freeze_eval[m] = freeze_eval;
            st.last_slope[m] = slope;
        }
    }
    if (lane == 0) {
        if (out_slopes) out_slopes[m] = slope;
        if (out_mask) out_mask[m] = (counter >= W) ? 1 : 0;
    }
}

__device__ __forceinline__ void plasticity_step_module(const SlopeState &st, int m, int W, int signed_test,
                                                       float reading, double *out_slopes, uint8_t *out_mask,
                                                       int lane) {
    StepLoaded L = plasticity_step_load(st, m, W, lane);
    plasticity_step_apply(st, L, m, W, signed_test, reading, out_slopes, out_mask, lane);
}

// One new reading per module.  grid = M warps (one 32-thread block each).
__global__ void __launch_bounds__(32) plasticity_step_kernel(SlopeState st, int M, int W, int signed_test,
                                                             const float *losses, double *out_slopes,
                                                             uint8_t *out_mask) {
    const int m = blockIdx.x, lane = threadIdx.x;
    if (m >= M) return;
    plasticity_step_module(st, m, W, signed_test, losses[m], out_slopes, out_mask, lane);
}

// Whole histories from a cleared private state (rings in shared memory: 2 * W doubles).
__global__ void __launch_bounds__(32) plasticity_replay_kernel(const float *T, int M, int W, int signed_test,
                                                               const float *hist, int H, double *out_slopes,
                                                               uint8_t *out_mask, int32_t *out_freeze_eval) {
    extern __shared__ double rings[];
    double *raw = rings, *plist = rings + W;
    const int m = blockIdx.x, lane = threadIdx.x;
    if (m >= M) return;
    int n_evals = 0, counter = 0, freeze_eval = -1;
    const double Tm = (double)T[m];
    for (int i = 0; i < H; ++i) {
        double slope = NAN;
        if (counter < W)
            slope = plasticity_advance(raw, plist, n_evals, counter, freeze_eval, (double)hist[(int64_t)m * H + i],
                                       W, Tm, signed_test != 0, lane);
        if (out_slopes && lane == 0) out_slopes[(int64_t)m * H + i] = slope;
    }
    if (lane == 0) {
        if (out_mask) out_mask[m] = (counter >= W) ? 1 : 0;
        if (out_freeze_eval) out_freeze_eval[m] = freeze_eval;
    }
}

__global__ void plasticity_clear_kernel(SlopeState st, int M) {
    const int m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m >= M) return;
    st.n_evals[m] = 0;
    st.counter[m] = 0;
    st.freeze_eval[m] = -1;
    st.last_slope[m] = INFINITY;
}

}  // namespace egeria
