// The freezing rule (Sec. 4.2.2, Eq. 2, Algorithm 1) for all modules: moving average
// of the raw plasticity readings, least-squares slope of the last W smoothed values,
// tolerance test, consecutive-stale counter.  One warp per module, float64 throughout.
#pragma once
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

namespace egeria {

struct SlopeState {     // per-module arrays (device)
    double *raw;        // [M][W_cap] ring of raw readings P_i
    double *plist;      // [M][W_cap] ring of smoothed readings (the last W of pList)
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

// One new reading for module m, by one warp: Algorithm 1 on the context's state.
__device__ __forceinline__ void plasticity_step_module(const SlopeState &st, int m, int W, int signed_test,
                                                       float reading, double *out_slopes, uint8_t *out_mask,
                                                       int lane) {
    int n_evals = st.n_evals[m], counter = st.counter[m], freeze_eval = st.freeze_eval[m];
    double slope = st.last_slope[m];
    __syncwarp();
    if (counter < W) {
        slope = plasticity_advance(st.raw + (int64_t)m * st.W_cap, st.plist + (int64_t)m * st.W_cap, n_evals,
                                   counter, freeze_eval, (double)reading, W, (double)st.T[m], signed_test != 0,
                                   lane);
        if (lane == 0) {
            st.n_evals[m] = n_evals;
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
