// Second half of the SP loss (Eq. 1): sum the partial Grams of every (module, side) in a
// fixed order, scale every row of G to unit L2 norm, and reduce the squared difference
// of the two normalised matrices to one number per module, divided by b^2.
// One warp per row of G; the last CTA of a module (ticket) adds the row terms in
// ascending order, so the result does not depend on scheduling.  Optionally the same
// warp then advances the module's freezing rule with the new reading (fused step).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "plan.h"
#include "slope.cuh"

namespace egeria {

constexpr int kFinThreads = 256;
constexpr int kFinRowsPerCta = kFinThreads / 32;
constexpr int kMaxB = 256;
constexpr double kNormEps = 1e-12;
constexpr int kFinBatch = 8;  // partial slots whose loads are issued together

struct FinParams {
    const float *slots;
    int64_t slot_floats;
    const SideInfo *sides;  // [2 * M]
    int32_t b;
    float *out_losses;      // [M]
    double *rowloss;        // [M][kMaxB] scratch
    int32_t *tickets;       // [M], zero between calls
    float *keep;            // [M][2][b*b] normalised matrices, or nullptr
    // fused freezing-rule step (fuse_step != 0): Algorithm 1 on the loss just computed
    int32_t fuse_step;
    int32_t W;
    int32_t signed_test;
    SlopeState st;
    double *out_slopes;     // [M] or nullptr
    uint8_t *out_mask;      // [M] or nullptr
};

// Row i of G for one side: NC columns per lane (column j = lane + 32 c), partial slots added
// in ascending slot order in float64.  Loads of kFinBatch slots are in flight together.
template <int NC>
__device__ __forceinline__ void sum_row_partials(const float *slots, int64_t slot_floats, const SideInfo si, int i,
                                                 int b, int lane, double (&g)[NC]) {
#pragma unroll
    for (int c = 0; c < NC; ++c) g[c] = 0.0;
    const float *row0 = slots + (int64_t)si.first_slot * slot_floats + si.side_off + (int64_t)i * si.pitch;
    for (int u0 = 0; u0 < si.n_slots; u0 += kFinBatch) {
        float v[kFinBatch][NC];
#pragma unroll
        for (int k = 0; k < kFinBatch; ++k) {
            const bool live = (u0 + k < si.n_slots);
            const float *row = row0 + (int64_t)(u0 + k) * slot_floats;
#pragma unroll
            for (int c = 0; c < NC; ++c) {
                const int j = lane + 32 * c;
                v[k][c] = (live && j < b) ? __ldcg(row + j) : 0.f;
            }
        }
#pragma unroll
        for (int k = 0; k < kFinBatch; ++k)
#pragma unroll
            for (int c = 0; c < NC; ++c) g[c] += (double)v[k][c];
    }
}

template <int NC>
__global__ void __launch_bounds__(kFinThreads) finalize_kernel(const FinParams p) {
    const int m = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = p.b;
    const int i = blockIdx.y * kFinRowsPerCta + warp;
    __shared__ int is_last;

    if (i < b) {
        double g[2][NC];
        sum_row_partials<NC>(p.slots, p.slot_floats, p.sides[2 * m], i, b, lane, g[0]);
        sum_row_partials<NC>(p.slots, p.slot_floats, p.sides[2 * m + 1], i, b, lane, g[1]);
#pragma unroll
        for (int side = 0; side < 2; ++side) {
            double ss = 0.0;
#pragma unroll
            for (int c = 0; c < NC; ++c) ss += g[side][c] * g[side][c];
            ss = warp_sum_f64(ss);
            double n = sqrt(ss);
            if (n < kNormEps) n = kNormEps;
#pragma unroll
            for (int c = 0; c < NC; ++c) g[side][c] = g[side][c] / n;
            if (p.keep) {
                float *dst = p.keep + ((int64_t)(2 * m + side) * b + i) * b;
#pragma unroll
                for (int c = 0; c < NC; ++c) {
                    const int j = lane + 32 * c;
                    if (j < b) dst[j] = (float)g[side][c];
                }
            }
        }
        double s = 0.0;
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            const double diff = g[0][c] - g[1][c];
            s += diff * diff;
        }
        s = warp_sum_f64(s);
        if (lane == 0) p.rowloss[(int64_t)m * kMaxB + i] = s;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const int t = atomicAdd(&p.tickets[m], 1);
        is_last = (t == (int)gridDim.y - 1);
    }
    __syncthreads();
    if (is_last && warp == 0) {
        __threadfence();
        double s = 0.0;
        for (int r = lane; r < b; r += 32) s += __ldcg(&p.rowloss[(int64_t)m * kMaxB + r]);
        s = warp_sum_f64(s);
        const float loss = (float)(s / ((double)b * (double)b));
        if (lane == 0) {
            p.out_losses[m] = loss;
            p.tickets[m] = 0;
        }
        if (p.fuse_step) plasticity_step_module(p.st, m, p.W, p.signed_test, loss, p.out_slopes, p.out_mask, lane);
    }
}

}  // namespace egeria
