// Second half of the SP loss (Eq. 1): sum the partial Grams of every (module, side) in a
// fixed order, scale every row of G to unit L2 norm, and reduce the squared difference
// of the two normalised matrices to one number per module, divided by b^2.
// One warp per row of G; the last CTA of a module (ticket) adds the row terms in
// ascending order, so the result does not depend on scheduling.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "plan.h"

namespace egeria {

constexpr int kFinThreads = 256;
constexpr int kFinRowsPerCta = kFinThreads / 32;
constexpr int kMaxB = 256;
constexpr double kNormEps = 1e-12;

struct FinParams {
    const float *slots;
    int64_t slot_floats;
    const SideInfo *sides;  // [2 * M]
    int32_t b;
    float *out_losses;      // [M]
    double *rowloss;        // [M][kMaxB] scratch
    int32_t *tickets;       // [M], zero between calls
    float *keep;            // [M][2][b*b] normalised matrices, or nullptr
};

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__global__ void __launch_bounds__(kFinThreads) finalize_kernel(const FinParams p) {
    const int m = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = p.b;
    const int i = blockIdx.y * kFinRowsPerCta + warp;
    __shared__ int is_last;

    if (i < b) {
        double g[2][kMaxB / 32];
#pragma unroll
        for (int side = 0; side < 2; ++side) {
            const SideInfo si = p.sides[2 * m + side];
#pragma unroll
            for (int c = 0; c < kMaxB / 32; ++c) g[side][c] = 0.0;
            for (int u = 0; u < si.n_slots; ++u) {
                const float *row = p.slots + (int64_t)(si.first_slot + u) * p.slot_floats + si.side_off +
                                   (int64_t)i * si.pitch;
#pragma unroll
                for (int c = 0; c < kMaxB / 32; ++c) {
                    const int j = lane + 32 * c;
                    if (j < b) g[side][c] += (double)__ldcg(row + j);
                }
            }
            double ss = 0.0;
#pragma unroll
            for (int c = 0; c < kMaxB / 32; ++c) ss += g[side][c] * g[side][c];
            ss = warp_sum(ss);
            double n = sqrt(ss);
            if (n < kNormEps) n = kNormEps;
#pragma unroll
            for (int c = 0; c < kMaxB / 32; ++c) g[side][c] = g[side][c] / n;
            if (p.keep) {
                float *dst = p.keep + ((int64_t)(2 * m + side) * b + i) * b;
#pragma unroll
                for (int c = 0; c < kMaxB / 32; ++c) {
                    const int j = lane + 32 * c;
                    if (j < b) dst[j] = (float)g[side][c];
                }
            }
        }
        double s = 0.0;
#pragma unroll
        for (int c = 0; c < kMaxB / 32; ++c) {
            const double diff = g[0][c] - g[1][c];
            s += diff * diff;
        }
        s = warp_sum(s);
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
        s = warp_sum(s);
        if (lane == 0) {
            p.out_losses[m] = (float)(s / ((double)b * (double)b));
            p.tickets[m] = 0;
        }
    }
}

}  // namespace egeria
