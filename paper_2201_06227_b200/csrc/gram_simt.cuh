// Partial Gram matrices on the CUDA cores: plain 2-byte loads, fp32 FMA.
// Takes the modules the tensor-core kernel cannot (d not a multiple of 8, or a base
// pointer that is not 16-byte aligned), or all of them when the context asks for it.
// Same work units and the same partial-slot layout as the tensor-core kernel.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "plan.h"

namespace egeria {

constexpr int kSimtThreads = 256;
constexpr int kSimtTile = 64;   // output tile is 64 x 64, 4 x 4 per thread
constexpr int kSimtKChunk = 32;

struct SimtParams {
    const ModulePtrs *modules;
    const Unit *units;         // CUDA-core units
    const int32_t *cta_begin;  // [gridDim.x + 1]
    float *slots;
    int64_t slot_floats;
    int32_t b;
    int32_t mode;
};

__global__ void __launch_bounds__(kSimtThreads) gram_simt_kernel(const SimtParams p) {
    __shared__ float As[kSimtKChunk][kSimtTile + 1];
    __shared__ float Bs[kSimtKChunk][kSimtTile + 1];
    const int tid = threadIdx.x;
    const int ty = tid >> 4, tx = tid & 15;
    const int b = p.b;
    const int pitch = pitch_of_mode(p.mode);
    const int nblk = (b + kSimtTile - 1) / kSimtTile;

    for (int ui = p.cta_begin[blockIdx.x]; ui < p.cta_begin[blockIdx.x + 1]; ++ui) {
        const Unit u = p.units[ui];
        const ModulePtrs mp = p.modules[u.module];
        const int64_t d = mp.d;
        const int64_t k_lo = (int64_t)u.kb0 * kKBlock;
        int64_t k_hi = k_lo + (int64_t)u.nkb * kKBlock;
        if (k_hi > d) k_hi = d;
        float *slot = p.slots + (int64_t)u.slot * p.slot_floats;
        for (int side = 0; side < 2; ++side) {
            if (u.side != 2 && u.side != side) continue;
            const __nv_bfloat16 *A = static_cast<const __nv_bfloat16 *>(side == 0 ? mp.At : mp.Ar);
            float *out = slot + (mode_is_stacked(p.mode) ? side * pitch * pitch : 0);
            for (int bi = 0; bi < nblk; ++bi) {
                for (int bj = bi; bj < nblk; ++bj) {
                    float acc[4][4];
#pragma unroll
                    for (int i = 0; i < 4; ++i)
#pragma unroll
                        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
                    for (int64_t k0 = k_lo; k0 < k_hi; k0 += kSimtKChunk) {
                        for (int idx = tid; idx < kSimtTile * kSimtKChunk; idx += kSimtThreads) {
                            const int row = idx / kSimtKChunk, kk = idx % kSimtKChunk;
                            const int64_t k = k0 + kk;
                            const int ri = bi * kSimtTile + row, rj = bj * kSimtTile + row;
                            As[kk][row] = (ri < b && k < k_hi) ? __bfloat162float(A[(int64_t)ri * d + k]) : 0.f;
                            Bs[kk][row] = (rj < b && k < k_hi) ? __bfloat162float(A[(int64_t)rj * d + k]) : 0.f;
                        }
                        __syncthreads();
#pragma unroll 8
                        for (int kk = 0; kk < kSimtKChunk; ++kk) {
                            float a[4], c[4];
#pragma unroll
                            for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
                            for (int j = 0; j < 4; ++j) c[j] = Bs[kk][tx * 4 + j];
#pragma unroll
                            for (int i = 0; i < 4; ++i)
#pragma unroll
                                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], c[j], acc[i][j]);
                        }
                        __syncthreads();
                    }
#pragma unroll
                    for (int i = 0; i < 4; ++i)
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const int r = bi * kSimtTile + ty * 4 + i, c = bj * kSimtTile + tx * 4 + j;
                            if (r < b && c < b) {
                                out[r * pitch + c] = acc[i][j];
                                if (bi != bj) out[c * pitch + r] = acc[i][j];
                            }
                        }
                }
            }
        }
    }
}

}  // namespace egeria
