// Partial Gram matrices G = A A^T on the 5th-generation tensor cores (sm_100a).
//
// One persistent CTA per SM walks its static list of work units (a K-range of one
// (module, side) tile).  Per 64-element block of the feature axis, one TMA box load
// brings all b rows into a 128-byte-swizzled shared-memory slab; the same slab is
// both the A and the B operand of tcgen05.mma (row block i against row block j,
// i <= j), accumulating in fp32 in tensor memory.  At the end of a unit the
// accumulator is drained to the unit's partial slot in the workspace.
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = MMA issuer and TMEM
// owner, warps 2..5 = epilogue (TMEM -> registers -> global).
// Every mbarrier wait is bounded; on expiry the CTA raises its abort flag, records
// EGERIA_ERR_TIMEOUT in the status word, drains what is in flight and returns.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "plan.h"
#include "ptx_sm100.cuh"

namespace egeria {

constexpr int kTcThreads = 192;
constexpr uint64_t kWaitLimitNs = 2000000000ull;  // 2 s per wait
constexpr int kStatusTimeout = 6;                 // == EGERIA_ERR_TIMEOUT

template <int MODE>
struct TcCfg {
    static constexpr int kSlabRows = (MODE == kSingle2) ? 256 : 128;
    static constexpr int kStageBytes = kSlabRows * 128;          // one 64-element block of all rows
    static constexpr int kStages = (MODE == kSingle2) ? 6 : 12;  // 192 KB of loads in flight
    static constexpr int kAccCols = (MODE == kSingle2) ? 384 : 128;
    static constexpr int kAccStages = (MODE == kSingle2) ? 1 : 2;
    static constexpr int kTmemCols = (MODE == kSingle2) ? 512 : 256;
    static constexpr int kBoxRows = (MODE == kStacked) ? 64 : kSlabRows;  // rows of one TMA box
    static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 512 /*barriers*/;
};

struct TcParams {
    const CUtensorMap *tmaps;  // [2 * M]: A_T and A_R of every module (device memory)
    const Unit *units;         // tensor-core units
    const int32_t *cta_begin;  // [gridDim.x + 1]
    float *slots;              // partial Gram slots
    int64_t slot_floats;
    int32_t b;
    int32_t *status;           // device status word
};

template <int MODE>
__global__ void __launch_bounds__(kTcThreads, 1) gram_tc_kernel(const TcParams p) {
    using Cfg = TcCfg<MODE>;
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte alignment: the 128-byte swizzle pattern is a function of address bits 4..9.
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_aligned = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_aligned + Cfg::kStages * Cfg::kStageBytes);
    // bars: full[kStages], empty[kStages], acc_full[kAccStages], acc_empty[kAccStages]
    const uint32_t full0 = ptx::smem_u32(bars);
    const uint32_t empty0 = full0 + 8 * Cfg::kStages;
    const uint32_t accfull0 = empty0 + 8 * Cfg::kStages;
    const uint32_t accempty0 = accfull0 + 8 * Cfg::kAccStages;
    volatile uint32_t *tmem_holder =
        reinterpret_cast<volatile uint32_t *>(bars + 2 * Cfg::kStages + 2 * Cfg::kAccStages);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_holder + 1);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int u_begin = p.cta_begin[blockIdx.x];
    const int u_end = p.cta_begin[blockIdx.x + 1];

    if (threadIdx.x == 0) {
        for (int s = 0; s < Cfg::kStages; ++s) {
            ptx::mbar_init(full0 + 8 * s, 1);
            ptx::mbar_init(empty0 + 8 * s, 1);
        }
        for (int s = 0; s < Cfg::kAccStages; ++s) {
            ptx::mbar_init(accfull0 + 8 * s, 1);
            ptx::mbar_init(accempty0 + 8 * s, 4);  // one arrival per epilogue warp
        }
        *abort_flag = 0;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async();
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(const_cast<uint32_t *>(tmem_holder)), Cfg::kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_holder;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const uint64_t policy = ptx::l2_policy_evict_first();
            uint32_t stage = 0, phase = 0;
            uint32_t issued = 0;
            bool ok = true;
            int last_module = -1;
            for (int ui = u_begin; ui < u_end && ok; ++ui) {
                const Unit u = p.units[ui];
                const CUtensorMap *tm_t = p.tmaps + 2 * u.module;
                const CUtensorMap *tm_r = tm_t + 1;
                if (u.module != last_module) {
                    ptx::tensormap_acquire(tm_t);
                    ptx::tensormap_acquire(tm_r);
                    last_module = u.module;
                }
                const CUtensorMap *tm_side = (u.side == 1) ? tm_r : tm_t;
                for (int kb = u.kb0; kb < u.kb0 + u.nkb; ++kb) {
                    if (!ptx::mbar_wait_bounded(empty0 + 8 * stage, phase ^ 1u, abort_flag, kWaitLimitNs)) {
                        ok = false;
                        break;
                    }
                    const uint32_t dst = smem_base + stage * Cfg::kStageBytes;
                    const uint32_t bar = full0 + 8 * stage;
                    ptx::mbar_arrive_expect_tx(bar, Cfg::kStageBytes);
                    if (MODE == kStacked) {
                        ptx::tma_load_2d(dst, tm_t, kb * kKBlock, 0, bar, policy);
                        ptx::tma_load_2d(dst + 64 * 128, tm_r, kb * kKBlock, 0, bar, policy);
                    } else {
                        ptx::tma_load_2d(dst, tm_side, kb * kKBlock, 0, bar, policy);
                    }
                    ++issued;
                    if (++stage == Cfg::kStages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
            if (!ok) {
                // Gave up: still wait (bounded) for every load already issued, so that no
                // copy is in flight into this CTA's shared memory when it exits.
                const uint32_t n = issued < (uint32_t)Cfg::kStages ? issued : (uint32_t)Cfg::kStages;
                for (uint32_t k = 1; k <= n; ++k) {
                    const uint32_t idx = issued - k;  // k-th most recent load
                    const uint32_t s = idx % Cfg::kStages, ph = (idx / Cfg::kStages) & 1u;
                    const uint64_t t0 = ptx::globaltimer_ns();
                    while (!ptx::mbar_try_wait(full0 + 8 * s, ph))
                        if (ptx::globaltimer_ns() - t0 > kWaitLimitNs) break;
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc128 = ptx::make_idesc_bf16_f32(128, 128);
            constexpr uint32_t idesc256 = ptx::make_idesc_bf16_f32(128, 256);
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            bool any_mma = false;
            for (int ui = u_begin; ui < u_end && ok; ++ui) {
                const Unit u = p.units[ui];
                if (!ptx::mbar_wait_bounded(accempty0 + 8 * acc, acc_phase ^ 1u, abort_flag, kWaitLimitNs)) {
                    ok = false;
                    break;
                }
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + acc * Cfg::kAccCols;
                for (int kb = 0; kb < u.nkb; ++kb) {
                    if (!ptx::mbar_wait_bounded(full0 + 8 * stage, phase, abort_flag, kWaitLimitNs)) {
                        ok = false;
                        break;
                    }
                    ptx::tc_fence_after_sync();
                    const uint32_t slab = smem_base + stage * Cfg::kStageBytes;
#pragma unroll
                    for (int k = 0; k < kKBlock / 16; ++k) {
                        const uint32_t accum = (kb > 0 || k > 0) ? 1u : 0u;
                        const uint64_t lo = ptx::make_desc_k_sw128(slab + k * 32);
                        if (MODE == kSingle2) {
                            const uint64_t hi = ptx::make_desc_k_sw128(slab + 128 * 128 + k * 32);
                            // [G00 | G01] = rows 0..127 against rows 0..255
                            ptx::mma_bf16_ss(d_tmem, lo, lo, idesc256, accum);
                            // G11 = rows 128..255 against themselves
                            ptx::mma_bf16_ss(d_tmem + 256, hi, hi, idesc128, accum);
                        } else {
                            ptx::mma_bf16_ss(d_tmem, lo, lo, idesc128, accum);
                        }
                    }
                    any_mma = true;
                    ptx::mma_commit(empty0 + 8 * stage);  // slab free once these MMAs have read it
                    if (++stage == Cfg::kStages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                if (!ok) break;
                ptx::mma_commit(accfull0 + 8 * acc);  // accumulator complete
                if (++acc == Cfg::kAccStages) {
                    acc = 0;
                    acc_phase ^= 1u;
                }
            }
            if (!ok && any_mma) {
                // Gave up: give the MMAs already issued time to finish before TMEM is freed
                // (2 ms is far longer than any queue of MMAs).
                const uint64_t t0 = ptx::globaltimer_ns();
                while (ptx::globaltimer_ns() - t0 < 2000000ull) {
                }
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ epilogue warps
        const int q = warp & 3;  // TMEM lane quarter this warp may read
        const int b = p.b;
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        for (int ui = u_begin; ui < u_end && ok; ++ui) {
            const Unit u = p.units[ui];
            if (!ptx::mbar_wait_bounded(accfull0 + 8 * acc, acc_phase, abort_flag, kWaitLimitNs)) {
                ok = false;
                break;
            }
            ptx::tc_fence_after_sync();
            float *slot = p.slots + (int64_t)u.slot * p.slot_floats;
            const uint32_t t_row = tmem_base + acc * Cfg::kAccCols + ((uint32_t)(q * 32) << 16);
            uint32_t v[32];
            if (MODE == kStacked) {
                // rows 0..63 x cols 0..63 = G_T, rows 64..127 x cols 64..127 = G_R
                const int side = q >> 1;
                const int r = (q & 1) * 32 + lane;
                if ((q & 1) * 32 < b) {
                    float *dst = slot + side * 64 * 64 + r * 64;
                    for (int c0 = 0; c0 < 64 && c0 < b; c0 += 32) {
                        ptx::tmem_ld_32x32(t_row + side * 64 + c0, v);
                        ptx::tmem_ld_wait();
                        if (r < b) {
#pragma unroll
                            for (int c = 0; c < 32; c += 4)
                                *reinterpret_cast<uint4 *>(dst + c0 + c) = make_uint4(v[c], v[c + 1], v[c + 2], v[c + 3]);
                        }
                    }
                }
            } else if (MODE == kSingle1) {
                const int r = q * 32 + lane;
                if (q * 32 < b) {
                    float *dst = slot + r * 128;
                    for (int c0 = 0; c0 < 128 && c0 < b; c0 += 32) {
                        ptx::tmem_ld_32x32(t_row + c0, v);
                        ptx::tmem_ld_wait();
                        if (r < b) {
#pragma unroll
                            for (int c = 0; c < 32; c += 4)
                                *reinterpret_cast<uint4 *>(dst + c0 + c) = make_uint4(v[c], v[c + 1], v[c + 2], v[c + 3]);
                        }
                    }
                }
            } else {
                // TMEM cols 0..255: rows 0..127 of G (all 256 columns); cols 256..383: G11.
                const int r = q * 32 + lane;  // 0..127, always < b in this mode
                float *dst = slot + r * 256;
                for (int c0 = 0; c0 < 256 && c0 < b; c0 += 32) {
                    ptx::tmem_ld_32x32(t_row + c0, v);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int c = 0; c < 32; c += 4)
                        *reinterpret_cast<uint4 *>(dst + c0 + c) = make_uint4(v[c], v[c + 1], v[c + 2], v[c + 3]);
                    if (c0 >= 128) {
                        // mirror G01 into the lower-left block: lanes write consecutive floats
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (c0 + c < b) slot[(c0 + c) * 256 + r] = __uint_as_float(v[c]);
                    }
                }
                if (128 + q * 32 < b) {
                    float *dst2 = slot + (128 + r) * 256 + 128;
                    for (int c0 = 0; c0 < 128 && 128 + c0 < b; c0 += 32) {
                        ptx::tmem_ld_32x32(t_row + 256 + c0, v);
                        ptx::tmem_ld_wait();
                        if (128 + r < b) {
#pragma unroll
                            for (int c = 0; c < 32; c += 4)
                                *reinterpret_cast<uint4 *>(dst2 + c0 + c) = make_uint4(v[c], v[c + 1], v[c + 2], v[c + 3]);
                        }
                    }
                }
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(accempty0 + 8 * acc);
            if (++acc == Cfg::kAccStages) {
                acc = 0;
                acc_phase ^= 1u;
            }
        }
    }

    // ---------------------------------------------------------------- teardown
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    if (warp == 1) ptx::tmem_dealloc(tmem_base, Cfg::kTmemCols);
    if (threadIdx.x == 0 && *abort_flag) atomicMax(p.status, kStatusTimeout);
}

}  // namespace egeria
