// Second half of the SP loss (Eq. 1): sum the partial Grams of every (module, side) in a
// fixed order, scale every row of G to unit L2 norm, and reduce the squared difference
// of the two normalised matrices to one number per module, divided by b^2.
//
// The work is cut into rows of G, one warp per row (finalize_row, finalize_row_staged), and one last step per
// module that adds the row terms in a fixed order (finalize_module_total), so the result
// does not depend on who did which row or when.  The tensor-core Gram kernel calls both
// from its own epilogue warps; finalize_kernel wraps them for the modules whose partial
// Grams came from the CUDA-core kernel.  Optionally the warp that finishes a module also
// advances the module's freezing rule with the new reading (fused step).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "check.cuh"
#include "plan.h"
#include "slope.cuh"

namespace egeria {

constexpr int kFinThreads = 256;
constexpr int kFinRowsPerCta = kFinThreads / 32;
constexpr int kMaxB = 256;
constexpr double kNormEps = 1e-12;

// What a partial slot holds where nothing has been written since it was last emptied: the
// tensor-core kernel's finish can tell a partial row that has arrived from one that has not by its
// values alone (no flag, no fence: every 4-byte element is its own flag).  The epilogue never
// stores this pattern as a value (a NaN with these bits becomes the canonical one); launches that
// work this way alternate between two sets of slots, and each empties, at its start, what the
// launch before wrote into the other set.
constexpr uint32_t kSlotEmpty = 0xffffffffu;
constexpr uint32_t kCanonicalNan = 0x7fc00000u;

struct FinCommon {
    float *slots;
    int64_t slot_floats;
    uint32_t sentinel;      // 1: a partial row has arrived when none of its elements is kSlotEmpty (no counters)
    uint64_t wait_limit_ns; // limit of the wait for partial rows that have not arrived
    int32_t *status;        // device status word (and the checked build's record after it)
    int64_t slots_floats;   // floats from `slots` to the end of the slots this launch may use
    int64_t chunk_doubles;  // doubles in chunk_sums
    const SideInfo *sides;  // [2 * M]
    int32_t b;
    float *out_losses;      // [M]
    double *rowloss;        // [M][kMaxB] scratch
    float *keep;            // [M][2][b*b] normalised matrices, or nullptr
    double *chunk_sums;     // scratch of the two-level finalisation (one module evaluated alone), or nullptr
    // fused freezing-rule step (fuse_step != 0): Algorithm 1 on the loss just computed
    int32_t fuse_step;
    int32_t rule_flags;     // RuleFlags
    uint32_t rule_serial;   // number of this evaluation of the rule, from 1 (frontmost policy)
    int32_t M;
    double lr;              // learning rate in force (not positive or NaN: unknown), for the unfreezing rule
    SlopeState st;
    double *out_slopes;     // [M] or nullptr
    uint8_t *out_mask;      // [M] or nullptr
};

// Columns per lane for a given b (column j = lane + 32 c, c < NC).
__host__ __device__ inline int fin_nc_of_b(int b) { return b <= 32 ? 1 : (b <= 64 ? 2 : (b <= 128 ? 4 : 8)); }

// Column of G that a lane's c-th value belongs to when a lane owns runs of consecutive columns
// (so that it can fetch them from shared memory with one vector load): 4-column runs, 128
// columns apart, for NC >= 4; a 2-column run for NC == 2; one column for NC == 1.
template <int NC>
__device__ __forceinline__ int fin_col(int lane, int c) {
    return NC >= 4 ? 4 * lane + (c & 3) + 128 * (c >> 2) : NC * lane + c;
}

// Second half of a row, given its two sums gT, gR (this lane's columns: lane + 32 c, or
// fin_col(lane, c) if kVec): scale each
// side to unit L2 norm (norm clamped at kNormEps), leave the normalised rows in `keep` if
// asked, and return sum_j (G~_T[i][j] - G~_R[i][j])^2 (all lanes).  Float64 throughout; one
// reciprocal per side instead of a division per entry, and the two sides' reductions are
// interleaved, because this runs at the very end of the kernel with nothing to overlap it.
template <int NC, bool kVec>
__device__ __forceinline__ double row_term(const FinCommon &p, int m, int i, int lane, double (&gT)[NC],
                                           double (&gR)[NC]) {
    const int b = p.b;
    double ssT = 0.0, ssR = 0.0;
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        ssT = fma(gT[c], gT[c], ssT);
        ssR = fma(gR[c], gR[c], ssR);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        ssT += __shfl_xor_sync(0xffffffffu, ssT, o);
        ssR += __shfl_xor_sync(0xffffffffu, ssR, o);
    }
    double nT = sqrt(ssT), nR = sqrt(ssR);
    if (nT < kNormEps) nT = kNormEps;
    if (nR < kNormEps) nR = kNormEps;
    const double invT = 1.0 / nT, invR = 1.0 / nR;
    double s = 0.0;
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        gT[c] *= invT;
        gR[c] *= invR;
        const double diff = gT[c] - gR[c];
        s = fma(diff, diff, s);
    }
    if (p.keep) {
        float *dT = p.keep + ((int64_t)(2 * m) * b + i) * b, *dR = dT + (int64_t)b * b;
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            const int j = kVec ? fin_col<NC>(lane, c) : lane + 32 * c;
            if (j < b) {
                dT[j] = (float)gT[c];
                dR[j] = (float)gR[c];
            }
        }
    }
    return warp_sum_f64(s);
}

// One warp: row i of module m with the partials read straight into registers.  Partial slots
// are added in ascending slot order in float64; the loads of KB slots per side go together.
template <int NC>
__device__ __forceinline__ double finalize_row(const FinCommon &p, const SideInfo sT, const SideInfo sR, int m, int i,
                                               int lane) {
    constexpr int KB = (32 / (2 * NC)) > 0 ? (32 / (2 * NC)) : 1;
    const int b = p.b;
    double gT[NC], gR[NC];
#pragma unroll
    for (int c = 0; c < NC; ++c) gT[c] = gR[c] = 0.0;
    const float *rowT = p.slots + (int64_t)sT.first_slot * p.slot_floats + sT.side_off + (int64_t)i * sT.pitch;
    const float *rowR = p.slots + (int64_t)sR.first_slot * p.slot_floats + sR.side_off + (int64_t)i * sR.pitch;
    const int n_max = sT.n_slots > sR.n_slots ? sT.n_slots : sR.n_slots;
    for (int u0 = 0; u0 < n_max; u0 += KB) {
        float vT[KB][NC], vR[KB][NC];
#pragma unroll
        for (int k = 0; k < KB; ++k) {
            const bool liveT = (u0 + k < sT.n_slots), liveR = (u0 + k < sR.n_slots);
            const float *pT = rowT + (int64_t)(u0 + k) * p.slot_floats;
            const float *pR = rowR + (int64_t)(u0 + k) * p.slot_floats;
#pragma unroll
            for (int c = 0; c < NC; ++c) {
                const int j = lane + 32 * c;
                vT[k][c] = (liveT && j < b) ? __ldcg(pT + j) : 0.f;
                vR[k][c] = (liveR && j < b) ? __ldcg(pR + j) : 0.f;
            }
        }
#pragma unroll
        for (int k = 0; k < KB; ++k)
#pragma unroll
            for (int c = 0; c < NC; ++c) {
                gT[c] += (double)vT[k][c];
                gR[c] += (double)vR[k][c];
            }
    }
    return row_term<NC, false>(p, m, i, lane, gT, gR);
}


// One warp: rows 0 .. G - 1 of the stage <- the partial rows src_of(0 .. G - 1) (32 * NC floats
// each), every 16-byte piece fetched with cp.async, all in flight together whatever the register
// budget.  With p.sentinel the rows need not have arrived yet: pieces that still hold kSlotEmpty
// in the columns the epilogue writes (the first b, rounded up to 32) are fetched again until they
// do not -- at most p.wait_limit_ns, then the CTA's abort flag is set and false returned.  (The
// slots are put back to kSlotEmpty by the launch after this one, which uses another set of them.)
template <int NC, class SrcOf>
__device__ __forceinline__ bool fetch_partial_rows(const FinCommon &p, int G, SrcOf src_of, int lane, float *stage,
                                                   volatile int *abort_flag) {
    constexpr int kPitch = 32 * NC;                          // floats per row of a partial
    constexpr int kPieces = kPitch / 4;                      // 16-byte pieces per row: 8, 16, 32, 64
    constexpr int kLanesPerRow = kPieces < 32 ? kPieces : 32;
    constexpr int kRowsPerIssue = 32 / kLanesPerRow;         // rows one cp.async of the warp covers
    constexpr int kIssuesPerRow = (kPieces + 31) / 32;
    const uint32_t stage_addr = static_cast<uint32_t>(__cvta_generic_to_shared(stage));
    const int sub = lane / kLanesPerRow, piece = lane % kLanesPerRow;
    if (!eg_check(G >= 0 && G * kPitch * 4 <= kFinStageBytes, p.status, kCheckFetch, G)) return false;
    if (kCheckedBuild) {
        bool inside = true;
        for (int sl = lane; sl < G; sl += 32) {
            const int64_t off = src_of(sl) - p.slots;
            inside = inside && off >= 0 && off + kPitch <= p.slots_floats;
        }
        if (!eg_check(__all_sync(0xffffffffu, inside), p.status, kCheckFetch, -1)) return false;
    }
    for (int sl0 = 0; sl0 < G; sl0 += kRowsPerIssue) {
        const int sl = sl0 + sub;
        if (sl < G) {
            const float *src = src_of(sl);
#pragma unroll
            for (int q = 0; q < kIssuesPerRow; ++q) {
                const int off = 4 * (piece + 32 * q);
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(stage_addr + (sl * kPitch + off) * 4),
                             "l"(src + off)
                             : "memory");
            }
        }
    }
    asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
    __syncwarp();
    if (!p.sentinel) return true;
    const int written = (p.b + 31) & ~31;  // columns the epilogue stores
    uint64_t t0 = 0;
    for (;;) {
        bool miss = false;
        for (int sl0 = 0; sl0 < G; sl0 += kRowsPerIssue) {
            const int sl = sl0 + sub;
            if (sl < G) {
#pragma unroll
                for (int q = 0; q < kIssuesPerRow; ++q) {
                    const int off = 4 * (piece + 32 * q);
                    if (off < written) {
                        const uint4 v = *reinterpret_cast<const uint4 *>(stage + sl * kPitch + off);
                        if (v.x == kSlotEmpty || v.y == kSlotEmpty || v.z == kSlotEmpty || v.w == kSlotEmpty) {
                            miss = true;
                            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(stage_addr +
                                                                                           (sl * kPitch + off) * 4),
                                         "l"(src_of(sl) + off)
                                         : "memory");
                        }
                    }
                }
            }
        }
        if (!__any_sync(0xffffffffu, miss)) break;
        asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
        __syncwarp();
        int stop = 0;
        if (lane == 0) {
            uint64_t now;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
            if (t0 == 0) t0 = now;
            stop = (*abort_flag != 0) || (now - t0 > p.wait_limit_ns);
            if (stop) *abort_flag = 1;
        }
        if (__shfl_sync(0xffffffffu, stop, 0)) return false;
    }
    return true;
}

// This lane's values of one staged partial row: the columns fin_col(lane, c).
template <int NC>
__device__ __forceinline__ void staged_row_values(const float *row, int lane, float (&v)[NC]) {
    if (NC >= 4) {
#pragma unroll
        for (int h = 0; h < NC / 4; ++h) {
            const float4 t = *reinterpret_cast<const float4 *>(row + 128 * h + 4 * lane);
            v[4 * h] = t.x;
            v[4 * h + 1] = t.y;
            v[4 * h + 2] = t.z;
            v[4 * h + 3] = t.w;
        }
    } else if (NC == 2) {
        const float2 t = *reinterpret_cast<const float2 *>(row + 2 * lane);
        v[0] = t.x;
        v[NC - 1] = t.y;
    } else {
        v[0] = row[lane];
    }
}

// One row with the partials staged through `stage` (kFinStageBytes of shared memory that only
// this warp touches), a stage-full at a time, added from shared memory in ascending slot order
// (A_T's partials, then A_R's).  A lane owns the columns fin_col(lane, c).  The partial slots of
// the tensor-core modes have a row pitch of exactly 32 * NC floats.  `ok` = false (and nothing
// to use) if the partial rows did not arrive in time.
template <int NC>
__device__ __forceinline__ double finalize_row_staged(const FinCommon &p, const SideInfo sT, const SideInfo sR, int m,
                                                      int i, int lane, float *stage, volatile int *abort_flag,
                                                      bool &ok) {
    constexpr int kPitch = 32 * NC;                          // floats per row of a partial
    constexpr int kCap = kFinStageBytes / (kPitch * 4);      // rows of partials the stage holds
    const int b = p.b;
    double gT[NC], gR[NC];
#pragma unroll
    for (int c = 0; c < NC; ++c) gT[c] = gR[c] = 0.0;
    const float *rowT = p.slots + (int64_t)sT.first_slot * p.slot_floats + sT.side_off + (int64_t)i * kPitch;
    const float *rowR = p.slots + (int64_t)sR.first_slot * p.slot_floats + sR.side_off + (int64_t)i * kPitch;
    const int nT = sT.n_slots, n_tot = sT.n_slots + sR.n_slots;
    ok = true;
    for (int s0 = 0; s0 < n_tot; s0 += kCap) {
        const int G = (n_tot - s0 < kCap) ? n_tot - s0 : kCap;
        const int64_t slot_floats = p.slot_floats;
        ok = fetch_partial_rows<NC>(
            p, G,
            [=](int sl) {
                const int s = s0 + sl;
                return (s < nT) ? rowT + (int64_t)s * slot_floats : rowR + (int64_t)(s - nT) * slot_floats;
            },
            lane, stage, abort_flag);
        if (!ok) return 0.0;
        for (int sl = 0; sl < G; ++sl) {
            float v[NC];
            staged_row_values<NC>(stage + sl * kPitch, lane, v);
            if (s0 + sl < nT) {  // uniform over the warp
#pragma unroll
                for (int c = 0; c < NC; ++c) gT[c] += (double)v[c];
            } else {
#pragma unroll
                for (int c = 0; c < NC; ++c) gR[c] += (double)v[c];
            }
        }
        __syncwarp();  // everyone has read the stage before the next pass overwrites it
    }
    // columns beyond b hold nothing of G: whatever was added there is dropped
#pragma unroll
    for (int c = 0; c < NC; ++c)
        if (fin_col<NC>(lane, c) >= b) gT[c] = gR[c] = 0.0;
    return row_term<NC, true>(p, m, i, lane, gT, gR);
}

// ---- Two levels, for a module evaluated alone.  Such a module is cut over all CTAs, so a row of G
// has a hundred or more partial rows per side, while there are far fewer rows than warps: one warp
// per row would add them one after the other for tens of microseconds with most warps idle.
// Instead a task is (row, chunk): a warp adds the row's partials of a few consecutive slots per
// side (one pass of its stage) and leaves the two float64 sums in scratch; the warp that delivers
// a row's last chunk adds the chunk sums in chunk order and finishes the row.  Which warp does
// what does not change any sum, so the result is as reproducible as the one-level one.

// Most slots per side in one chunk: half the stage each for T and R (chunk_slots_of_mode).
template <int NC>
__host__ __device__ constexpr int fin_chunk_slots() { return kFinStageBytes / (32 * NC * 4) / 2; }
// Doubles of scratch one (row, chunk) task leaves: both sides, this row, every column.
template <int NC>
__host__ __device__ constexpr int fin_chunk_doubles() { return 2 * 32 * NC; }

// One warp: chunk `ch` of row i: fetch, add, store to scratch[(i * n_chunks + ch)].  False if the
// partial rows did not arrive in time.
template <int NC>
__device__ __forceinline__ bool finalize_row_chunk(const FinCommon &p, const SideInfo &sT, const SideInfo &sR, int i,
                                                   int ch, int n_chunks, int lane, float *stage,
                                                   volatile int *abort_flag) {
    constexpr int kPitch = 32 * NC;
    const int chunk = chunk_slots(sT.n_slots > sR.n_slots ? sT.n_slots : sR.n_slots, n_chunks);  // <= fin_chunk_slots<NC>()
    const float *rowT = p.slots + (int64_t)sT.first_slot * p.slot_floats + sT.side_off + (int64_t)i * kPitch;
    const float *rowR = p.slots + (int64_t)sR.first_slot * p.slot_floats + sR.side_off + (int64_t)i * kPitch;
    const int t0 = ch * chunk, r0 = ch * chunk;
    const int nT = (sT.n_slots - t0 < chunk) ? (sT.n_slots - t0 > 0 ? sT.n_slots - t0 : 0) : chunk;
    const int nR = (sR.n_slots - r0 < chunk) ? (sR.n_slots - r0 > 0 ? sR.n_slots - r0 : 0) : chunk;
    const int G = nT + nR;
    const int64_t slot_floats = p.slot_floats;
    if (!fetch_partial_rows<NC>(
            p, G,
            [=](int sl) {
                return (sl < nT) ? rowT + (int64_t)(t0 + sl) * slot_floats : rowR + (int64_t)(r0 + sl - nT) * slot_floats;
            },
            lane, stage, abort_flag))
        return false;
    double gT[NC], gR[NC];
#pragma unroll
    for (int c = 0; c < NC; ++c) gT[c] = gR[c] = 0.0;
    for (int sl = 0; sl < G; ++sl) {
        float v[NC];
        staged_row_values<NC>(stage + sl * kPitch, lane, v);
        if (sl < nT) {
#pragma unroll
            for (int c = 0; c < NC; ++c) gT[c] += (double)v[c];
        } else {
#pragma unroll
            for (int c = 0; c < NC; ++c) gR[c] += (double)v[c];
        }
    }
    __syncwarp();  // the stage is free again
    if (!eg_check(((int64_t)i * n_chunks + ch + 1) * fin_chunk_doubles<NC>() <= p.chunk_doubles && chunk <= fin_chunk_slots<NC>(),
                  p.status, kCheckChunkSum, (int64_t)i * n_chunks + ch))
        return false;
    double *out = p.chunk_sums + ((int64_t)i * n_chunks + ch) * fin_chunk_doubles<NC>();
#pragma unroll
    for (int c = 0; c < NC; ++c) {  // [side][c][lane]: consecutive lanes, consecutive doubles
        out[c * 32 + lane] = gT[c];
        out[(NC + c) * 32 + lane] = gR[c];
    }
    return true;
}

// One warp, once all chunks of row i are in scratch and visible: add them in chunk order and
// finish the row.  Returns the row's term (all lanes).
template <int NC>
__device__ __forceinline__ double finalize_row_from_chunks(const FinCommon &p, int m, int i, int n_chunks, int lane) {
    double gT[NC], gR[NC];
#pragma unroll
    for (int c = 0; c < NC; ++c) gT[c] = gR[c] = 0.0;
    const double *in = p.chunk_sums + (int64_t)i * n_chunks * fin_chunk_doubles<NC>();
    for (int ch = 0; ch < n_chunks; ++ch, in += fin_chunk_doubles<NC>()) {
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            gT[c] += __ldcg(in + c * 32 + lane);
            gR[c] += __ldcg(in + (NC + c) * 32 + lane);
        }
    }
#pragma unroll
    for (int c = 0; c < NC; ++c)
        if (fin_col<NC>(lane, c) >= p.b) gT[c] = gR[c] = 0.0;
    return row_term<NC, true>(p, m, i, lane, gT, gR);
}

// The rows' terms of one module are added up in ONE 64-bit integer that also counts the rows, so
// that a single atomic add per warp both delivers its terms and tells it whether it was the last
// (the value it gets back plus its own is then the complete sum: no scratch to re-read), and so
// that the sum does not depend on the order of arrival (integer addition is associative):
//   bits  0..45  sum of the terms in units of 2^-35 (a term is at most 4: both rows have unit norm;
//                256 rows x 4 x 2^35 = 2^45)
//   bits 46..54  rows whose term was not a finite number in [0, 4.5]  (NaN / Inf in the inputs)
//   bits 55..63  rows delivered
// A term is rounded to the nearest multiple of 2^-35 = 2.9e-11; over b rows and divided by b^2
// that is at most 1.5e-11 / b on the loss.
constexpr double kRowAccScale = 34359738368.0;  // 2^35
constexpr int kRowAccBadShift = 46, kRowAccCountShift = 55;

__device__ __forceinline__ unsigned long long row_acc_of(double term) {
    unsigned long long v = 1ull << kRowAccCountShift;
    if (term >= 0.0 && term <= 4.5) {  // false for NaN
        if (term > 4.0) term = 4.0;
        v += (unsigned long long)__double2ll_rn(term * kRowAccScale);
    } else {
        v += 1ull << kRowAccBadShift;
    }
    return v;
}
__device__ __forceinline__ int row_acc_rows(unsigned long long acc) { return (int)(acc >> kRowAccCountShift); }
// Sum of the terms, NaN if any row's term was not a number in range.
__device__ __forceinline__ double row_acc_sum(unsigned long long acc) {
    if ((acc >> kRowAccBadShift) & 0x1ffull) return NAN;
    return (double)(long long)(acc & ((1ull << kRowAccBadShift) - 1)) / kRowAccScale;
}

// One warp, with the sum of all row terms of module m: the loss (Eq. 1), then optionally one
// evaluation of the freezing rule from the state loaded in L.
__device__ __forceinline__ void finalize_module_finish(const FinCommon &p, int m, double sum_terms, StepLoaded &L,
                                                       int lane) {
    const double b = (double)p.b;
    const float loss = (float)(sum_terms / (b * b));
    if (lane == 0) p.out_losses[m] = loss;
    if (p.fuse_step)
        plasticity_rule_step(p.st, L, m, p.M, p.rule_flags, p.rule_serial, loss, p.lr, p.out_slopes, p.out_mask, lane);
}

// One warp, once every row term of module m is in p.rowloss and visible (the modules of the
// CUDA-core kernel): add them in a fixed order, then as above.
__device__ __forceinline__ void finalize_module_total(const FinCommon &p, int m, int lane) {
    const int b = p.b;
    double v[kMaxB / 32];
#pragma unroll
    for (int j = 0; j < kMaxB / 32; ++j) {
        const int r = lane + 32 * j;
        v[j] = (r < b) ? __ldcg(&p.rowloss[(int64_t)m * kMaxB + r]) : 0.0;
    }
    StepLoaded L;
    if (p.fuse_step) L = plasticity_step_load(p.st, m, lane);  // in flight together with the row terms
    double s = 0.0;
#pragma unroll
    for (int j = 0; j < kMaxB / 32; ++j) s += v[j];
    s = warp_sum_f64(s);
    finalize_module_finish(p, m, s, L, lane);
}

struct FinParams {
    FinCommon c;
    int32_t *tickets;  // [M], zero between calls
};

// Modules whose partial Grams came from the CUDA-core kernel.  grid = (M, ceil(b / 8)).
template <int NC>
__global__ void __launch_bounds__(kFinThreads) finalize_kernel(const FinParams p) {
    const int m = blockIdx.x;
    const SideInfo s0 = p.c.sides[2 * m];
    if (s0.tensor_core || s0.module_units == 0) return;  // finished inside the tensor-core kernel / not evaluated
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = p.c.b;
    const int i = blockIdx.y * kFinRowsPerCta + warp;
    __shared__ int is_last;

    if (i < b) {
        const double s = finalize_row<NC>(p.c, p.c.sides[2 * m], p.c.sides[2 * m + 1], m, i, lane);
        if (lane == 0) p.c.rowloss[(int64_t)m * kMaxB + i] = s;
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
        if (lane == 0) p.tickets[m] = 0;
        finalize_module_total(p.c, m, lane);
    }
}

}  // namespace egeria
