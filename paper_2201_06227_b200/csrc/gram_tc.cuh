// The SP loss (Eq. 1) of all tensor-core modules in ONE launch on sm_100a: partial Gram
// matrices G = A A^T on the 5th-generation tensor cores, then row normalisation, difference
// and Frobenius reduction by the same kernel.
//
// One persistent CTA per SM walks its static list of work units (a K-range of one
// (module, side) tile).  Per 64-element block of the feature axis, one TMA box load
// brings all b rows into a 128-byte-swizzled shared-memory slab; the same slab is
// both the A and the B operand of tcgen05.mma (row block i against row block j,
// i <= j), accumulating in fp32 in tensor memory.  At the end of a unit the
// accumulator is drained to the unit's partial slot in the workspace (L2-resident).
//
// A module is finished by the CTAs that worked on it.  Every unit bumps the module's
// units_done counter.  A CTA that has done all its units goes through the modules it worked
// on: where all units of the module are in (for the module of its last unit it waits briefly),
// its epilogue warps claim rows of G one by one from the module's row cursor, fetch the row
// of every partial into shared memory (the operand ring is idle by then), add them in a
// fixed order, normalise, take the difference, square, and reduce with warp shuffles.  The
// warp that delivers the module's last row adds the row terms in a fixed order and writes the
// loss (and, if asked, advances the freezing rule).  Whoever delivers a module's last unit
// always gets to this point after it, so every module is finished; and the result never
// depends on which warp did what.
//
// The first task of every epilogue warp is planned on the host (Plan::first_task): no claim to
// wait for.  Where that gives every row of the launch a warp of its own (Plan::validate_rows), the
// finish does not go by the counters at all: a partial slot holds a bit pattern no value has
// (kSlotEmpty) except between a launch's store and its read, so a warp fetches its row of every
// partial until none of it is empty -- each 4-byte element is its own flag; no fence, no look
// at a counter, no claim.  Such launches alternate between two sets of slots, and each puts
// back to "empty", at its start, what the launch before wrote into the other set.
//
// Warp roles (448 threads): warp 0 = TMA producer, warp 1 = MMA issuer and TMEM
// owner, warps 2..13 = epilogue (TMEM -> registers -> global, then the finalisation); a warp
// may read only the TMEM lane quarter (warp index mod 4), so three warps share each quarter
// and split its columns.
// Every wait is bounded; on expiry the CTA raises its abort flag, records
// EGERIA_ERR_TIMEOUT in the status word, drains what is in flight and returns.
//
// The kernel is launched as a programmatic dependent of the kernel before it in the stream: a CTA
// gets an SM as soon as that kernel's CTA there has ended and sets itself up while that kernel's
// last CTAs are still running.  Nothing that kernel may have produced is consumed early: the
// producer executes grid_dependency_wait() before its first load, and everything the launches of a
// context share -- partial slots, progress counters, the rule's state, the outputs, the status
// word, the log -- is touched only after it as well.  If the caller vouches that the activations
// were complete before the preceding kernel (early_inputs), the producer does not wait: the next
// evaluation then streams while this one is still finishing its modules.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "finalize.cuh"
#include "plan.h"
#include "ptx_sm100.cuh"

namespace egeria {

constexpr int kEpiWarps = 12;                     // three per TMEM lane quarter
constexpr int kEpiThreads = 32 * kEpiWarps;
constexpr int kTcThreads = 64 + kEpiThreads;      // + TMA producer warp + MMA warp
constexpr uint64_t kWaitLimitNs = 2000000000ull;  // 2 s per wait
constexpr uint64_t kHelpWaitNs = 1000000ull;      // 1 ms: how long a finished CTA waits to help
constexpr int kStatusTimeout = 6;                 // == EGERIA_ERR_TIMEOUT

template <int MODE>
struct TcCfg {
    static constexpr bool kStacked = (MODE == kStacked32 || MODE == kStacked64);
    static constexpr int kBoxRows = (MODE == kStacked32) ? 32 : (MODE == kStacked64 ? 64 : (MODE == kSingle1 ? 128 : 256));
    static constexpr int kSlabRows = kStacked ? 2 * kBoxRows : kBoxRows;   // rows of one 64-column slab
    static constexpr int kSlabBytes = kSlabRows * 128;
    // Slabs per pipeline stage.  The 8 KB slabs of kStacked32 go six to a stage: with 16 KB stages
    // the per-stage hand-shakes (not the loads) set the pace there, 20 % slower on 150 MB of input.
    static constexpr int kKbPerStage = (MODE == kStacked32) ? 6 : 1;
    static constexpr int kStageBytes = kSlabBytes * kKbPerStage;           // 48 KB, 16 KB, 16 KB, 32 KB
    static constexpr int kStages = (MODE == kStacked32) ? 4 : (MODE == kSingle2 ? 6 : 12);  // 192 KB of loads in flight
    static constexpr int kAccCols = (MODE == kStacked32) ? 64 : (MODE == kSingle2 ? 384 : 128);
    static constexpr int kAccStages = (MODE == kSingle2) ? 1 : 2;
    static constexpr int kTmemCols = (MODE == kStacked32) ? 128 : (MODE == kSingle2 ? 512 : 256);
    static constexpr int kNC = (MODE == kStacked32) ? 1 : (MODE == kStacked64 ? 2 : (MODE == kSingle1 ? 4 : 8));
    static constexpr int kSmemBytes =
        kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/ + kEpiWarps * 2 * (int)sizeof(SideInfo);
};

struct TcParams {
    const CUtensorMap *tmaps;  // [2 * M]: A_T and A_R of every module (device memory)
    const Unit *units;         // tensor-core units
    const int32_t *cta_begin;  // [gridDim.x + 1]
    const CtaHelp *cta_help;   // [gridDim.x] planned help at the end of the launch, or nullptr
    // Front-only evaluation (else nullptr): the word that holds the number of frozen modules; the
    // work split of front f starts at cta_begin + f * cta_stride, and with every module frozen
    // there is no work.
    const unsigned long long *front_word;
    int32_t cta_stride;
    float *slots;              // partial Gram slots
    int32_t *status;           // device status word
    FinCounters *ctr;          // [M] progress counters of this launch (all zero at launch)
    FinCounters *ctr_next;     // [M] the set the next launch will use: cleared here
    CtaLog *log;               // [gridDim.x] what each CTA reports about this launch, or nullptr
    uint32_t serial;           // tag of this launch in the log
    // Test hook for the give-up path (0 in every ordinary launch).  1: the TMA producer of CTA 0
    // issues no load at all, so its MMA warp's wait for the first stage runs out.  2: the MMA warp of
    // CTA 0 stops after its first stage, so no accumulator is ever complete and (given more blocks
    // than pipeline stages) the producer runs out of free stages with loads in flight behind it.
    // Either way the waits run out, the CTA leaves through the give-up path and the kernel returns.
    // 1: the activations were complete before the kernel that precedes this launch in the stream
    // (the caller's promise, EGERIA_FLAG_OVERLAP), so the loads need not wait for that kernel.
    uint32_t early_inputs;
    uint32_t test_stall;
    uint64_t wait_limit_ns;    // limit of every bounded wait of this launch (kWaitLimitNs, shorter for the hook)
    uint4 *empty_ptr;          // the set of slots this launch does NOT use: what the launch before wrote there
    uint32_t empty_n;          // ... is put back to kSlotEmpty at the start (empty_n 16-byte pieces; 0: nothing)
    int64_t empty_floats;      // floats in that set (the checked build compares empty_n with it)
    const int32_t *first_task; // [gridDim.x * kEpiWarps] the task each epilogue warp starts the finish with
                               // ((module << 16) | task, -1: none), or nullptr; front-only: one table per front
    int32_t first_stride;      // front-only: entries from one front's table to the next
    int32_t n_units;           // entries of `units` (the checked build compares unit indices with it)
    int32_t M;
    int32_t n_active;          // tensor-core modules this launch evaluates (front-only: 1)
    FinCommon fin;             // slots, sides, b, outputs, freezing-rule state
};

namespace detail {
__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory"); }
// All epilogue threads: AND of `pred` over them.
__device__ __forceinline__ bool epi_bar_and(bool pred) {
    uint32_t out;
    asm volatile(
        "{\n\t"
        ".reg .pred p, q;\n\t"
        "setp.ne.b32 p, %1, 0;\n\t"
        "bar.red.and.pred q, 1, %2, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t"
        "}"
        : "=r"(out)
        : "r"((uint32_t)pred), "n"(kEpiThreads)
        : "memory");
    return out != 0;
}
__device__ __forceinline__ int ld_acquire(const int32_t *p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// One 32-row x 32-column piece of an accumulator, as one epilogue warp sees it: where it is in
// tensor memory and where this lane's row of it goes in the partial slot.
struct Chunk {
    uint32_t col;      // first TMEM column
    float *dst;        // this lane's 32 floats in the slot
    bool valid;        // this lane's row is a row of G
    int mirror_c0;     // kSingle2: first column of a G01 chunk that is also written transposed, else -1
};

// Chunk k of the accumulator of one unit, for the warp of TMEM lane quarter q.  False if there
// is no such chunk (warp-uniform).  Layouts per mode:
//   kStacked32: one M = 64 accumulator: rows 0..31 x cols 0..31 = G_T, rows 32..63 x cols 32..63 = G_R
//               (an M = 64 accumulator keeps row r in TMEM lane (r % 16) + 32 * (r / 16): the lower
//               16 lanes of every lane quarter)
//   kStacked64: rows 0..63 x cols 0..63 = G_T, rows 64..127 x cols 64..127 = G_R
//   kSingle1:   rows 0..127 x cols 0..127 = G
//   kSingle2:   cols 0..255 = rows 0..127 of G (all 256 columns); cols 256..383 = G11
template <int MODE>
__device__ __forceinline__ bool chunk_of(int k, int q, int lane, int b, float *slot, Chunk &ch) {
    ch.mirror_c0 = -1;
    if (MODE == kStacked32) {
        // quarter q holds accumulator rows 16 q .. 16 q + 15: quarters 0, 1 = G_T, 2, 3 = G_R
        const int side = q >> 1, r = 16 * (q & 1) + lane;
        if (k != 0 || 16 * (q & 1) >= b) return false;
        ch.col = side * 32;
        ch.dst = slot + side * 32 * 32 + r * 32;
        ch.valid = lane < 16 && r < b;
        return true;
    } else if (MODE == kStacked64) {
        const int side = q >> 1, r = (q & 1) * 32 + lane, c0 = 32 * k;
        if (k >= 2 || c0 >= b || (q & 1) * 32 >= b) return false;
        ch.col = side * 64 + c0;
        ch.dst = slot + side * 64 * 64 + r * 64 + c0;
        ch.valid = r < b;
        return true;
    } else if (MODE == kSingle1) {
        // pieces of 16 columns: eight of them split 3 + 3 + 2 over the quarter's three warps (four
        // pieces of 32 would be 2 + 1 + 1, and the warp with two is what the others wait for);
        // every piece up to b rounded up to 32 columns is stored, as in the other modes
        const int r = q * 32 + lane, c0 = 16 * k;
        if (k >= 8 || c0 >= ((b + 31) & ~31) || q * 32 >= b) return false;
        ch.col = c0;
        ch.dst = slot + r * 128 + c0;
        ch.valid = r < b;
        return true;
    } else {
        const int r = q * 32 + lane;  // 0..127, always < b in this mode
        if (k < 8) {
            const int c0 = 32 * k;
            if (c0 >= b) return false;
            ch.col = c0;
            ch.dst = slot + r * 256 + c0;
            ch.valid = true;
            if (c0 >= 128) ch.mirror_c0 = c0;
            return true;
        }
        const int l = 32 * (k - 8);
        if (k >= 12 || 128 + l >= b || 128 + q * 32 >= b) return false;
        ch.col = 256 + l;
        ch.dst = slot + (128 + r) * 256 + 128 + l;
        ch.valid = 128 + r < b;
        return true;
    }
}

// First existing chunk among k, k + 3, k + 6, ... (k is advanced to it).  Warp-uniform.
template <int MODE>
__device__ __forceinline__ bool next_chunk(int &k, int q, int lane, int b, float *slot, Chunk &ch) {
    constexpr int kChunks = (MODE == kStacked32) ? 1 : (MODE == kStacked64 ? 2 : (MODE == kSingle1 ? 8 : 12));
    for (; k < kChunks; k += 3)
        if (chunk_of<MODE>(k, q, lane, b, slot, ch)) return true;
    return false;
}

// Tasks of module m that its cursor hands out (the others have a warp each from the start).
__device__ __forceinline__ int module_cursor_tasks(const TcParams &p, int m) {
    const SideInfo si = p.fin.sides[2 * m];
    return si.n_tasks - si.n_static;
}

// One warp: do task `first` of module m (if not negative), then take tasks from the module's
// cursor until none is left.  A task is a row of G, or -- a module evaluated alone and cut into many
// partials at b <= 64, where one warp per row would add a hundred partial rows one after the
// other with most warps idle -- a (row, chunk) pair (see finalize_row_chunk; measured 66 -> 55 us
// at b = 64, 27 -> 23 us at b = 32; at b > 64 the chunk sums are 2 to 4 KB per task and the
// scratch traffic eats the gain).  The claim of the next task is in flight while the current one
// is worked on; the rows' terms are delivered together.  `stage` is kFinStageBytes of shared
// memory for this warp alone.
template <int NC>
__device__ __forceinline__ void finish_module_rows(const TcParams &p, int m, int lane, float *stage,
                                                   volatile int *abort_flag, int first = -1,
                                                   const SideInfo *cached = nullptr) {
    const int b = p.fin.b;
    FinCounters *c = p.ctr + m;
    unsigned long long mine = 0;  // this warp's rows and their terms, packed (row_acc_of)
    int r = 0;
    if (first < 0 && lane == 0) r = atomicAdd(&c->row_cursor, 1);
    // (in flight with the claim; a first task's were fetched into shared memory long ago)
    const SideInfo sT = cached ? cached[0] : p.fin.sides[2 * m], sR = cached ? cached[1] : p.fin.sides[2 * m + 1];
    const int n_tasks = sT.n_tasks, n_static = sT.n_static;
    r = (first < 0) ? n_static + __shfl_sync(0xffffffffu, r, 0) : first;
    if (!eg_check(n_static >= 0 && n_static <= n_tasks && n_tasks >= b && n_tasks % b == 0 && r >= 0 &&
                      sT.n_slots >= 0 && sR.n_slots >= 0 && sT.first_slot >= 0 && sR.first_slot >= 0 &&
                      ((int64_t)sT.first_slot + sT.n_slots) * p.fin.slot_floats <= p.fin.slots_floats &&
                      ((int64_t)sR.first_slot + sR.n_slots) * p.fin.slot_floats <= p.fin.slots_floats,
                  p.status, kCheckTask, ((long long)m << 32) | (uint32_t)r))
        return;
    if (n_tasks > b) {
        // (row, chunk) tasks: task v is chunk v % n_chunks of row v / n_chunks
        const int n_chunks = n_tasks / b;
        while (r < n_tasks) {
            int r_next = 0;
            if (lane == 0) r_next = atomicAdd(&c->row_cursor, 1);
            const int row = r / n_chunks, ch = r % n_chunks;
            if (!finalize_row_chunk<NC>(p.fin, sT, sR, row, ch, n_chunks, lane, stage, abort_flag)) return;
            __threadfence();  // every lane's sums, before the count
            __syncwarp();
            int done = 0;
            if (lane == 0) done = atomicAdd(&c->row_chunks_done[row], 1);
            done = __shfl_sync(0xffffffffu, done, 0);
            if (done == n_chunks - 1) {
                __threadfence();
                mine += row_acc_of(finalize_row_from_chunks<NC>(p.fin, m, row, n_chunks, lane));
            }
            r = n_static + __shfl_sync(0xffffffffu, r_next, 0);
        }
    } else {
        while (r < b) {
            int r_next = 0;
            if (lane == 0) r_next = atomicAdd(&c->row_cursor, 1);
            bool ok;
            const double term = finalize_row_staged<NC>(p.fin, sT, sR, m, r, lane, stage, abort_flag, ok);
            if (!ok) return;
            mine += row_acc_of(term);
            r = n_static + __shfl_sync(0xffffffffu, r_next, 0);
        }
    }
    if (mine == 0) return;
    // One atomic add delivers the terms and says whether these were the module's last rows; what
    // the rule needs is loaded meanwhile (only the last warp uses it).
    unsigned long long before = 0;
    if (lane == 0) before = atomicAdd(&c->row_acc, mine);
    StepLoaded L;
    if (p.fin.fuse_step) L = plasticity_step_load(p.fin.st, m, lane);
    before = __shfl_sync(0xffffffffu, before, 0);
    const unsigned long long all = before + mine;
    if (row_acc_rows(all) == b) finalize_module_finish(p.fin, m, row_acc_sum(all), L, lane);
}
}  // namespace detail

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
    // where the partials of each epilogue warp's first task are (two SideInfo per warp), fetched early
    SideInfo *side_cache = reinterpret_cast<SideInfo *>(smem_aligned + Cfg::kStages * Cfg::kStageBytes + 256);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    int u_begin = 0, u_end = 0;
    bool all_frozen = false;  // front-only evaluation with nothing left to monitor
    const int32_t *first_task = p.first_task;
    {
        const int32_t *cta_begin = p.cta_begin;
        if (p.front_word) {
            ptx::grid_dependency_wait();
            const int front = (int)(uint32_t)*reinterpret_cast<const volatile unsigned long long *>(p.front_word);
            all_frozen = (front >= p.M);
            cta_begin += (int64_t)(all_frozen ? 0 : front) * p.cta_stride;
            if (first_task) first_task += (int64_t)(all_frozen ? 0 : front) * p.first_stride;
        }
        if (!all_frozen) {
            u_begin = cta_begin[blockIdx.x];
            u_end = cta_begin[blockIdx.x + 1];
        }
        if (!eg_check(u_begin >= 0 && u_begin <= u_end && u_end <= p.n_units, p.status, kCheckUnitRange,
                      ((long long)u_begin << 32) | (uint32_t)u_end))
            u_begin = u_end = 0;
    }

    // The launch after this one may begin (its CTAs get an SM when one of ours ends).  A front-only
    // launch reads the front the launch before it wrote, so it waits for that one here and now.
    ptx::grid_launch_dependents();

    if (threadIdx.x == 0) {
        for (int s = 0; s < Cfg::kStages; ++s) {
            ptx::mbar_init(full0 + 8 * s, 1);
            ptx::mbar_init(empty0 + 8 * s, 1);
        }
        for (int s = 0; s < Cfg::kAccStages; ++s) {
            ptx::mbar_init(accfull0 + 8 * s, 1);
            ptx::mbar_init(accempty0 + 8 * s, kEpiWarps);  // one arrival per epilogue warp
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
            // Whatever wrote the activations must have ended before the first load -- unless the caller
            // vouches that it was not the kernel before this one.
            if (!p.early_inputs) ptx::grid_dependency_wait();
            const uint64_t policy = ptx::l2_policy_evict_first();
            uint32_t stage = 0, phase = 0;
            uint32_t issued = 0;
            bool ok = true;
            int last_module = -1;
            const int u_stop = (p.test_stall == 1 && blockIdx.x == 0) ? u_begin : u_end;  // test hook: no loads
            for (int ui = u_begin; ui < u_stop && ok; ++ui) {
                const Unit u = p.units[ui];
                if (!eg_check(u.module >= 0 && u.module < p.M && u.kb0 >= 0 && u.nkb >= 1 && u.side >= 0 && u.side <= 2,
                              p.status, kCheckUnit, ui)) {
                    ok = false;
                    break;
                }
                const CUtensorMap *tm_t = p.tmaps + 2 * u.module;
                const CUtensorMap *tm_r = tm_t + 1;
                if (u.module != last_module) {
                    ptx::tensormap_acquire(tm_t);
                    ptx::tensormap_acquire(tm_r);
                    last_module = u.module;
                }
                const CUtensorMap *tm_side = (u.side == 1) ? tm_r : tm_t;
                const int kb_end = u.kb0 + u.nkb;
                for (int kb = u.kb0; kb < kb_end; kb += Cfg::kKbPerStage) {
                    if (!ptx::mbar_wait_bounded(empty0 + 8 * stage, phase ^ 1u, abort_flag, p.wait_limit_ns)) {
                        ok = false;
                        break;
                    }
                    if (!eg_check(stage < (uint32_t)Cfg::kStages, p.status, kCheckStage, stage)) {
                        ok = false;
                        break;
                    }
                    const uint32_t dst = smem_base + stage * Cfg::kStageBytes;
                    const uint32_t bar = full0 + 8 * stage;
                    const int nk = (kb_end - kb < Cfg::kKbPerStage) ? kb_end - kb : Cfg::kKbPerStage;
                    ptx::mbar_arrive_expect_tx(bar, (uint32_t)nk * Cfg::kSlabBytes);
#pragma unroll
                    for (int j = 0; j < Cfg::kKbPerStage; ++j) {
                        if (j >= nk) break;
                        const uint32_t slab = dst + j * Cfg::kSlabBytes;
                        if (Cfg::kStacked) {
                            ptx::tma_load_2d(slab, tm_t, (kb + j) * kKBlock, 0, bar, policy);
                            ptx::tma_load_2d(slab + Cfg::kBoxRows * 128, tm_r, (kb + j) * kKBlock, 0, bar, policy);
                        } else {
                            ptx::tma_load_2d(slab, tm_side, (kb + j) * kKBlock, 0, bar, policy);
                        }
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
                        if (ptx::globaltimer_ns() - t0 > p.wait_limit_ns) break;
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc64x64 = ptx::make_idesc_bf16_f32(64, 64);
            constexpr uint32_t idesc128 = ptx::make_idesc_bf16_f32(128, 128);
            constexpr uint32_t idesc256 = ptx::make_idesc_bf16_f32(128, 256);
            // start of the streaming the launch log reports: the arrival of the first stage (not the
            // kernel's entry: a programmatic dependent enters while the launch before is still running
            // and then waits for it, each CTA for a different time)
            uint64_t t_entry = ptx::globaltimer_ns();
            uint32_t blocks_done = 0;
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            bool any_mma = false;
            const bool stall_after_first_stage = (p.test_stall == 2 && blockIdx.x == 0);  // test hook
            for (int ui = u_begin; ui < u_end && ok; ++ui) {
                const Unit u = p.units[ui];
                if (!ptx::mbar_wait_bounded(accempty0 + 8 * acc, acc_phase ^ 1u, abort_flag, p.wait_limit_ns)) {
                    ok = false;
                    break;
                }
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + acc * Cfg::kAccCols;
                for (int kb = 0; kb < u.nkb; kb += Cfg::kKbPerStage) {
                    if (!ptx::mbar_wait_bounded(full0 + 8 * stage, phase, abort_flag, p.wait_limit_ns)) {
                        ok = false;
                        break;
                    }
                    ptx::tc_fence_after_sync();
                    if (!any_mma && p.log) t_entry = ptx::globaltimer_ns();
                    if (stall_after_first_stage && any_mma) {  // stop here: no further stage is released
                        ok = false;
                        break;
                    }
                    const int nk = (u.nkb - kb < Cfg::kKbPerStage) ? u.nkb - kb : Cfg::kKbPerStage;
#pragma unroll
                    for (int j = 0; j < Cfg::kKbPerStage; ++j) {
                        if (j >= nk) break;
                        const uint32_t slab = smem_base + stage * Cfg::kStageBytes + j * Cfg::kSlabBytes;
#pragma unroll
                        for (int k = 0; k < kKBlock / 16; ++k) {
                            const uint32_t accum = (kb > 0 || j > 0 || k > 0) ? 1u : 0u;
                            const uint64_t lo = ptx::make_desc_k_sw128(slab + k * 32);
                            if (MODE == kSingle2) {
                                const uint64_t hi = ptx::make_desc_k_sw128(slab + 128 * 128 + k * 32);
                                // [G00 | G01] = rows 0..127 against rows 0..255
                                ptx::mma_bf16_ss(d_tmem, lo, lo, idesc256, accum);
                                // G11 = rows 128..255 against themselves
                                ptx::mma_bf16_ss(d_tmem + 256, hi, hi, idesc128, accum);
                            } else if (MODE == kStacked32) {
                                // the whole 64-row slab against itself
                                ptx::mma_bf16_ss(d_tmem, lo, lo, idesc64x64, accum);
                            } else {
                                // kStacked64 too: two M = 64 MMAs without the cross terms draw less power but
                                // take longer (the issue rate of small MMAs, not their size, sets the pace)
                                ptx::mma_bf16_ss(d_tmem, lo, lo, idesc128, accum);
                            }
                        }
                    }
                    any_mma = true;
                    ptx::mma_commit(empty0 + 8 * stage);  // stage free once these MMAs have read it
                    if (++stage == Cfg::kStages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                if (!ok) break;
                blocks_done += (uint32_t)u.nkb;
                ptx::mma_commit(accfull0 + 8 * acc);  // accumulator complete
                if (++acc == Cfg::kAccStages) {
                    acc = 0;
                    acc_phase ^= 1u;
                }
            }
            if (p.log) {
                ptx::grid_dependency_wait();  // the log is shared with the launch before
                CtaLog e;
                e.serial = p.serial;
                e.duration_ns = (uint32_t)(ptx::globaltimer_ns() - t_entry);
                e.blocks = ok ? blocks_done : 0u;
                e.pad = 0;
                p.log[blockIdx.x] = e;
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
        const int q = warp & 3;           // TMEM lane quarter this warp may read
        const int part = (warp - 2) >> 2;  // which third of the quarter's columns this warp drains
        const int b = p.fin.b;
        const bool epi_leader = (threadIdx.x == 64);
        // asked for now, needed at the end of the launch
        const CtaHelp planned_help = p.cta_help ? p.cta_help[blockIdx.x] : CtaHelp{-1, 0};
        const int my_first = (first_task && !all_frozen) ? first_task[blockIdx.x * kEpiWarps + (warp - 2)] : -1;
        if (my_first >= 0 && (!kCheckedBuild || (my_first >> 16) < p.M) && lane < 16)  // 64 bytes: both sides of the module
            reinterpret_cast<int32_t *>(side_cache + 2 * (warp - 2))[lane] =
                reinterpret_cast<const int32_t *>(p.fin.sides + 2 * (my_first >> 16))[lane];
        uint32_t acc = 0, acc_phase = 0;
        bool aborted = false;
        bool prior_done = false;  // the launch before has ended: the shared workspace is ours
        // Once the launch before has ended: the counters of the NEXT launch start at zero (the set
        // this launch does not use; the launch before used it until its end).
        auto claim_workspace = [&]() {
            if (prior_done) return;
            ptx::grid_dependency_wait();
            prior_done = true;
            int32_t *z = reinterpret_cast<int32_t *>(p.ctr_next);
            const int n = p.M * (int)(sizeof(FinCounters) / sizeof(int32_t));
            for (int i = blockIdx.x * kEpiThreads + (threadIdx.x - 64); i < n; i += gridDim.x * kEpiThreads) z[i] = 0;
            // ... and the partial slots the launch before wrote and read are empty again for the
            // launch after this one (this launch uses the other set)
            const uint4 empty = make_uint4(kSlotEmpty, kSlotEmpty, kSlotEmpty, kSlotEmpty);
            if (eg_check((int64_t)p.empty_n * 4 <= p.empty_floats, p.status, kCheckEmpty, p.empty_n))
                for (uint32_t i = blockIdx.x * kEpiThreads + (threadIdx.x - 64); i < p.empty_n; i += gridDim.x * kEpiThreads)
                    p.empty_ptr[i] = empty;
        };
        for (int ui = u_begin; ui < u_end; ++ui) {
            const Unit u = p.units[ui];
            const bool got = ptx::mbar_wait_bounded(accfull0 + 8 * acc, acc_phase, abort_flag, p.wait_limit_ns);
            if (!detail::epi_bar_and(got)) {  // the epilogue warps leave together
                aborted = true;
                break;
            }
            claim_workspace();  // the first unit's streaming is over by now; usually so is the launch before
            ptx::tc_fence_after_sync();
            const bool slot_ok = eg_check(u.slot >= 0 && ((int64_t)u.slot + 1) * p.fin.slot_floats <= p.fin.slots_floats &&
                                              u.module >= 0 && u.module < p.M,
                                          p.status, kCheckUnit, ui);
            float *slot = p.slots + (int64_t)(slot_ok ? u.slot : 0) * p.fin.slot_floats;
            const uint32_t t_row = tmem_base + acc * Cfg::kAccCols + ((uint32_t)(q * 32) << 16);
            // This warp's share of the accumulator: 32 x 32 chunks part, part + 3, ...; the load of
            // the next chunk is in flight while the current one is stored.
            detail::Chunk ch, nx;
            int k = part;
            bool have = slot_ok && detail::next_chunk<MODE>(k, q, lane, b, slot, ch);
            uint32_t v[32], w[32];
            constexpr int kCols = (MODE == kSingle1) ? 16 : 32;  // columns of one piece
            auto load_piece = [&](uint32_t col) {
                if (MODE == kSingle1)
                    ptx::tmem_ld_32x16(t_row + col, w);
                else
                    ptx::tmem_ld_32x32(t_row + col, w);
            };
            if (have) load_piece(ch.col);
            while (have) {
                ptx::tmem_ld_wait();
#pragma unroll
                for (int c = 0; c < kCols; ++c) v[c] = (w[c] == kSlotEmpty) ? kCanonicalNan : w[c];  // never stored as a value
                k += 3;
                const bool have_next = detail::next_chunk<MODE>(k, q, lane, b, slot, nx);
                if (have_next) load_piece(nx.col);
                if (kCheckedBuild) {
                    const int64_t off = ch.dst - slot;
                    const bool fine = ch.col + kCols <= (uint32_t)Cfg::kAccCols &&
                                      (!ch.valid || (off >= 0 && off + kCols <= p.fin.slot_floats));
                    if (!eg_check(__all_sync(0xffffffffu, fine), p.status, ch.col + kCols <= (uint32_t)Cfg::kAccCols ? kCheckSlotStore : kCheckTmem, off))
                        ch.valid = false;
                }
                if (ch.valid) {
#pragma unroll
                    for (int c = 0; c < kCols; c += 8) ptx::st_global_v8(ch.dst + c, v + c);
                }
                if (MODE == kSingle2 && ch.mirror_c0 >= 0) {
                    // mirror G01 into the lower-left block: lanes write consecutive floats
                    const int r = q * 32 + lane;
#pragma unroll
                    for (int c = 0; c < 32; ++c)
                        if (ch.mirror_c0 + c < b) slot[(ch.mirror_c0 + c) * 256 + r] = __uint_as_float(v[c]);
                }
                ch = nx;
                have = have_next;
            }
            // Hand the accumulator back before anything else: the next unit's MMAs can start.
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(accempty0 + 8 * acc);
            if (++acc == Cfg::kAccStages) {
                acc = 0;
                acc_phase ^= 1u;
            }

            // Publish the partial: every thread's stores, then one count for the unit.  (Where the
            // readers validate what they read, the count is a hint and needs no fence before it.)
            if (!p.fin.sentinel) __threadfence();
            detail::epi_bar_sync();
            if (epi_leader && slot_ok) atomicAdd(&p.ctr[u.module].units_done, 1);
        }
        claim_workspace();  // (CTAs without a unit, and the counters' clearing if the wait above gave up)
        if (all_frozen && blockIdx.x == 0 && warp == 2) {
            // nothing is monitored any more: the rule only reports (prefix mask of ones, final slopes)
            StepLoaded L = plasticity_step_load(p.fin.st, p.M - 1, lane);
            plasticity_rule_step(p.fin.st, L, p.M - 1, p.M, p.fin.rule_flags, p.fin.rule_serial, 0.f, p.fin.lr,
                                 p.fin.out_slopes, p.fin.out_mask, lane);
        }
        if (!aborted) {
            // All of this CTA's units are in and its pipeline is idle, so the operand ring is free:
            // each epilogue warp takes kFinStageBytes of it as its staging area and helps finish the
            // modules this CTA worked on, as far as they are complete.
            static_assert(kEpiWarps * kFinStageBytes <= Cfg::kStages * Cfg::kStageBytes, "ring too small to stage");
            float *stage = reinterpret_cast<float *>(smem_aligned + (warp - 2) * kFinStageBytes);
            ptx::fence_proxy_async();  // the ring was last touched by TMA and the tensor cores
            // The task planned for this warp first (Plan::first_task): no cursor to ask, and no
            // counter to wait for either -- the partial rows say themselves whether they are here.
            if (my_first >= 0) {
                const int fm = my_first >> 16;
                __syncwarp();  // (side_cache was written by lanes 0..15)
                bool go = eg_check(fm < p.M && (my_first & 0xffff) < side_cache[2 * (warp - 2)].n_static &&
                                       side_cache[2 * (warp - 2)].n_static <= side_cache[2 * (warp - 2)].n_tasks,
                                   p.status, kCheckFirstTask, my_first);
                if (go && !p.fin.sentinel) {
                    // ... by the counter, then: this task is nobody else's, so the wait is not a
                    // courtesy and runs to the launch's limit
                    const int total = p.fin.sides[2 * fm].module_units;
                    const uint64_t t_wait = ptx::globaltimer_ns();
                    int state = 0;  // 1 complete, 2 gave up
                    while (state == 0) {
                        if (lane == 0) {
                            if (detail::ld_acquire(&p.ctr[fm].units_done) >= total)
                                state = 1;
                            else if (*abort_flag || ptx::globaltimer_ns() - t_wait > p.wait_limit_ns) {
                                *abort_flag = 1;
                                state = 2;
                            }
                        }
                        state = __shfl_sync(0xffffffffu, state, 0);
                        if (state == 0) __nanosleep(100);
                    }
                    go = (state == 1);
                    __threadfence();
                }
                __syncwarp();
                if (go)
                    detail::finish_module_rows<Cfg::kNC>(p, fm, lane, stage, abort_flag, my_first & 0xffff,
                                                         side_cache + 2 * (warp - 2));
            }
            // Planned help: the last few warps of a CTA whose own module has warps to spare
            // start with the rows of a module that is short of them (see CtaHelp), once that module
            // is complete; the wait for it is a courtesy like the others.
            {
                const CtaHelp h = planned_help;
                if (h.warps > 0 && warp - 2 >= kEpiWarps - h.warps && !(my_first >= 0 && (my_first >> 16) == h.module)) {
                    const int total = p.fin.sides[2 * h.module].module_units;
                    const uint64_t t_wait = ptx::globaltimer_ns();
                    int state = 0;  // 1 complete, 2 gave up
                    while (state == 0) {
                        if (lane == 0) {
                            if (detail::ld_acquire(&p.ctr[h.module].units_done) >= total)
                                state = 1;
                            else if (*abort_flag || ptx::globaltimer_ns() - t_wait > kHelpWaitNs)
                                state = 2;
                        }
                        state = __shfl_sync(0xffffffffu, state, 0);
                        if (state == 0) __nanosleep(100);
                    }
                    if (state == 1) {
                        __threadfence();
                        detail::finish_module_rows<Cfg::kNC>(p, h.module, lane, stage, abort_flag);
                    }
                }
            }
            // The modules this CTA worked on, 32 units at a time: lane j looks after the module of
            // unit j (the first unit of each module only; a module's units are adjacent).  The warp
            // polls their counters together, finishes rows wherever a module is complete and has
            // rows nobody has claimed -- warps start at different modules, so that a CTA whose range
            // covers parts of several modules works on all of them at once -- and waits (a while)
            // for those that are not complete yet.  The wait is a courtesy, see above.
            for (int base = u_begin; base < u_end; base += 32) {
                int my_m = -1, my_total = 0, my_tasks = b;
                if (base + lane < u_end) {
                    my_m = p.units[base + lane].module;
                    if (base + lane > u_begin && p.units[base + lane - 1].module == my_m) my_m = -1;
                }
                if (my_m >= 0) {
                    my_total = p.fin.sides[2 * my_m].module_units;
                    my_tasks = detail::module_cursor_tasks(p, my_m);
                    // With many CTAs on a module and few rows, most claims would find nothing and only
                    // crowd the cursor: as many warps of this CTA as its share of the rows (or of the
                    // (row, chunk) tasks), plus one.
                    const int ctas_on_m = Cfg::kStacked ? my_total : (my_total + 1) / 2;
                    if (my_tasks <= 0 || warp - 2 > (my_tasks + ctas_on_m - 1) / ctas_on_m) my_m = -1;
                }
                uint32_t pending = __ballot_sync(0xffffffffu, my_m >= 0);
                uint64_t t_wait = ptx::globaltimer_ns();
                while (pending) {
                    bool ready = false;
                    int left = 0;
                    if ((pending >> lane) & 1u) {
                        const int done = detail::ld_acquire(&p.ctr[my_m].units_done);
                        const int cur = detail::ld_acquire(&p.ctr[my_m].row_cursor);
                        ready = (done >= my_total);
                        left = my_tasks - cur;
                    }
                    pending &= ~__ballot_sync(0xffffffffu, ready && left <= 0);  // complete, every row claimed
                    const uint32_t cand = __ballot_sync(0xffffffffu, ready && left > 0);
                    if (cand) {
                        const int pick = (int)__fns(cand, 0, 1 + (warp - 2) % __popc(cand));
                        const int m = __shfl_sync(0xffffffffu, my_m, pick);
                        __threadfence();
                        detail::finish_module_rows<Cfg::kNC>(p, m, lane, stage, abort_flag);  // returns when no row is left to claim
                        pending &= ~(1u << pick);
                        t_wait = ptx::globaltimer_ns();
                    } else if (pending) {
                        int stop = 0;
                        if (lane == 0) stop = (*abort_flag != 0) || (ptx::globaltimer_ns() - t_wait > kHelpWaitNs);
                        if (__shfl_sync(0xffffffffu, stop, 0)) break;
                        __nanosleep(100);
                    }
                }
            }
            // Then look at all the other modules, a few times: where one is complete and still has
            // many rows nobody has claimed (few CTAs worked on it, so its rows go slowly), lend a
            // hand to the one with the most rows left.
            // (With fewer rows in all than half the epilogue warps of the grid there is nothing to
            // lend a hand with, and the look itself would be the last thing the kernel waits for.)
            // (Nor where every task had a warp of its own from the start: p.fin.sentinel.)
            const int help_rounds =
                (p.fin.sentinel || 2 * (int64_t)b * p.n_active < (int64_t)gridDim.x * kEpiWarps) ? 0 : 3;
            for (int round = 0; round < help_rounds; ++round) {
                int best_left = 0, best_m = -1;
                for (int mm = lane; mm < p.M; mm += 32) {
                    const SideInfo si = p.fin.sides[2 * mm];
                    if (!si.tensor_core || si.module_units == 0) continue;
                    const int done = detail::ld_acquire(&p.ctr[mm].units_done);
                    const int cur = detail::ld_acquire(&p.ctr[mm].row_cursor);
                    const int left = (done >= si.module_units) ? si.n_tasks - si.n_static - cur : 0;
                    if (left > best_left) {
                        best_left = left;
                        best_m = mm;
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    const int ol = __shfl_xor_sync(0xffffffffu, best_left, o);
                    const int om = __shfl_xor_sync(0xffffffffu, best_m, o);
                    if (ol > best_left || (ol == best_left && om > best_m)) {
                        best_left = ol;
                        best_m = om;
                    }
                }
                if (best_left < 2 * kEpiWarps) break;  // not worth a round trip: its own CTAs are about done
                __threadfence();
                detail::finish_module_rows<Cfg::kNC>(p, best_m, lane, stage, abort_flag);
            }
        }
    }

    // ---------------------------------------------------------------- teardown
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    if (warp == 1) ptx::tmem_dealloc(tmem_base, Cfg::kTmemCols);
    if (threadIdx.x == 0 && *abort_flag) {
        ptx::grid_dependency_wait();
        atomicMax(p.status, kStatusTimeout);
    }
}

}  // namespace egeria
