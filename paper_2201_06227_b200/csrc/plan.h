// Work split of one plasticity evaluation: plain host/device structs and the
// pure host routine that builds them.  No CUDA calls in here.
#pragma once
#include <stdint.h>

#include <vector>

#ifndef __CUDACC__
#define __host__
#define __device__
#endif

namespace egeria {

// The feature axis is cut into blocks of 64 bf16 values (128 bytes: one swizzle row).
constexpr int kKBlock = 64;

// How the b rows of A_T / A_R are laid into MMA tiles.
//   kStacked32 : b <= 32.  One tile per module: A_T in rows 0..31 and A_R in rows 32..63 of a
//                64-row slab, one 64x64 MMA; the two diagonal 32x32 blocks are G_T and G_R.
//   kStacked64 : b <= 64.  Same with 64 rows per side: 128-row slab, one 128x128 MMA.
//   kSingle1   : b <= 128. One tile per (module, side): 128-row slab, one 128x128 MMA.
//   kSingle2   : b <= 256. One tile per (module, side): 256-row slab, the upper triangle of
//                2x2 blocks of 128 (G00|G01 as one 128x256 MMA, G11 as one 128x128 MMA).
enum Mode : int { kStacked32 = 0, kStacked64 = 1, kSingle1 = 2, kSingle2 = 3 };
constexpr int kNumModes = 4;

__host__ __device__ inline int mode_of_b(int b) {
    return b <= 32 ? kStacked32 : (b <= 64 ? kStacked64 : (b <= 128 ? kSingle1 : kSingle2));
}
__host__ __device__ inline bool mode_is_stacked(int mode) { return mode <= kStacked64; }
// Row pitch (floats) of a partial Gram; for the stacked modes also the rows per side.
__host__ __device__ inline int pitch_of_mode(int mode) {
    return mode == kStacked32 ? 32 : (mode == kStacked64 ? 64 : (mode == kSingle1 ? 128 : 256));
}
// fp32 values of one partial-Gram slot ([2][h][h] when stacked, else [pitch][pitch]).
__host__ __device__ inline int64_t slot_floats_of_mode(int mode) {
    const int64_t p = pitch_of_mode(mode);
    return mode_is_stacked(mode) ? 2 * p * p : p * p;
}

// One work unit: a K-range of one tile, done by one CTA, leaving one partial Gram in `slot`.
struct Unit {
    int32_t module;
    int32_t side;  // 0 = A_T, 1 = A_R, 2 = both (stacked modes)
    int32_t kb0;   // first 64-element block
    int32_t nkb;   // number of blocks
    int32_t slot;  // partial slot index
    int32_t cta;   // owning CTA
};

// Where the partial Grams of one (module, side) are.
struct SideInfo {
    int32_t first_slot;
    int32_t n_slots;
    int32_t side_off;      // float offset of this side inside a slot (stacked: side * h * h)
    int32_t pitch;         // row pitch of the partial, in floats
    int32_t tensor_core;   // 1: the module's units belong to the tensor-core kernel, which also
                           //    finishes the module; 0: CUDA-core kernel + finalisation kernel
    int32_t module_units;  // work units of the whole module (both sides)
    int32_t n_tasks;       // what the module's finish is cut into: its b rows, or (row, chunk) tasks
    int32_t n_static;      // the first n_static tasks belong to warps named in Plan::first_task; the
                           // module's cursor hands out the rest
};

// What one CTA of the tensor-core kernel reports about a launch: how long it streamed and how
// much.  The host turns the blocks-per-nanosecond of a few launches into the split weights.
struct CtaLog {
    uint32_t serial;       // launch this entry belongs to
    uint32_t duration_ns;  // arrival of the first stage to last MMA issued
    uint32_t blocks;       // 64-element blocks it processed
    uint32_t pad;
};

// End-of-launch help, planned on the host.  The rows of a module are finished by the warps of the
// CTAs that worked on it; a module that got few CTAs (a small one) has many rows per warp, a big
// one less than one.  So some warps of the CTAs of big modules are told to start with a small
// module's rows instead: `warps` of this CTA's epilogue warps (the last ones) first help `module`
// (-1, 0: nobody).
struct CtaHelp {
    int32_t module;
    int32_t warps;
};

// Progress counters of one module inside the tensor-core kernel (zero before a launch).  Each
// is polled or bumped by many CTAs at the end of a launch, so each has a 128-byte line of its own.
struct FinCounters {
    int32_t units_done;  // work units whose partial Gram is complete and visible
    int32_t pad0[31];
    int32_t row_cursor;  // next row of G nobody has claimed yet
    int32_t pad1[31];
    unsigned long long row_acc;  // the rows' terms of the loss so far and how many rows they are (packed:
                                 // one atomic add per warp carries both, see finalize.cuh)
    int32_t pad2[30];
    int32_t row_chunks_done[256];  // two-level finalisation: chunks of each row whose sums are in scratch
};

// Per-module pointers for the CUDA-core kernel.
struct ModulePtrs {
    const void *At;
    const void *Ar;
    int64_t d;
};

struct Plan {
    int mode = 0;
    int n_ctas = 0;
    std::vector<Unit> units;        // tensor-core units first, then CUDA-core units
    int n_units_tc = 0;
    bool all_ctas_busy_tc = false;        // every CTA of the tensor-core kernel has at least one unit
    std::vector<int32_t> cta_begin_tc;    // [n_ctas + 1] into units[0 .. n_units_tc)
    std::vector<int32_t> cta_begin_simt;  // [n_ctas + 1] into units[n_units_tc ..), relative to 0
    std::vector<SideInfo> sides;    // [2 * M]
    std::vector<CtaHelp> cta_help;  // [n_ctas] which module some warps of the CTA lend a hand to first
    // [n_ctas * warps_per_cta] the task an epilogue warp starts the finish with, without asking the
    // module's cursor: (module << 16) | task, or -1
    std::vector<int32_t> first_task;
    // How the finish learns that a partial row has arrived.  false: from the units-done counter of
    // its module, which a unit bumps after a fence.  true: from the row itself -- slots are
    // "empty" (a bit pattern no value has) except between the store and the read of a launch, and
    // the reader fetches until nothing it needs is empty.  That saves the fence, the look at the
    // counter and the claim (2 to 3 us of a 10 to 40 us evaluation); it needs a second set of
    // slots (a launch empties what the launch before wrote), so it is chosen for b <= 128, where
    // the slots are small and the end of a launch is a large part of it, and where every task has
    // a warp of its own from the start and its partial rows fit one pass of the warp's stage.
    bool validate_rows = false;
};

// Bytes of shared memory one epilogue warp stages partial rows in at the end of a launch.
constexpr int kFinStageBytes = 16384;
// Two-level finish of a module evaluated alone (stacked modes).  A (row, chunk) task adds the
// row's partials of `chunk` consecutive slots per side; at most half a stage per side:
inline int chunk_slots_of_mode(int mode) { return kFinStageBytes / (pitch_of_mode(mode) * 4) / 2; }
// How many chunks a row is cut into.  A task costs about a microsecond plus 60 ns per slot, the
// second level 50 ns per chunk: about kTwoLevelChunk slots per chunk, fewer chunks if the tasks
// would outnumber the warps of the grid, more if a chunk would not fit the stage.  1: one level.
constexpr int kTwoLevelChunk = 8;
inline int two_level_chunks(int mode, int most, int b, int total_warps) {
    if (most <= 2 * kTwoLevelChunk) return 1;
    int n = (most + kTwoLevelChunk - 1) / kTwoLevelChunk;
    if (n > total_warps / b) n = total_warps / b;
    const int cap = chunk_slots_of_mode(mode);
    if (n < (most + cap - 1) / cap) n = (most + cap - 1) / cap;
    return n < 1 ? 1 : n;
}
// Slots per side in one chunk when a row with `most` slots on its longer side is cut into n chunks.
__host__ __device__ inline int chunk_slots(int most, int n_chunks) { return (most + n_chunks - 1) / n_chunks; }

inline int64_t kblocks_of(int64_t d) { return (d + kKBlock - 1) / kKBlock; }

// Upper bound on the number of units (hence slots) for any b of one mode: every tile, plus
// one extra unit per CTA boundary in each of the two splits (tensor-core and CUDA-core).
inline int64_t max_units(int M, int mode, int n_ctas) {
    int64_t tiles = mode_is_stacked(mode) ? M : 2 * (int64_t)M;
    return tiles + 2 * (int64_t)n_ctas;
}

namespace detail {
struct Tile {
    int32_t module;
    int32_t side;
    int64_t nkb;
};

// Cut the concatenated block sequence of `tiles` into near-equal contiguous ranges, one per
// CTA; every (tile, range) intersection becomes a unit.  Small problems use fewer CTAs, so
// that a range has at least kMinBlocksPerCta blocks: a shorter range costs the same latency
// and only adds partial slots for the finaliser to read.
constexpr int kMinBlocksPerCta = 8;

// `weights` (optional, [n_ctas], positive): CTA c's range is proportional to weights[c] instead
// of equal -- the caller's estimate of how fast each CTA streams.  Ignored when fewer CTAs than
// n_ctas are used.
inline void split_tiles(const std::vector<Tile> &tiles, int n_ctas, int slot0, std::vector<Unit> &units,
                        std::vector<int32_t> &cta_begin, const float *weights = nullptr) {
    int64_t total = 0;
    for (const Tile &t : tiles) total += t.nkb;
    cta_begin.assign(n_ctas + 1, 0);
    const int base = (int)units.size();
    size_t ti = 0;
    int64_t tile_start = 0;  // global block index of tiles[ti]'s first block
    int64_t used = (total + kMinBlocksPerCta - 1) / kMinBlocksPerCta;
    if (used > n_ctas) used = n_ctas;
    if (used < 1) used = 1;
    // cut[c] .. cut[c + 1]: the blocks of CTA c
    std::vector<int64_t> cut(used + 1);
    bool weighted = (weights != nullptr && used == n_ctas);
    double wsum = 0.0;
    if (weighted)
        for (int c = 0; c < n_ctas; ++c) {
            if (!(weights[c] > 0.f) || weights[c] > 1e30f) weighted = false;  // also rejects NaN
            wsum += weights[c];
        }
    double acc = 0.0;
    for (int64_t c = 0; c <= used; ++c) {
        if (weighted) {
            int64_t v = (c == used) ? total : (int64_t)((double)total * (acc / wsum) + 0.5);
            if (c > 0 && v < cut[c - 1]) v = cut[c - 1];
            if (v > total) v = total;
            cut[c] = v;
            if (c < used) acc += weights[c];
        } else {
            cut[c] = total * c / used;
        }
    }
    for (int c = 0; c < n_ctas; ++c) {
        cta_begin[c] = (int)units.size() - base;
        if (c >= used) continue;  // idle CTA: empty range
        const int64_t lo = cut[c], hi = cut[c + 1];
        int64_t pos = lo;
        while (pos < hi) {
            while (ti < tiles.size() && tile_start + tiles[ti].nkb <= pos) {
                tile_start += tiles[ti].nkb;
                ++ti;
            }
            const Tile &t = tiles[ti];
            const int64_t end = (tile_start + t.nkb < hi) ? tile_start + t.nkb : hi;
            Unit u;
            u.module = t.module;
            u.side = t.side;
            u.kb0 = (int32_t)(pos - tile_start);
            u.nkb = (int32_t)(end - pos);
            u.slot = slot0 + (int)units.size() - base;
            u.cta = c;
            units.push_back(u);
            pos = end;
        }
    }
    cta_begin[n_ctas] = (int)units.size() - base;
}
// Who lends a hand to whom at the end of a launch (CtaHelp).  A CTA's warps are credited to the
// modules it worked on in proportion to its blocks there; a module's need is its b rows at the
// launch's average rows per warp.  CTAs whose main module has more warps than it needs give the
// surplus share of their warps (at most two thirds) to the module that lacks the most at that
// point.  Nothing is planned when no module has more than 1.5 times the average rows per warp.
inline void plan_help(Plan &plan, int M, int b, int warps_per_cta) {
    const int n_ctas = plan.n_ctas;
    plan.cta_help.assign(n_ctas, CtaHelp{-1, 0});
    std::vector<double> have(M, 0.0);
    std::vector<int> main_module(n_ctas, -1);
    for (int c = 0; c < n_ctas; ++c) {
        const int u0 = plan.cta_begin_tc[c], u1 = plan.cta_begin_tc[c + 1];
        int64_t blocks = 0, best = 0;
        for (int u = u0; u < u1; ++u) blocks += plan.units[u].nkb;
        std::vector<int64_t> per;  // blocks per module, in unit order (few entries)
        std::vector<int> mods;
        for (int u = u0; u < u1; ++u) {
            const int m = plan.units[u].module;
            if (mods.empty() || mods.back() != m) {
                mods.push_back(m);
                per.push_back(0);
            }
            per.back() += plan.units[u].nkb;
        }
        for (size_t k = 0; k < mods.size(); ++k) {
            have[mods[k]] += (double)warps_per_cta * (double)per[k] / (double)blocks;
            if (per[k] > best) {
                best = per[k];
                main_module[c] = mods[k];
            }
        }
    }
    double rows = 0.0, warps = 0.0;
    for (int m = 0; m < M; ++m)
        if (have[m] > 0.0) {
            rows += b;
            warps += have[m];
        }
    if (warps <= 0.0) return;
    const double rho = rows / warps;  // rows per warp if every warp took its share
    std::vector<double> lack(M, 0.0);
    bool worth = false;
    for (int m = 0; m < M; ++m) {
        if (have[m] <= 0.0) continue;
        lack[m] = b / rho - have[m];  // warps the module is short of (negative: it has some to spare)
        if (b / have[m] > 1.5 * rho && b / have[m] > 1.5) worth = true;
    }
    if (!worth) return;
    for (int c = 0; c < n_ctas; ++c) {
        const int mm = main_module[c];
        if (mm < 0 || lack[mm] >= 0.0) continue;
        int give = (int)(warps_per_cta * (-lack[mm]) / have[mm]);
        const int cap = 2 * warps_per_cta / 3;
        if (give > cap) give = cap;
        if (give < 1) continue;
        int to = -1;
        for (int m = 0; m < M; ++m)
            if (lack[m] > 0.5 && (to < 0 || lack[m] > lack[to])) to = m;
        if (to < 0) break;
        plan.cta_help[c] = CtaHelp{to, give};
        lack[to] -= give;
    }
}

// The finish of each tensor-core module as tasks, and who starts with which (Plan::first_task).
// A module evaluated alone in a stacked mode and cut into many partials is finished in two
// levels if the caller has scratch for the chunk sums (two_level_chunks): its tasks are (row,
// chunk) pairs, task v = chunk v % n_chunks of row v / n_chunks.  Otherwise a task is a row.
// The warps of a CTA serve the modules it worked on in turn (warp w the (w mod j)-th of its j
// modules), its planned-help warps the module they help; a module's tasks go to its servers one
// each, warp 0 of every CTA first, so that they spread over the SMs.
inline void plan_first_tasks(Plan &plan, int M, int b, int warps_per_cta, bool two_level_ok, bool static_tasks) {
    const int n_ctas = plan.n_ctas;
    plan.first_task.assign((size_t)n_ctas * warps_per_cta, -1);
    int n_active = 0;
    for (int m = 0; m < M; ++m)
        if (plan.sides[2 * (size_t)m].tensor_core && plan.sides[2 * (size_t)m].module_units > 0) ++n_active;
    for (int m = 0; m < M; ++m) {
        SideInfo &t = plan.sides[2 * (size_t)m], &r = plan.sides[2 * (size_t)m + 1];
        int tasks = b;
        const int most = t.n_slots > r.n_slots ? t.n_slots : r.n_slots;
        if (two_level_ok && mode_is_stacked(plan.mode) && n_active == 1 && t.tensor_core)
            tasks = b * two_level_chunks(plan.mode, most, b, n_ctas * warps_per_cta);
        t.n_tasks = r.n_tasks = tasks;
        t.n_static = r.n_static = 0;
    }
    plan.validate_rows = false;
    if (!static_tasks) return;  // every task from the cursor
    std::vector<std::vector<int32_t>> servers(M);
    std::vector<std::vector<int>> mods(n_ctas);
    for (int c = 0; c < n_ctas; ++c)
        for (int u = plan.cta_begin_tc[c]; u < plan.cta_begin_tc[c + 1]; ++u) {
            const int m = plan.units[u].module;
            if (mods[c].empty() || mods[c].back() != m) mods[c].push_back(m);
        }
    for (int w = 0; w < warps_per_cta; ++w)
        for (int c = 0; c < n_ctas; ++c) {
            if (mods[c].empty()) continue;
            const CtaHelp h = plan.cta_help.empty() ? CtaHelp{-1, 0} : plan.cta_help[c];
            const int regular = warps_per_cta - (h.warps > 0 ? h.warps : 0);
            const int m = (w >= regular) ? h.module : mods[c][(size_t)w % mods[c].size()];
            if (m >= 0 && m < M) servers[m].push_back(c * warps_per_cta + w);
        }
    bool one_pass = true, all_static = true;
    for (int m = 0; m < M; ++m) {
        SideInfo &t = plan.sides[2 * (size_t)m], &r = plan.sides[2 * (size_t)m + 1];
        if (!t.tensor_core || t.module_units == 0) continue;
        int n = (int)servers[m].size();
        if (n > t.n_tasks) n = t.n_tasks;
        if (n > 0xffff) n = 0xffff;
        for (int k = 0; k < n; ++k) plan.first_task[servers[m][k]] = (m << 16) | k;
        t.n_static = r.n_static = n;
        if (n < t.n_tasks) all_static = false;
        int rows_per_task = t.n_slots + r.n_slots;  // partial rows a task fetches
        if (t.n_tasks > b) rows_per_task = 2 * chunk_slots(t.n_slots > r.n_slots ? t.n_slots : r.n_slots, t.n_tasks / b);
        if ((int64_t)rows_per_task * pitch_of_mode(plan.mode) * 4 > kFinStageBytes) one_pass = false;
    }
    // (measured slower that way: a row that takes several passes of the stage -- one big module
    // alone at b = 128 -- 23.8 against 20.5 us; more rows than warps -- 27 modules at b = 128 --
    // 40.2 against 38.5 us)
    plan.validate_rows = n_active > 0 && plan.mode <= kSingle1 && one_pass && all_static;
}
}  // namespace detail

// tc_ok[m]: 1 = module m takes the TMA + tcgen05 kernel, 0 = the CUDA-core kernel, 2 = module m
// is not evaluated in this plan (no units, never finished).  weights: see split_tiles (applies
// to the tensor-core split only).
inline void build_plan(int M, const int64_t *d, int b, int n_ctas, const uint8_t *tc_ok, Plan &plan,
                       const float *weights = nullptr, int warps_per_cta = 12, bool two_level_ok = false,
                       bool static_tasks = true) {
    plan.mode = mode_of_b(b);
    plan.n_ctas = n_ctas;
    plan.units.clear();
    plan.sides.assign(2 * (size_t)M, SideInfo{0, 0, 0, 0, 0, 0, 0, 0});
    std::vector<detail::Tile> tc, simt;
    for (int m = 0; m < M; ++m) {
        if (tc_ok[m] == 2) continue;
        std::vector<detail::Tile> &dst = tc_ok[m] ? tc : simt;
        if (mode_is_stacked(plan.mode)) {
            dst.push_back({m, 2, kblocks_of(d[m])});
        } else {
            dst.push_back({m, 0, kblocks_of(d[m])});
            dst.push_back({m, 1, kblocks_of(d[m])});
        }
    }
    detail::split_tiles(tc, n_ctas, 0, plan.units, plan.cta_begin_tc, weights);
    plan.n_units_tc = (int)plan.units.size();
    plan.all_ctas_busy_tc = true;
    for (int c = 0; c < n_ctas; ++c)
        if (plan.cta_begin_tc[c + 1] == plan.cta_begin_tc[c]) plan.all_ctas_busy_tc = false;
    detail::split_tiles(simt, n_ctas, plan.n_units_tc, plan.units, plan.cta_begin_simt);
    const int pitch = pitch_of_mode(plan.mode);
    for (const Unit &u : plan.units) {
        for (int s = 0; s < 2; ++s) {
            if (u.side != 2 && u.side != s) continue;
            SideInfo &si = plan.sides[2 * (size_t)u.module + s];
            if (si.n_slots == 0) si.first_slot = u.slot;
            si.n_slots += 1;
            si.side_off = mode_is_stacked(plan.mode) ? s * pitch * pitch : 0;
            si.pitch = pitch;
        }
    }
    for (int m = 0; m < M; ++m) {
        SideInfo &t = plan.sides[2 * (size_t)m], &r = plan.sides[2 * (size_t)m + 1];
        const int32_t units = mode_is_stacked(plan.mode) ? t.n_slots : t.n_slots + r.n_slots;
        t.tensor_core = r.tensor_core = (tc_ok[m] == 1) ? 1 : 0;
        t.module_units = r.module_units = units;
    }
    detail::plan_help(plan, M, b, warps_per_cta);
    detail::plan_first_tasks(plan, M, b, warps_per_cta, two_level_ok, static_tasks);
}

}  // namespace egeria
