// C ABI of the plasticity-evaluation library: argument checks, workspace layout, the
// static work split, tensor-map encoding and kernel launches.  See include/egeria.h.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

#include <new>
#include <vector>

#include <nvtx3/nvToolsExt.h>  // header-only; a no-op unless a profiler is attached

#include "../../include/egeria.h"
#include "finalize.cuh"
#include "gram_simt.cuh"
#include "gram_tc.cuh"
#include "plan.h"
#include "slope.cuh"

namespace egeria {

constexpr int kMaxCtas = 160;  // sizing bound for the work split (a B200 has 148 SMs)
constexpr int kMaxW = 2048;    // replay keeps 2 * W doubles in shared memory
constexpr int kPlanSlots = 16; // device-side plans kept, keyed by (b, activation pointers)
constexpr int kCalibLaunches = 3;  // launches whose per-CTA streaming rates set the split weights
constexpr size_t kMaxTimedCalls = 4096;  // EGERIA_FLAG_TIME_GRAM: calls timed between two queries
constexpr int kCalibRounds = 3;    // times the weights are (re-)measured; one more round then decides whether they stay
constexpr uint64_t kTestWaitLimitNs = 1000000ull;  // 1 ms: wait limit of a launch under egeria_debug_stall_next

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// A named range around the host side of a call, for timelines (Nsight Systems and the like).
struct HostRange {
    explicit HostRange(const char *name) { nvtxRangePushA(name); }
    ~HostRange() { nvtxRangePop(); }
};

// Host-side check of a work split before it goes to the device: every unit lies inside its tile
// and its slot inside the reserved slots, every CTA's range is a contiguous piece of the unit
// table, every (module, side) has its slots in a row.  A split that fails is never uploaded.
static bool plan_is_sane(const Plan &P, int M, const int64_t *d, int n_ctas, int64_t slot_cap) {
    const int n_tc = P.n_units_tc, n_all = (int)P.units.size();
    if (n_tc < 0 || n_tc > n_all) return false;
    if ((int)P.cta_begin_tc.size() != n_ctas + 1 || (int)P.cta_begin_simt.size() != n_ctas + 1) return false;
    if (P.cta_begin_tc[0] != 0 || P.cta_begin_tc[n_ctas] != n_tc) return false;
    if (P.cta_begin_simt[0] != 0 || P.cta_begin_simt[n_ctas] != n_all - n_tc) return false;
    for (int c = 0; c < n_ctas; ++c)
        if (P.cta_begin_tc[c] > P.cta_begin_tc[c + 1] || P.cta_begin_simt[c] > P.cta_begin_simt[c + 1]) return false;
    for (const Unit &u : P.units) {
        if (u.module < 0 || u.module >= M || u.side < 0 || u.side > 2) return false;
        if (u.kb0 < 0 || u.nkb < 1 || (int64_t)u.kb0 + u.nkb > kblocks_of(d[u.module])) return false;
        if (u.slot < 0 || u.slot >= slot_cap || u.cta < 0 || u.cta >= n_ctas) return false;
    }
    if ((int)P.sides.size() != 2 * M) return false;
    for (const SideInfo &si : P.sides)
        if (si.n_slots < 0 || si.first_slot < 0 || (int64_t)si.first_slot + si.n_slots > slot_cap) return false;
    return true;
}

// Offsets of everything the library keeps in the caller's workspace.
struct Layout {
    size_t status, cta_log, rowloss, tickets, fin_ctr, T, losses, keep, chunk, slots, staging, total;
    // the freezing-rule state, one contiguous region [rule0, rule_end) (what export / import copy)
    size_t rule0, raw, plist, n_evals, counter, freeze_eval, last_slope, Tauto, smax, front, unfreeze, boot_raw,
        boot_plist, boot_ints, rule_end;
    size_t replay_raw, replay_plist;  // windows of egeria_plasticity_replay_lr ([M][W] doubles each)
    size_t chunk_bytes;     // bytes of the chunk-sum scratch
    size_t slot_bytes_cap;  // bytes reserved for partial slots
    size_t slot_set_bytes;  // launches that validate partial rows by their contents (b <= 128) alternate
                            // between the sets [0, slot_set_bytes) and [slot_set_bytes, 2 slot_set_bytes)
    // Device-side plans (tensor maps, pointers, unit table, per-CTA ranges, slot ranges): kPlanSlots
    // regions of plan_stride bytes from plan0; the offsets below are relative to a region.
    size_t plan0, plan_stride;
    size_t tmaps, modules, units, cta_begin_tc, cta_begin_simt, sides, cta_help, first_task;
    size_t first_task_bytes;
};

// Units of one device-side plan: all modules in one split, or (front-only contexts) one split per
// possible front, each over a single module.
static int64_t units_cap(int M, int b_max, uint32_t flags) {
    int64_t cap = 0;
    for (int mode = 0; mode <= mode_of_b(b_max); ++mode) {
        int64_t u = max_units(M, mode, kMaxCtas);
        if (flags & EGERIA_FLAG_FRONT_ONLY) {
            const int64_t f = (int64_t)M * max_units(1, mode, kMaxCtas);
            if (f > u) u = f;
        }
        if (u > cap) cap = u;
    }
    return cap;
}

static bool make_layout(int M, const int64_t *d, int b_max, int W, uint32_t flags, Layout &L) {
    size_t off = 0;
    auto take = [&](size_t bytes) {
        const size_t o = off;
        off = align_up(off + bytes, 256);
        return o;
    };
    L.status = take(256);
    L.cta_log = take(kMaxCtas * sizeof(CtaLog));
    {
        size_t saved = off;
        off = 0;
        L.tmaps = take((size_t)2 * M * sizeof(CUtensorMap));
        L.modules = take((size_t)M * sizeof(ModulePtrs));
        L.units = take((size_t)units_cap(M, b_max, flags) * sizeof(Unit));
        L.cta_begin_tc = take((size_t)((flags & EGERIA_FLAG_FRONT_ONLY) ? M : 1) * (kMaxCtas + 1) * sizeof(int32_t));
        L.cta_begin_simt = take((kMaxCtas + 1) * sizeof(int32_t));
        L.sides = take((size_t)2 * M * sizeof(SideInfo));
        L.cta_help = take((size_t)kMaxCtas * sizeof(CtaHelp));
        L.first_task_bytes = (size_t)((flags & EGERIA_FLAG_FRONT_ONLY) ? M : 1) * kMaxCtas * kEpiWarps * sizeof(int32_t);
        L.first_task = take(L.first_task_bytes);
        L.plan_stride = off;
        off = saved;
        L.plan0 = take(L.plan_stride * kPlanSlots);
    }
    L.rowloss = take((size_t)M * kMaxB * sizeof(double));
    L.tickets = take((size_t)M * sizeof(int32_t));
    L.fin_ctr = take((size_t)2 * M * sizeof(FinCounters));  // two sets, used by alternate launches
    L.T = take((size_t)M * sizeof(float));
    L.rule0 = off;
    L.raw = take((size_t)M * W * sizeof(double));
    L.plist = take((size_t)M * W * sizeof(double));
    L.n_evals = take((size_t)M * sizeof(int32_t));
    L.counter = take((size_t)M * sizeof(int32_t));
    L.freeze_eval = take((size_t)M * sizeof(int32_t));
    L.last_slope = take((size_t)M * sizeof(double));
    L.Tauto = take((size_t)M * sizeof(double));
    L.smax = take((size_t)M * sizeof(double));
    L.front = take(sizeof(unsigned long long));
    L.unfreeze = take(32);  // reference learning rate (8 bytes), window in force, restarts
    L.boot_raw = take((size_t)W * sizeof(double));
    L.boot_plist = take((size_t)W * sizeof(double));
    L.boot_ints = take(2 * sizeof(int32_t));
    L.rule_end = off;
    L.replay_raw = take((size_t)M * W * sizeof(double));
    L.replay_plist = take((size_t)M * W * sizeof(double));
    L.losses = take((size_t)M * sizeof(float));
    L.keep = off;
    if (flags & EGERIA_FLAG_KEEP_GRAMS) take((size_t)M * 2 * b_max * b_max * sizeof(float));
    {
        // scratch of the two-level finalisation (one module evaluated alone): rows x chunks x both
        // sides x columns, float64; a chunk has at least one slot per side, and two_level_chunks aims
        // at kTwoLevelChunk of them
        size_t bytes = 0;
        for (int mode = 0; mode <= mode_of_b(b_max) && mode <= kStacked64; ++mode) {  // used at b <= 64 only
            const int nc = pitch_of_mode(mode) / 32;
            const size_t chunks = (size_t)(max_units(1, mode, kMaxCtas) + kTwoLevelChunk - 1) / kTwoLevelChunk + 1;
            const size_t rows = (size_t)(pitch_of_mode(mode) < b_max ? pitch_of_mode(mode) : b_max);
            const size_t v = rows * chunks * 2 * 32 * nc * sizeof(double);
            if (v > bytes) bytes = v;
        }
        L.chunk_bytes = bytes;
        L.chunk = take(bytes);
    }
    size_t slot_bytes = 0, set_bytes = 0;
    for (int mode = 0; mode <= mode_of_b(b_max); ++mode) {
        const size_t s = (size_t)max_units(M, mode, kMaxCtas) * slot_floats_of_mode(mode) * sizeof(float);
        if (s > slot_bytes) slot_bytes = s;
        if (mode <= kSingle1 && s > set_bytes) set_bytes = s;
    }
    set_bytes = align_up(set_bytes, 256);
    if (2 * set_bytes > slot_bytes) slot_bytes = 2 * set_bytes;
    L.slot_set_bytes = set_bytes;
    L.slot_bytes_cap = slot_bytes;
    L.slots = take(slot_bytes);
    L.staging = off;
    if (flags & EGERIA_FLAG_HOST_STAGING) {
        for (int m = 0; m < M; ++m) {
            take((size_t)b_max * d[m] * 2);
            take((size_t)b_max * d[m] * 2);
        }
    }
    L.total = align_up(off, EGERIA_WORKSPACE_ALIGN);
    return true;
}

static egeria_status check_shapes(int M, const int64_t *d, int b_max, int W) {
    if (M < 1 || !d || W < 1 || W > kMaxW) return EGERIA_ERR_INVALID_ARG;
    if (b_max < 2) return EGERIA_ERR_INVALID_ARG;
    if (b_max > EGERIA_MAX_B) return EGERIA_ERR_UNSUPPORTED_SHAPE;
    for (int m = 0; m < M; ++m) {
        if (d[m] < 1) return EGERIA_ERR_UNSUPPORTED_SHAPE;
        // TMA coordinates are 32-bit element indices
        if (d[m] > (int64_t)0x7fffffff - 2 * kKBlock) return EGERIA_ERR_UNSUPPORTED_SHAPE;
    }
    return EGERIA_OK;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

typedef CUresult (*ReplaceAddressFn)(CUtensorMap *, void *);

// A work split as built for one (b, kind of evaluation, split weights, which modules take which
// kernel): it does not depend on where the activations are, so a caller whose buffers move from
// call to call gets it from here instead of having it rebuilt.
struct BuiltPlan {
    int b = -1;
    bool front_only = false;
    int weights_version = -1;
    std::vector<uint8_t> tc_ok;
    Plan plan;
    std::vector<int32_t> front_cta_begin;
    std::vector<int32_t> front_first_task;  // [M][kMaxCtas * kEpiWarps]
    int slot_units = 0;  // partial slots a launch of this plan may write (front-only: of the largest front)
    uint64_t last_use = 0;
};
constexpr int kBuiltPlans = 4;

}  // namespace egeria

using namespace egeria;

struct egeria_ctx {
    int M = 0, b_max = 0, W_cap = 0;  // W_cap: the window given at creation (the one in force is on the device)
    double lr = NAN;        // learning rate in force (egeria_plasticity_set_lr); NaN: never given
    double lr_checked = NAN;  // rate of the last evaluation of the rule (the unfreezing test runs when it changes)
    uint32_t flags = 0;
    std::vector<int64_t> d;
    uint8_t *ws = nullptr;
    size_t ws_bytes = 0;
    Layout L{};
    int n_ctas = 0;
    EncodeTiledFn encode = nullptr;
    ReplaceAddressFn replace_address = nullptr;  // may be missing: then every map is encoded afresh
    bool attrs_set = false;
    BuiltPlan built[kBuiltPlans];
    // Tensor maps of every (module, side) for tmpl_b rows, encoded once; a new pointer set copies
    // them and only swaps the address in.
    std::vector<CUtensorMap> tmpl;
    std::vector<uint8_t> tmpl_valid;
    int tmpl_b = -1;
    // device-side plans, least recently used one is replaced
    struct PlanEntry {
        int b = -1;
        bool front_only = false;  // one split per possible front (plan.units is their concatenation)
        int weights_version = 0;
        std::vector<const void *> At, Ar;
        Plan plan;
        int slot_units = 0;  // partial slots a launch of this plan may write
        uint64_t last_use = 0;
    };
    PlanEntry plans[kPlanSlots];
    int cur = 0;           // entry the last egeria_sp_loss_batch used
    int plan_b = -1;       // its b
    uint64_t use_clock = 0;
    std::vector<uint8_t> pack;  // host image of one plan region (when there is no pinned one)
    uint8_t *pinned_plans = nullptr;  // kPlanSlots images of plan_stride bytes: uploads that do not stall the stream
    cudaEvent_t plan_uploaded[kPlanSlots] = {};  // recorded after the upload from image i: the image is free again
    bool plan_upload_pending[kPlanSlots] = {};   // once the event has completed
    uint8_t *plan_region(int i) const { return ws + L.plan0 + (size_t)i * L.plan_stride; }
    cudaStream_t last_stream = nullptr;
    int64_t launches = 0;
    uint32_t tc_launches = 0;  // selects the set of progress counters the next tensor-core launch uses
    uint32_t rule_evals = 0;   // evaluations of the freezing rule enqueued so far (the serial of the last one)
    bool slots_dirty = false;  // a launch that does not validate rows has left its partials in the slots
    int val_set = 0;           // set of slots the next launch that validates rows uses
    size_t set_dirty[2] = {0, 0};  // bytes from the start of each set that a launch wrote and nobody has emptied
    uint32_t stall_next = 0;   // test hook: give-up path of the next tensor-core launch (egeria_debug_stall_next)
    // Split weights: one per CTA, from the streaming rates the CTAs report (SMs do not all get
    // the same share of HBM bandwidth; the CTA -> SM placement repeats from launch to launch).
    std::vector<float> weights;
    std::vector<double> rate_sum;  // blocks per nanosecond of every CTA, summed over the later rounds
    double makespan_equal = 0.0;   // longest streaming time of a CTA under the equal split (mean of the round's launches)
    int weights_version = 0;
    bool calibrated = false;   // no more measuring
    int calib_round = 0;
    int calib_enqueued = 0;
    uint32_t calib_serial[kCalibLaunches] = {};
    CtaLog *host_log = nullptr;  // pinned, kCalibLaunches x kMaxCtas
    std::vector<void *> staging_t, staging_r;
    std::vector<const void *> subset_t, subset_r;  // pointer arrays of a subset call (left-out modules nulled)
    // EGERIA_FLAG_TIME_GRAM: event pairs around the Gram kernel launches since the last query
    std::vector<cudaEvent_t> ev_pool;
    size_t ev_used = 0;

    template <class T>
    T *at(size_t off) const {
        return reinterpret_cast<T *>(ws + off);
    }
    int rule_flags() const {
        return ((flags & EGERIA_FLAG_SIGNED_SLOPE) ? kRuleSigned : 0) | ((flags & EGERIA_FLAG_AUTO_T) ? kRuleAutoT : 0) |
               ((flags & EGERIA_FLAG_FRONTMOST) ? kRuleFrontmost : 0);
    }
    BootState boot_state() const {
        BootState bs;
        bs.raw = at<double>(L.boot_raw);
        bs.plist = at<double>(L.boot_plist);
        bs.n_evals = at<int32_t>(L.boot_ints);
        bs.end = at<int32_t>(L.boot_ints) + 1;
        return bs;
    }
    SlopeState slope_state() const {
        SlopeState st;
        st.raw = at<double>(L.raw);
        st.plist = at<double>(L.plist);
        st.n_evals = at<int32_t>(L.n_evals);
        st.counter = at<int32_t>(L.counter);
        st.freeze_eval = at<int32_t>(L.freeze_eval);
        st.last_slope = at<double>(L.last_slope);
        st.Tauto = at<double>(L.Tauto);
        st.smax = at<double>(L.smax);
        st.front = at<unsigned long long>(L.front);
        st.T = at<float>(L.T);
        st.W_cap = W_cap;
        st.lr_ref = at<unsigned long long>(L.unfreeze);
        st.W_cur = at<int32_t>(L.unfreeze + 8);
        st.restarts = at<int32_t>(L.unfreeze + 12);
        return st;
    }
};

namespace egeria {
static void poll_calibration(egeria_ctx *ctx);
}

#define EG_CUDA(call)                                   \
    do {                                                \
        cudaError_t e_ = (call);                        \
        if (e_ != cudaSuccess) return EGERIA_ERR_CUDA;  \
    } while (0)

extern "C" {

const char *egeria_status_string(egeria_status s) {
    switch (s) {
        case EGERIA_OK: return "ok";
        case EGERIA_ERR_INVALID_ARG: return "invalid argument";
        case EGERIA_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case EGERIA_ERR_UNSUPPORTED_DEVICE: return "unsupported device (needs compute capability 10.x)";
        case EGERIA_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case EGERIA_ERR_CUDA: return "CUDA call failed";
        case EGERIA_ERR_TIMEOUT: return "bounded device-side wait ran out";
        case EGERIA_ERR_CHECK: return "index check inside a kernel failed (checked build)";
    }
    return "unknown status";
}

size_t egeria_workspace_bytes(int M, const int64_t *d, int b_max, int W, uint32_t flags) {
    if (check_shapes(M, d, b_max, W) != EGERIA_OK) return 0;
    Layout L;
    make_layout(M, d, b_max, W, flags, L);
    return L.total;
}

egeria_status egeria_debug_plan(int M, const int64_t *d, int b, int n_ctas, int32_t *out_units, int max_units_out,
                                int *n_units) {
    return egeria_debug_plan_weighted(M, d, b, n_ctas, nullptr, out_units, max_units_out, n_units);
}

egeria_status egeria_debug_plan_weighted(int M, const int64_t *d, int b, int n_ctas, const float *weights,
                                         int32_t *out_units, int max_units_out, int *n_units) {
    if (!out_units || !n_units || n_ctas < 1 || max_units_out < 0) return EGERIA_ERR_INVALID_ARG;
    egeria_status s = check_shapes(M, d, b, 1);
    if (s != EGERIA_OK) return s;
    std::vector<uint8_t> tc_ok(M);
    for (int m = 0; m < M; ++m) tc_ok[m] = (d[m] % 8 == 0);
    Plan plan;
    build_plan(M, d, b, n_ctas, tc_ok.data(), plan, weights);
    *n_units = (int)plan.units.size();
    for (int i = 0; i < (int)plan.units.size() && i < max_units_out; ++i) {
        const Unit &u = plan.units[i];
        int32_t *row = out_units + 5 * i;
        row[0] = u.module;
        row[1] = u.side;
        row[2] = u.kb0;
        row[3] = u.nkb;
        row[4] = u.cta;
    }
    return EGERIA_OK;
}

egeria_status egeria_debug_plan_help(int M, const int64_t *d, int b, int n_ctas, int32_t *out_help) {
    if (!out_help || n_ctas < 1) return EGERIA_ERR_INVALID_ARG;
    egeria_status s = check_shapes(M, d, b, 1);
    if (s != EGERIA_OK) return s;
    std::vector<uint8_t> tc_ok(M);
    for (int m = 0; m < M; ++m) tc_ok[m] = (d[m] % 8 == 0);
    Plan plan;
    build_plan(M, d, b, n_ctas, tc_ok.data(), plan, nullptr);
    for (int c = 0; c < n_ctas; ++c) {
        out_help[2 * c] = plan.cta_help[c].module;
        out_help[2 * c + 1] = plan.cta_help[c].warps;
    }
    return EGERIA_OK;
}

egeria_status egeria_debug_plan_tasks(int M, const int64_t *d, int b, int n_ctas, int only_module, int32_t *out_first,
                                      int32_t *out_tasks, int *out_validate) {
    if (!out_first || !out_tasks || !out_validate || n_ctas < 1 || only_module >= M) return EGERIA_ERR_INVALID_ARG;
    egeria_status s = check_shapes(M, d, b, 1);
    if (s != EGERIA_OK) return s;
    std::vector<uint8_t> tc_ok(M);
    for (int m = 0; m < M; ++m) tc_ok[m] = (only_module >= 0 && m != only_module) ? 2 : (d[m] % 8 == 0);
    Plan plan;
    build_plan(M, d, b, n_ctas, tc_ok.data(), plan, nullptr, kEpiWarps, true);
    memcpy(out_first, plan.first_task.data(), plan.first_task.size() * sizeof(int32_t));
    for (int m = 0; m < M; ++m) {
        out_tasks[2 * m] = plan.sides[2 * (size_t)m].n_tasks;
        out_tasks[2 * m + 1] = plan.sides[2 * (size_t)m].n_static;
    }
    *out_validate = plan.validate_rows ? 1 : 0;
    return EGERIA_OK;
}

egeria_status egeria_plasticity_create(egeria_ctx **out, int M, const int64_t *d, int b_max, int W, const float *T,
                                       float T_all, void *workspace, size_t workspace_bytes, uint32_t flags) {
    if (!out) return EGERIA_ERR_INVALID_ARG;
    *out = nullptr;
    egeria_status s = check_shapes(M, d, b_max, W);
    if (s != EGERIA_OK) return s;
    if ((flags & EGERIA_FLAG_FRONT_ONLY) && !(flags & EGERIA_FLAG_FRONTMOST)) return EGERIA_ERR_INVALID_ARG;
    Layout L;
    make_layout(M, d, b_max, W, flags, L);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) % EGERIA_WORKSPACE_ALIGN) != 0 ||
        workspace_bytes < L.total)
        return EGERIA_ERR_WORKSPACE;

    int dev = 0;
    cudaDeviceProp prop;
    EG_CUDA(cudaGetDevice(&dev));
    EG_CUDA(cudaGetDeviceProperties(&prop, dev));
    if (prop.major != 10) return EGERIA_ERR_UNSUPPORTED_DEVICE;

    egeria_ctx *ctx = new (std::nothrow) egeria_ctx();
    if (!ctx) return EGERIA_ERR_INVALID_ARG;
    ctx->M = M;
    ctx->b_max = b_max;
    ctx->W_cap = W;
    ctx->flags = flags;
    ctx->d.assign(d, d + M);
    ctx->ws = static_cast<uint8_t *>(workspace);
    ctx->ws_bytes = workspace_bytes;
    ctx->L = L;
    ctx->n_ctas = prop.multiProcessorCount < kMaxCtas ? prop.multiProcessorCount : kMaxCtas;

    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !fn) {
        delete ctx;
        return EGERIA_ERR_CUDA;
    }
    ctx->encode = reinterpret_cast<EncodeTiledFn>(fn);
    fn = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapReplaceAddress", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess && fn)
        ctx->replace_address = reinterpret_cast<ReplaceAddressFn>(fn);
    else
        (void)cudaGetLastError();

    if (flags & EGERIA_FLAG_HOST_STAGING) {
        size_t off = L.staging;  // same walk as make_layout
        for (int m = 0; m < M; ++m) {
            ctx->staging_t.push_back(ctx->ws + off);
            off = align_up(off + (size_t)b_max * d[m] * 2, 256);
            ctx->staging_r.push_back(ctx->ws + off);
            off = align_up(off + (size_t)b_max * d[m] * 2, 256);
        }
    }

    std::vector<float> Th(M);
    for (int m = 0; m < M; ++m) Th[m] = T ? T[m] : T_all;
    ctx->weights.assign(ctx->n_ctas, 1.0f);
    {
        void *hp = nullptr;
        bool ok = (cudaHostAlloc(&hp, L.plan_stride * kPlanSlots, cudaHostAllocDefault) == cudaSuccess);
        for (int i = 0; ok && i < kPlanSlots; ++i)
            ok = (cudaEventCreateWithFlags(&ctx->plan_uploaded[i], cudaEventDisableTiming) == cudaSuccess);
        if (ok) {
            ctx->pinned_plans = static_cast<uint8_t *>(hp);
        } else {
            (void)cudaGetLastError();  // fall back to pageable staging
            if (hp) cudaFreeHost(hp);
        }
    }
    if (!(flags & EGERIA_FLAG_EQUAL_SPLIT)) {
        void *hp = nullptr;
        if (cudaHostAlloc(&hp, sizeof(CtaLog) * kCalibLaunches * kMaxCtas, cudaHostAllocDefault) == cudaSuccess) {
            memset(hp, 0, sizeof(CtaLog) * kCalibLaunches * kMaxCtas);
            ctx->host_log = static_cast<CtaLog *>(hp);
        } else {
            (void)cudaGetLastError();  // no pinned memory: keep the equal split
        }
    }
    cudaError_t e = cudaMemset(ctx->ws + L.status, 0, 256);
    if (e == cudaSuccess) e = cudaMemset(ctx->ws + L.cta_log, 0, kMaxCtas * sizeof(CtaLog));
    if (e == cudaSuccess) e = cudaMemset(ctx->ws + L.tickets, 0, (size_t)M * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemset(ctx->ws + L.fin_ctr, 0, (size_t)2 * M * sizeof(FinCounters));
    if (e == cudaSuccess) e = cudaMemset(ctx->ws + L.slots, 0xff, L.slot_bytes_cap);  // every partial slot empty (kSlotEmpty)
    if (e == cudaSuccess) e = cudaMemcpy(ctx->ws + L.T, Th.data(), (size_t)M * sizeof(float), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) {
        plasticity_clear_kernel<<<(M + 127) / 128, 128>>>(ctx->slope_state(), M, W, 0);
        bootstrap_clear_kernel<<<1, 1>>>(ctx->boot_state());
        ctx->launches += 2;
        e = cudaDeviceSynchronize();
    }
    if (e != cudaSuccess) {
        egeria_plasticity_destroy(ctx);
        return EGERIA_ERR_CUDA;
    }
    *out = ctx;
    return EGERIA_OK;
}

egeria_status egeria_plasticity_destroy(egeria_ctx *ctx) {
    if (!ctx) return EGERIA_ERR_INVALID_ARG;
    for (cudaEvent_t e : ctx->ev_pool) cudaEventDestroy(e);
    for (cudaEvent_t e : ctx->plan_uploaded)
        if (e) cudaEventDestroy(e);
    if (ctx->host_log) cudaFreeHost(ctx->host_log);
    if (ctx->pinned_plans) cudaFreeHost(ctx->pinned_plans);
    delete ctx;
    return EGERIA_OK;
}

// The window in force and the number of restarts live on the device (the device halves the one
// and counts the other): wait for the stream and read them.
static int read_unfreeze_word(const egeria_ctx *ctx, size_t byte_off) {
    if (!ctx) return 0;
    if (cudaStreamSynchronize(ctx->last_stream) != cudaSuccess) return -1;
    int32_t v = 0;
    if (cudaMemcpy(&v, ctx->ws + ctx->L.unfreeze + byte_off, sizeof(v), cudaMemcpyDeviceToHost) != cudaSuccess)
        return -1;
    return v;
}
int egeria_plasticity_window(const egeria_ctx *ctx) { return read_unfreeze_word(ctx, 8); }
int egeria_plasticity_restarts(const egeria_ctx *ctx) { return read_unfreeze_word(ctx, 12); }

egeria_status egeria_plasticity_set_lr(egeria_ctx *ctx, double lr) {
    if (!ctx) return EGERIA_ERR_INVALID_ARG;
    ctx->lr = lr;
    return EGERIA_OK;
}

int egeria_split_weights(egeria_ctx *ctx, float *out_weights, int max_weights) {
    if (!ctx) return -1;
    poll_calibration(ctx);
    if (out_weights)
        for (int c = 0; c < ctx->n_ctas && c < max_weights; ++c) out_weights[c] = ctx->weights[c];
    return (ctx->weights_version > 0) ? ctx->n_ctas : 0;
}
int64_t egeria_launch_count(const egeria_ctx *ctx) { return ctx ? ctx->launches : 0; }

}  // extern "C"

namespace egeria {

static egeria_status encode_map(egeria_ctx *ctx, CUtensorMap *tm, const void *base, int b, int64_t d, int box_rows) {
    cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)b};
    cuuint64_t strides[1] = {(cuuint64_t)d * 2};
    cuuint32_t box[2] = {(cuuint32_t)kKBlock, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = ctx->encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box,
                             estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? EGERIA_OK : EGERIA_ERR_CUDA;
}

// If the logs of all calibration launches have arrived on the host, turn them into split
// weights: CTA c gets work in proportion to the blocks per nanosecond it managed.  Never waits.
static void poll_calibration(egeria_ctx *ctx) {
    if (ctx->calibrated || !ctx->host_log || ctx->calib_enqueued < kCalibLaunches) return;
    const int n = ctx->n_ctas;
    std::vector<double> rate(n, 0.0);
    double makespan = 0.0;  // the slowest CTA's streaming time, mean over the round's launches
    for (int k = 0; k < kCalibLaunches; ++k) {
        const volatile CtaLog *log = ctx->host_log + (size_t)k * kMaxCtas;
        uint32_t longest = 0;
        for (int c = 0; c < n; ++c) {
            if (log[c].serial != ctx->calib_serial[k]) return;  // this copy has not landed yet
            const uint32_t ns = log[c].duration_ns, blocks = log[c].blocks;
            if (ns == 0 || blocks == 0) {  // a launch that gave up: stay with the equal split
                ctx->calibrated = true;
                return;
            }
            rate[c] += (double)blocks / (double)ns;
            if (ns > longest) longest = ns;
        }
        makespan += (double)longest / kCalibLaunches;
    }
    if (ctx->calib_round == 0) ctx->makespan_equal = makespan;
    if (ctx->calib_round >= kCalibRounds) {
        // The decision: this round of launches ran under the final shares.  They stay only if the slowest CTA
        // now finishes at least 1 % earlier than under the equal split; on a GPU whose SMs stream
        // alike the measured rates are noise, and shares that follow noise lose to equal ones.
        if (!(makespan < 0.99 * ctx->makespan_equal)) {
            for (int c = 0; c < n; ++c) ctx->weights[c] = 1.0f;
            ctx->weights_version++;
        }
        ctx->calibrated = true;
        return;
    }
    // From the second round on the rates were measured under shares close to the final ones: keep
    // adding them up, so that the last word is an average over six launches, not three.
    if (ctx->calib_round >= 1) {
        if (ctx->rate_sum.size() != (size_t)n) ctx->rate_sum.assign(n, 0.0);
        for (int c = 0; c < n; ++c) rate[c] = (ctx->rate_sum[c] += rate[c]);
    }
    double mean = 0.0;
    for (int c = 0; c < n; ++c) mean += rate[c];
    mean /= n;
    for (int c = 0; c < n; ++c) {
        double w = rate[c] / mean;
        if (w < 0.5) w = 0.5;
        if (w > 2.0) w = 2.0;
        ctx->weights[c] = (float)w;
    }
    ctx->weights_version++;  // plans made with the previous shares are rebuilt on their next use
    // Under the equal split the fast CTAs finish early and leave the slow ones more bandwidth, which
    // flatters the slow ones: measure again under the new shares, a few times.
    ctx->calib_round++;
    ctx->calib_enqueued = 0;  // (after kCalibRounds rounds: one more, for the decision above)
}

// The work split for b rows: all evaluated modules in one split, or (front-only) one split per
// possible front, each with module f alone over all CTAs, their units concatenated (slots are
// numbered from 0 in each: only one of them runs in a launch).
static egeria_status build_split(egeria_ctx *ctx, int b, bool front_only, const std::vector<uint8_t> &tc_ok,
                                 const float *weights, BuiltPlan &out) {
    const int M = ctx->M;
    out.front_cta_begin.clear();
    out.front_first_task.clear();
    if (!front_only) {
        build_plan(M, ctx->d.data(), b, ctx->n_ctas, tc_ok.data(), out.plan, weights, kEpiWarps, true);
        out.slot_units = (int)out.plan.units.size();
        const int64_t slot_cap = (int64_t)(ctx->L.slot_bytes_cap / (slot_floats_of_mode(out.plan.mode) * sizeof(float)));
        return plan_is_sane(out.plan, M, ctx->d.data(), ctx->n_ctas, slot_cap) ? EGERIA_OK : EGERIA_ERR_WORKSPACE;
    }
    for (int m = 0; m < M; ++m)
        if (tc_ok[m] != 1) return EGERIA_ERR_UNSUPPORTED_SHAPE;
    Plan &all = out.plan;
    all = Plan{};
    all.mode = mode_of_b(b);
    all.n_ctas = ctx->n_ctas;
    all.sides.assign(2 * (size_t)M, SideInfo{0, 0, 0, 0, 0, 0, 0, 0});
    all.all_ctas_busy_tc = true;
    out.front_cta_begin.assign((size_t)M * (kMaxCtas + 1), 0);
    out.front_first_task.assign((size_t)M * kMaxCtas * kEpiWarps, -1);
    all.validate_rows = true;  // (one protocol for whichever front the device picks)
    out.slot_units = 0;
    std::vector<uint8_t> only(M);
    Plan one;
    for (int f = 0; f < M; ++f) {
        for (int m = 0; m < M; ++m) only[m] = (m == f) ? 1 : 2;
        build_plan(M, ctx->d.data(), b, ctx->n_ctas, only.data(), one, weights, kEpiWarps, true);
        memcpy(&out.front_first_task[(size_t)f * kMaxCtas * kEpiWarps], one.first_task.data(),
               one.first_task.size() * sizeof(int32_t));
        if (!plan_is_sane(one, M, ctx->d.data(), ctx->n_ctas,
                          (int64_t)(ctx->L.slot_bytes_cap / (slot_floats_of_mode(one.mode) * sizeof(float)))))
            return EGERIA_ERR_WORKSPACE;
        const int32_t base = (int32_t)all.units.size();
        all.units.insert(all.units.end(), one.units.begin(), one.units.end());
        for (int c = 0; c <= ctx->n_ctas; ++c)
            out.front_cta_begin[(size_t)f * (kMaxCtas + 1) + c] = base + one.cta_begin_tc[c];
        all.sides[2 * (size_t)f] = one.sides[2 * (size_t)f];
        all.sides[2 * (size_t)f + 1] = one.sides[2 * (size_t)f + 1];
        all.all_ctas_busy_tc = all.all_ctas_busy_tc && one.all_ctas_busy_tc;
        all.validate_rows = all.validate_rows && one.validate_rows;
        if ((int)one.units.size() > out.slot_units) out.slot_units = (int)one.units.size();
        if ((size_t)one.units.size() * slot_floats_of_mode(one.mode) * sizeof(float) > ctx->L.slot_bytes_cap)
            return EGERIA_ERR_WORKSPACE;
    }
    all.n_units_tc = (int)all.units.size();
    all.cta_begin_tc.assign(ctx->n_ctas + 1, 0);
    all.cta_begin_simt.assign(ctx->n_ctas + 1, 0);
    return EGERIA_OK;
}

// Select (or build and upload) the device-side plan for this (b, pointers).
static egeria_status refresh_plan(egeria_ctx *ctx, cudaStream_t stream, const void *const *At, const void *const *Ar,
                                  int b, bool front_only) {
    const int M = ctx->M;
    const size_t pbytes = (size_t)M * sizeof(void *);
    int lru = 0;
    for (int i = 0; i < kPlanSlots; ++i) {
        egeria_ctx::PlanEntry &e = ctx->plans[i];
        if (e.b == b && e.front_only == front_only && e.weights_version == ctx->weights_version &&
            memcmp(e.At.data(), At, pbytes) == 0 &&
            memcmp(e.Ar.data(), Ar, pbytes) == 0) {
            e.last_use = ++ctx->use_clock;
            ctx->cur = i;
            ctx->plan_b = b;
            return EGERIA_OK;
        }
        if (e.last_use < ctx->plans[lru].last_use) lru = i;
    }
    egeria_ctx::PlanEntry &e = ctx->plans[lru];
    e.b = -1;  // invalid until the upload below has been enqueued

    std::vector<uint8_t> tc_ok(M);
    for (int m = 0; m < M; ++m) {
        if (!At[m]) {  // not evaluated in this call (subset entry points)
            tc_ok[m] = 2;
            continue;
        }
        const bool aligned = (reinterpret_cast<uintptr_t>(At[m]) % 16 == 0) &&
                             (reinterpret_cast<uintptr_t>(Ar[m]) % 16 == 0) && (ctx->d[m] % 8 == 0);
        tc_ok[m] = (aligned && !(ctx->flags & EGERIA_FLAG_FORCE_SIMT)) ? 1 : 0;
    }
    const float *weights = ctx->weights_version > 0 ? ctx->weights.data() : nullptr;
    BuiltPlan *bp = nullptr;
    {
        int oldest = 0;
        for (int i = 0; i < kBuiltPlans; ++i) {
            BuiltPlan &c = ctx->built[i];
            if (c.b == b && c.front_only == front_only && c.weights_version == ctx->weights_version && c.tc_ok == tc_ok) {
                bp = &c;
                break;
            }
            if (c.last_use < ctx->built[oldest].last_use) oldest = i;
        }
        if (!bp) {
            bp = &ctx->built[oldest];
            bp->b = -1;
            egeria_status bs = build_split(ctx, b, front_only, tc_ok, weights, *bp);
            if (bs != EGERIA_OK) return bs;
            bp->b = b;
            bp->front_only = front_only;
            bp->weights_version = ctx->weights_version;
            bp->tc_ok = tc_ok;
        }
        bp->last_use = ++ctx->use_clock;
    }
    e.plan = bp->plan;
    e.slot_units = bp->slot_units;
    const std::vector<int32_t> &front_cta_begin = bp->front_cta_begin;
    const Plan &P = e.plan;
    const Layout &L = ctx->L;
    if ((!front_only && (size_t)P.units.size() * slot_floats_of_mode(P.mode) * sizeof(float) > L.slot_bytes_cap) ||
        L.units + P.units.size() * sizeof(Unit) > L.cta_begin_tc)
        return EGERIA_ERR_WORKSPACE;

    uint8_t *img;
    if (ctx->pinned_plans) {
        // One pinned image per plan slot: the copy below is truly asynchronous, so the image must not
        // be rewritten while an earlier upload from it is still queued (a caller whose pointers change
        // on every call can run more than kPlanSlots evaluations ahead of the GPU).
        if (ctx->plan_upload_pending[lru]) {
            EG_CUDA(cudaEventSynchronize(ctx->plan_uploaded[lru]));
            ctx->plan_upload_pending[lru] = false;
        }
        img = ctx->pinned_plans + (size_t)lru * L.plan_stride;
        memset(img, 0, L.plan_stride);
    } else {
        ctx->pack.assign(L.plan_stride, 0);
        img = ctx->pack.data();
    }
    const int box_rows = pitch_of_mode(P.mode);  // rows of one TMA box: all rows of one side
    CUtensorMap *maps = reinterpret_cast<CUtensorMap *>(img + L.tmaps);
    ModulePtrs *mods = reinterpret_cast<ModulePtrs *>(img + L.modules);
    if (ctx->tmpl_b != b) {  // the maps kept as templates are for another batch size
        ctx->tmpl.assign(2 * (size_t)M, CUtensorMap{});
        ctx->tmpl_valid.assign(2 * (size_t)M, 0);
        ctx->tmpl_b = b;
    }
    for (int m = 0; m < M; ++m) {
        mods[m] = ModulePtrs{At[m], Ar[m], ctx->d[m]};
        if (tc_ok[m] != 1) continue;
        const void *base[2] = {At[m], Ar[m]};
        for (int side = 0; side < 2; ++side) {
            const size_t k = 2 * (size_t)m + side;
            if (ctx->replace_address && ctx->tmpl_valid[k]) {
                // same shape, new place: copy the map and swap the address in (no re-encoding)
                maps[k] = ctx->tmpl[k];
                if (ctx->replace_address(&maps[k], const_cast<void *>(base[side])) == CUDA_SUCCESS) continue;
            }
            egeria_status s = encode_map(ctx, &maps[k], base[side], b, ctx->d[m], box_rows);
            if (s != EGERIA_OK) return s;
            ctx->tmpl[k] = maps[k];
            ctx->tmpl_valid[k] = 1;
        }
    }
    if (!P.units.empty()) memcpy(img + L.units, P.units.data(), P.units.size() * sizeof(Unit));
    if (front_only)
        memcpy(img + L.cta_begin_tc, front_cta_begin.data(), front_cta_begin.size() * sizeof(int32_t));
    else
        memcpy(img + L.cta_begin_tc, P.cta_begin_tc.data(), P.cta_begin_tc.size() * sizeof(int32_t));
    memcpy(img + L.cta_begin_simt, P.cta_begin_simt.data(), P.cta_begin_simt.size() * sizeof(int32_t));
    memcpy(img + L.sides, P.sides.data(), P.sides.size() * sizeof(SideInfo));
    if (!front_only && !P.cta_help.empty())  // (the image is zeroed: no help planned otherwise)
        memcpy(img + L.cta_help, P.cta_help.data(), P.cta_help.size() * sizeof(CtaHelp));
    memset(img + L.first_task, 0xff, L.first_task_bytes);  // -1: no task
    if (front_only)
        memcpy(img + L.first_task, bp->front_first_task.data(), bp->front_first_task.size() * sizeof(int32_t));
    else
        memcpy(img + L.first_task, P.first_task.data(), P.first_task.size() * sizeof(int32_t));
    // From pageable memory the runtime stages the bytes before returning, so `pack` may be reused.
    EG_CUDA(cudaMemcpyAsync(ctx->plan_region(lru), img, L.plan_stride, cudaMemcpyHostToDevice, stream));
    if (ctx->pinned_plans) {
        EG_CUDA(cudaEventRecord(ctx->plan_uploaded[lru], stream));
        ctx->plan_upload_pending[lru] = true;
    }
    e.b = b;
    e.front_only = front_only;
    e.weights_version = ctx->weights_version;
    e.At.assign(At, At + M);
    e.Ar.assign(Ar, Ar + M);
    e.last_use = ++ctx->use_clock;
    ctx->cur = lru;
    ctx->plan_b = b;
    return EGERIA_OK;
}

static cudaError_t launch_finalize(const FinParams &fp, int M, int b, cudaStream_t stream) {
    const dim3 grid(M, (b + kFinRowsPerCta - 1) / kFinRowsPerCta);
    switch (fin_nc_of_b(b)) {
        case 1: finalize_kernel<1><<<grid, kFinThreads, 0, stream>>>(fp); break;
        case 2: finalize_kernel<2><<<grid, kFinThreads, 0, stream>>>(fp); break;
        case 4: finalize_kernel<4><<<grid, kFinThreads, 0, stream>>>(fp); break;
        default: finalize_kernel<8><<<grid, kFinThreads, 0, stream>>>(fp); break;
    }
    return cudaGetLastError();
}

// Launched as a programmatic dependent of whatever kernel precedes it in the stream: its CTAs may
// become resident and set themselves up (barriers, tensor memory, their share of the plan) while
// that kernel's last CTAs are still running -- an evaluation kernel of this library says so early,
// any other kernel implicitly as its CTAs end.  The kernel itself waits (griddepcontrol.wait) before
// it reads an activation or touches anything in the workspace, so nothing is consumed early.
template <int MODE>
static cudaError_t launch_tc(int n_ctas, cudaStream_t stream, const TcParams &tp, bool programmatic) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_ctas);
    cfg.blockDim = dim3(kTcThreads);
    cfg.dynamicSmemBytes = TcCfg<MODE>::kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = programmatic ? 1 : 0;  // (not after a memset: an ordinary, fully serialised launch)
    return cudaLaunchKernelEx(&cfg, gram_tc_kernel<MODE>, tp);
}

static cudaError_t launch_tc_mode(int mode, int n_ctas, cudaStream_t stream, const TcParams &tp,
                                  bool programmatic = true) {
    switch (mode) {
        case kStacked32: return launch_tc<kStacked32>(n_ctas, stream, tp, programmatic);
        case kStacked64: return launch_tc<kStacked64>(n_ctas, stream, tp, programmatic);
        case kSingle1: return launch_tc<kSingle1>(n_ctas, stream, tp, programmatic);
        default: return launch_tc<kSingle2>(n_ctas, stream, tp, programmatic);
    }
}

static cudaError_t set_tc_attrs() {
    cudaError_t e = cudaFuncSetAttribute(gram_tc_kernel<kStacked32>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         TcCfg<kStacked32>::kSmemBytes);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(gram_tc_kernel<kStacked64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 TcCfg<kStacked64>::kSmemBytes);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(gram_tc_kernel<kSingle1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 TcCfg<kSingle1>::kSmemBytes);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(gram_tc_kernel<kSingle2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 TcCfg<kSingle2>::kSmemBytes);
    return e;
}

static egeria_status set_attrs(egeria_ctx *ctx) {
    if (ctx->attrs_set) return EGERIA_OK;
    EG_CUDA(set_tc_attrs());
    ctx->attrs_set = true;
    return EGERIA_OK;
}

}  // namespace egeria

// The unfreezing test of Algorithm 1 after an evaluation of the rule [Sec. 4.2.2 "Unfreezing"].
// Its outcome can change only when the learning rate does (the reference rate is set at a freeze
// to the rate then in force, which is not a tenth of itself), so the kernel is launched only after
// the first evaluation under a new rate.
static egeria_status unfreeze_test(egeria_ctx *ctx, cudaStream_t stream, uint8_t *out_mask) {
    const double lr = ctx->lr;
    if (!(lr > 0.0)) return EGERIA_OK;  // no rate given (or not a usable one): the rule is off
    const bool changed = (ctx->lr_checked > 0.0) && (lr != ctx->lr_checked);
    ctx->lr_checked = lr;
    if (!changed) return EGERIA_OK;
    unfreeze_check_kernel<<<1, 128, 0, stream>>>(ctx->slope_state(), ctx->M, lr, out_mask);
    if (cudaGetLastError() != cudaSuccess) return EGERIA_ERR_CUDA;
    ctx->launches++;
    return EGERIA_OK;
}

static egeria_status sp_loss_impl(egeria_ctx *ctx, void *cuda_stream, const void *const *At_in,
                                  const void *const *Ar_in, int b, const int64_t *d, float *out_losses, bool fuse_step,
                                  double *out_slopes, uint8_t *out_mask, const uint8_t *active = nullptr) {
    if (!ctx || !At_in || !Ar_in || !d || !out_losses) return EGERIA_ERR_INVALID_ARG;
    if (b < 2 || b > ctx->b_max) return EGERIA_ERR_INVALID_ARG;
    const void *const *At = At_in, *const *Ar = Ar_in;
    if (active) {  // the plan is keyed by the pointers: a module left out has none
        ctx->subset_t.assign(At_in, At_in + ctx->M);
        ctx->subset_r.assign(Ar_in, Ar_in + ctx->M);
        int n_active = 0;
        for (int m = 0; m < ctx->M; ++m) {
            if (active[m])
                ++n_active;
            else
                ctx->subset_t[m] = ctx->subset_r[m] = nullptr;
        }
        if (n_active == 0) return EGERIA_ERR_INVALID_ARG;
        At = ctx->subset_t.data();
        Ar = ctx->subset_r.data();
    }
    for (int m = 0; m < ctx->M; ++m) {
        if (d[m] != ctx->d[m]) return EGERIA_ERR_INVALID_ARG;
        if (active && !active[m]) continue;
        if (!At[m] || !Ar[m]) return EGERIA_ERR_INVALID_ARG;
        if ((reinterpret_cast<uintptr_t>(At[m]) | reinterpret_cast<uintptr_t>(Ar[m])) & 1) return EGERIA_ERR_INVALID_ARG;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    {
        // An evaluation carries state that belongs to this one call (which set of counters and of
        // partial slots, the rule's serial number): a graph would replay it with that state, and
        // read the partial rows of the replay before as its own.  Turned away, nothing recorded.
        cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(stream, &capturing) != cudaSuccess) return EGERIA_ERR_CUDA;
        if (capturing != cudaStreamCaptureStatusNone) return EGERIA_ERR_INVALID_ARG;
    }
    ctx->last_stream = stream;
    egeria_status s = set_attrs(ctx);
    if (s != EGERIA_OK) return s;
    poll_calibration(ctx);
    const bool front_only = fuse_step && (ctx->flags & EGERIA_FLAG_FRONT_ONLY);
    if (front_only && active) return EGERIA_ERR_INVALID_ARG;
    s = refresh_plan(ctx, stream, At, Ar, b, front_only);
    if (s != EGERIA_OK) return s;

    const Layout &L = ctx->L;
    const Plan &P = ctx->plans[ctx->cur].plan;
    const uint8_t *region = ctx->plan_region(ctx->cur);
    const int64_t slot_floats = slot_floats_of_mode(P.mode);
    cudaEvent_t ev0 = nullptr, ev1 = nullptr;
    if ((ctx->flags & EGERIA_FLAG_TIME_GRAM) && ctx->ev_used < kMaxTimedCalls * 2) {
        if (ctx->ev_used + 2 > ctx->ev_pool.size()) {
            cudaEvent_t a, c;
            EG_CUDA(cudaEventCreate(&a));
            EG_CUDA(cudaEventCreate(&c));
            ctx->ev_pool.push_back(a);
            ctx->ev_pool.push_back(c);
        }
        ev0 = ctx->ev_pool[ctx->ev_used];
        ev1 = ctx->ev_pool[ctx->ev_used + 1];
        ctx->ev_used += 2;
        EG_CUDA(cudaEventRecord(ev0, stream));
    }
    FinCommon fc;
    // How the finish learns that a partial row has arrived (Plan::validate_rows), and which slots
    // the launch uses.  Launches that validate alternate between two sets of slots; each empties what
    // the one before wrote into the other set (the tensor-core kernel does, so there must be one).
    const size_t plan_slot_bytes = (size_t)ctx->plans[ctx->cur].slot_units * slot_floats * sizeof(float);
    fc.sentinel = (P.validate_rows && P.n_units_tc > 0 && plan_slot_bytes <= L.slot_set_bytes) ? 1u : 0u;
    fc.wait_limit_ns = ctx->stall_next ? kTestWaitLimitNs : kWaitLimitNs;
    bool after_memset = false;
    float *slot_base = ctx->at<float>(L.slots);
    uint4 *empty_ptr = nullptr;
    uint32_t empty_n = 0;
    if (fc.sentinel) {
        if (ctx->slots_dirty) {
            // the launch before left what it wrote all over the slots (the other protocol)
            EG_CUDA(cudaMemsetAsync(ctx->ws + L.slots, 0xff, L.slot_bytes_cap, stream));
            ctx->slots_dirty = false;
            ctx->set_dirty[0] = ctx->set_dirty[1] = 0;
            after_memset = true;
        }
        const int set = ctx->val_set, other = set ^ 1;
        slot_base = reinterpret_cast<float *>(ctx->ws + L.slots + (size_t)set * L.slot_set_bytes);
        empty_ptr = reinterpret_cast<uint4 *>(ctx->ws + L.slots + (size_t)other * L.slot_set_bytes);
        empty_n = (uint32_t)(ctx->set_dirty[other] / sizeof(uint4));
        ctx->set_dirty[other] = 0;
        if (plan_slot_bytes > ctx->set_dirty[set]) ctx->set_dirty[set] = plan_slot_bytes;
        ctx->val_set = other;
    } else if (!P.units.empty()) {
        ctx->slots_dirty = true;
    }
    fc.slots = slot_base;
    fc.slot_floats = slot_floats;
    fc.status = ctx->at<int32_t>(L.status);
    fc.slots_floats = (int64_t)((fc.sentinel ? L.slot_set_bytes : L.slot_bytes_cap) / sizeof(float));
    fc.chunk_doubles = (int64_t)(L.chunk_bytes / sizeof(double));
    fc.sides = reinterpret_cast<const SideInfo *>(region + L.sides);
    fc.b = b;
    fc.out_losses = out_losses;
    fc.rowloss = ctx->at<double>(L.rowloss);
    fc.keep = (ctx->flags & EGERIA_FLAG_KEEP_GRAMS) ? ctx->at<float>(L.keep) : nullptr;
    fc.chunk_sums = ctx->at<double>(L.chunk);
    fc.fuse_step = fuse_step ? 1 : 0;
    fc.lr = ctx->lr;
    fc.rule_flags = ctx->rule_flags();
    if (fuse_step) ctx->rule_evals++;
    fc.rule_serial = ctx->rule_evals;
    fc.M = ctx->M;
    fc.st = ctx->slope_state();
    fc.out_slopes = out_slopes;
    fc.out_mask = out_mask;
    if (P.n_units_tc > 0) {
        TcParams tp;
        tp.tmaps = reinterpret_cast<const CUtensorMap *>(region + L.tmaps);
        tp.units = reinterpret_cast<const Unit *>(region + L.units);
        tp.cta_begin = reinterpret_cast<const int32_t *>(region + L.cta_begin_tc);
        tp.cta_help = front_only ? nullptr : reinterpret_cast<const CtaHelp *>(region + L.cta_help);
        tp.front_word = front_only ? ctx->slope_state().front : nullptr;
        tp.cta_stride = kMaxCtas + 1;
        tp.first_task = reinterpret_cast<const int32_t *>(region + L.first_task);
        tp.first_stride = kMaxCtas * kEpiWarps;
        tp.empty_ptr = empty_ptr;
        tp.empty_n = empty_n;
        tp.empty_floats = (int64_t)(L.slot_set_bytes / sizeof(float));
        tp.n_units = front_only ? (int)P.units.size() : P.n_units_tc;
        tp.slots = slot_base;
        tp.status = ctx->at<int32_t>(L.status);
        FinCounters *sets = ctx->at<FinCounters>(L.fin_ctr);
        const uint32_t set = ctx->tc_launches & 1u;
        tp.ctr = sets + (size_t)set * ctx->M;
        tp.ctr_next = sets + (size_t)(set ^ 1u) * ctx->M;
        tp.M = ctx->M;
        tp.n_active = 0;
        if (front_only) {
            tp.n_active = 1;
        } else {
            for (int m = 0; m < ctx->M; ++m) tp.n_active += (P.sides[2 * (size_t)m].tensor_core && P.sides[2 * (size_t)m].module_units > 0);
        }
        tp.fin = fc;
        const bool log_it = !ctx->calibrated && ctx->host_log && ctx->calib_enqueued < kCalibLaunches &&
                            P.all_ctas_busy_tc;
        tp.log = log_it ? ctx->at<CtaLog>(L.cta_log) : nullptr;
        tp.serial = ctx->tc_launches + 1;
        tp.early_inputs = (ctx->flags & EGERIA_FLAG_OVERLAP) ? 1u : 0u;
        tp.test_stall = ctx->stall_next;
        tp.wait_limit_ns = ctx->stall_next ? kTestWaitLimitNs : kWaitLimitNs;
        ctx->stall_next = 0;
        if (launch_tc_mode(P.mode, ctx->n_ctas, stream, tp, !after_memset) != cudaSuccess) return EGERIA_ERR_CUDA;
        if (log_it) {
            const int k = ctx->calib_enqueued;
            EG_CUDA(cudaMemcpyAsync(ctx->host_log + (size_t)k * kMaxCtas, tp.log, (size_t)ctx->n_ctas * sizeof(CtaLog),
                                    cudaMemcpyDeviceToHost, stream));
            ctx->calib_serial[k] = tp.serial;
            ctx->calib_enqueued = k + 1;
        }
        ctx->tc_launches++;
        ctx->launches++;
    }
    const bool any_simt = (int)P.units.size() > P.n_units_tc;
    if (any_simt) {
        SimtParams sp;
        sp.modules = reinterpret_cast<const ModulePtrs *>(region + L.modules);
        sp.units = reinterpret_cast<const Unit *>(region + L.units) + P.n_units_tc;
        sp.cta_begin = reinterpret_cast<const int32_t *>(region + L.cta_begin_simt);
        sp.slots = slot_base;
        sp.slot_floats = slot_floats;
        sp.b = b;
        sp.mode = P.mode;
        gram_simt_kernel<<<ctx->n_ctas, kSimtThreads, 0, stream>>>(sp);
        if (cudaGetLastError() != cudaSuccess) return EGERIA_ERR_CUDA;
        ctx->launches++;
    }
    if (ev1) EG_CUDA(cudaEventRecord(ev1, stream));
    if (any_simt) {
        // the CUDA-core modules are finished by a kernel of their own
        FinParams fp;
        fp.c = fc;
        fp.tickets = ctx->at<int32_t>(L.tickets);
        if (launch_finalize(fp, ctx->M, b, stream) != cudaSuccess) return EGERIA_ERR_CUDA;
        ctx->launches++;
    }
    if (fuse_step) return unfreeze_test(ctx, stream, out_mask);
    return EGERIA_OK;
}

extern "C" {

egeria_status egeria_sp_loss_batch(egeria_ctx *ctx, void *cuda_stream, const void *const *At, const void *const *Ar,
                                   int b, const int64_t *d, float *out_losses) {
    HostRange range("egeria_sp_loss_batch");
    return sp_loss_impl(ctx, cuda_stream, At, Ar, b, d, out_losses, false, nullptr, nullptr);
}

egeria_status egeria_plasticity_evaluate(egeria_ctx *ctx, void *cuda_stream, const void *const *At,
                                         const void *const *Ar, int b, const int64_t *d, float *out_losses,
                                         double *out_slopes, uint8_t *out_mask) {
    HostRange range("egeria_plasticity_evaluate");
    return sp_loss_impl(ctx, cuda_stream, At, Ar, b, d, out_losses, true, out_slopes, out_mask);
}

egeria_status egeria_sp_loss_subset(egeria_ctx *ctx, void *cuda_stream, const void *const *At, const void *const *Ar,
                                    int b, const int64_t *d, const uint8_t *active, float *out_losses) {
    if (!active) return EGERIA_ERR_INVALID_ARG;
    return sp_loss_impl(ctx, cuda_stream, At, Ar, b, d, out_losses, false, nullptr, nullptr, active);
}

egeria_status egeria_plasticity_evaluate_subset(egeria_ctx *ctx, void *cuda_stream, const void *const *At,
                                                const void *const *Ar, int b, const int64_t *d, const uint8_t *active,
                                                float *out_losses, double *out_slopes, uint8_t *out_mask) {
    if (!active) return EGERIA_ERR_INVALID_ARG;
    return sp_loss_impl(ctx, cuda_stream, At, Ar, b, d, out_losses, true, out_slopes, out_mask, active);
}

egeria_status egeria_sp_loss_batch_host(egeria_ctx *ctx, void *cuda_stream, const void *const *At_host,
                                        const void *const *Ar_host, int b, const int64_t *d, float *out_losses_host) {
    if (!ctx || !At_host || !Ar_host || !d || !out_losses_host) return EGERIA_ERR_INVALID_ARG;
    if (!(ctx->flags & EGERIA_FLAG_HOST_STAGING)) return EGERIA_ERR_WORKSPACE;
    if (b < 2 || b > ctx->b_max) return EGERIA_ERR_INVALID_ARG;
    HostRange range("egeria_sp_loss_batch_host");
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    {
        // (the call synchronises the stream, which a capturing stream cannot do; and see sp_loss_impl)
        cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(stream, &capturing) != cudaSuccess) return EGERIA_ERR_CUDA;
        if (capturing != cudaStreamCaptureStatusNone) return EGERIA_ERR_INVALID_ARG;
    }
    for (int m = 0; m < ctx->M; ++m) {
        if (d[m] != ctx->d[m] || !At_host[m] || !Ar_host[m]) return EGERIA_ERR_INVALID_ARG;
        const size_t bytes = (size_t)b * d[m] * 2;
        EG_CUDA(cudaMemcpyAsync(ctx->staging_t[m], At_host[m], bytes, cudaMemcpyHostToDevice, stream));
        EG_CUDA(cudaMemcpyAsync(ctx->staging_r[m], Ar_host[m], bytes, cudaMemcpyHostToDevice, stream));
    }
    float *dev_losses = ctx->at<float>(ctx->L.losses);
    egeria_status s = egeria_sp_loss_batch(ctx, cuda_stream, ctx->staging_t.data(), ctx->staging_r.data(), b, d,
                                           dev_losses);
    if (s != EGERIA_OK) return s;
    EG_CUDA(cudaMemcpyAsync(out_losses_host, dev_losses, (size_t)ctx->M * sizeof(float), cudaMemcpyDeviceToHost,
                            stream));
    EG_CUDA(cudaStreamSynchronize(stream));
    return EGERIA_OK;
}

egeria_status egeria_plasticity_step(egeria_ctx *ctx, void *cuda_stream, const float *losses, double *out_slopes,
                                     uint8_t *out_mask) {
    if (!ctx || !losses) return EGERIA_ERR_INVALID_ARG;
    HostRange range("egeria_plasticity_step");
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    ctx->last_stream = stream;
    ctx->rule_evals++;
    plasticity_step_kernel<<<ctx->M, 32, 0, stream>>>(ctx->slope_state(), ctx->M, ctx->rule_flags(), ctx->rule_evals,
                                                      ctx->lr, losses, out_slopes, out_mask);
    if (cudaGetLastError() != cudaSuccess) return EGERIA_ERR_CUDA;
    ctx->launches++;
    return unfreeze_test(ctx, stream, out_mask);
}

egeria_status egeria_plasticity_replay(egeria_ctx *ctx, void *cuda_stream, const float *hist, int H,
                                       double *out_slopes, uint8_t *out_mask, int32_t *out_freeze_eval) {
    if (!ctx || !hist || H < 0 || !out_mask) return EGERIA_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    ctx->last_stream = stream;
    const int grid = (ctx->flags & EGERIA_FLAG_FRONTMOST) ? 1 : ctx->M;
    plasticity_replay_kernel<<<grid, 32, 2 * (size_t)ctx->W_cap * sizeof(double), stream>>>(
        ctx->at<float>(ctx->L.T), ctx->M, ctx->slope_state().W_cur, ctx->W_cap, ctx->rule_flags(), hist, H, out_slopes,
        out_mask, out_freeze_eval);
    if (cudaGetLastError() != cudaSuccess) return EGERIA_ERR_CUDA;
    ctx->launches++;
    return EGERIA_OK;
}

egeria_status egeria_plasticity_replay_lr(egeria_ctx *ctx, void *cuda_stream, const float *hist, const double *lr,
                                          int H, double *out_slopes, uint8_t *out_frozen, int32_t *out_window,
                                          uint8_t *out_restarted, uint8_t *out_mask, int32_t *out_freeze_eval) {
    if (!ctx || !hist || H < 0) return EGERIA_ERR_INVALID_ARG;
    const size_t smem = (size_t)ctx->M * sizeof(ReplayModule);
    if (smem > 40 * 1024) return EGERIA_ERR_UNSUPPORTED_SHAPE;  // per-module scalars live in shared memory
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    ctx->last_stream = stream;
    int warps = ctx->M < 32 ? ctx->M : 32;
    plasticity_replay_lr_kernel<<<1, 32 * warps, smem, stream>>>(
        ctx->at<float>(ctx->L.T), ctx->at<double>(ctx->L.replay_raw), ctx->at<double>(ctx->L.replay_plist), ctx->W_cap,
        ctx->slope_state().W_cur, ctx->M, ctx->rule_flags(), hist, lr, H, out_slopes, out_frozen, out_window,
        out_restarted, out_mask, out_freeze_eval);
    if (cudaGetLastError() != cudaSuccess) return EGERIA_ERR_CUDA;
    ctx->launches++;
    return EGERIA_OK;
}

egeria_status egeria_plasticity_reset(egeria_ctx *ctx, void *cuda_stream, int halve_W) {
    if (!ctx) return EGERIA_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    ctx->last_stream = stream;
    plasticity_clear_kernel<<<(ctx->M + 127) / 128, 128, 0, stream>>>(ctx->slope_state(), ctx->M, 0, halve_W ? 1 : 0);
    if (cudaGetLastError() != cudaSuccess) return EGERIA_ERR_CUDA;
    ctx->launches++;
    return EGERIA_OK;
}

egeria_status egeria_bootstrap_step(egeria_ctx *ctx, void *cuda_stream, const float *train_loss, float rate_tol,
                                    double *out_rate, uint8_t *out_done) {
    if (!ctx || !train_loss || !(rate_tol > 0.f)) return EGERIA_ERR_INVALID_ARG;
    if (ctx->W_cap < 2) return EGERIA_ERR_INVALID_ARG;  // no line through one point
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    ctx->last_stream = stream;
    bootstrap_step_kernel<<<1, 32, 0, stream>>>(ctx->boot_state(), ctx->W_cap, (double)rate_tol, train_loss, out_rate,
                                                out_done);
    if (cudaGetLastError() != cudaSuccess) return EGERIA_ERR_CUDA;
    ctx->launches++;
    return EGERIA_OK;
}

egeria_status egeria_bootstrap_replay(egeria_ctx *ctx, void *cuda_stream, const float *loss_hist, int H, float rate_tol,
                                      double *out_rates, int32_t *out_end) {
    if (!ctx || !loss_hist || H < 0 || !(rate_tol > 0.f) || !out_end) return EGERIA_ERR_INVALID_ARG;
    if (ctx->W_cap < 2) return EGERIA_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    ctx->last_stream = stream;
    bootstrap_replay_kernel<<<1, 32, 2 * (size_t)ctx->W_cap * sizeof(double), stream>>>(
        ctx->W_cap, (double)rate_tol, loss_hist, H, out_rates, out_end);
    if (cudaGetLastError() != cudaSuccess) return EGERIA_ERR_CUDA;
    ctx->launches++;
    return EGERIA_OK;
}

egeria_status egeria_bootstrap_reset(egeria_ctx *ctx, void *cuda_stream) {
    if (!ctx) return EGERIA_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    ctx->last_stream = stream;
    bootstrap_clear_kernel<<<1, 1, 0, stream>>>(ctx->boot_state());
    if (cudaGetLastError() != cudaSuccess) return EGERIA_ERR_CUDA;
    ctx->launches++;
    return EGERIA_OK;
}

// What export writes in front of the raw state: enough to refuse a buffer from another set-up.
struct StateHeader {
    uint32_t magic;
    int32_t M, W_cap, pad;
    uint32_t rule_evals, flags;
    uint64_t state_bytes;
    double lr, lr_checked;
};
constexpr uint32_t kStateMagic = 0x45474552u;  // "EGER"

size_t egeria_plasticity_state_bytes(const egeria_ctx *ctx) {
    return ctx ? sizeof(StateHeader) + (ctx->L.rule_end - ctx->L.rule0) : 0;
}

egeria_status egeria_plasticity_export(egeria_ctx *ctx, void *cuda_stream, void *host_buffer, size_t buffer_bytes) {
    if (!ctx || !host_buffer) return EGERIA_ERR_INVALID_ARG;
    if (buffer_bytes < egeria_plasticity_state_bytes(ctx)) return EGERIA_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    ctx->last_stream = stream;
    StateHeader h;
    h.magic = kStateMagic;
    h.M = ctx->M;
    h.W_cap = ctx->W_cap;
    h.pad = 0;
    h.lr = ctx->lr;
    h.lr_checked = ctx->lr_checked;
    h.rule_evals = ctx->rule_evals;
    h.flags = ctx->flags & (EGERIA_FLAG_SIGNED_SLOPE | EGERIA_FLAG_AUTO_T | EGERIA_FLAG_FRONTMOST);
    h.state_bytes = ctx->L.rule_end - ctx->L.rule0;
    memcpy(host_buffer, &h, sizeof(h));
    EG_CUDA(cudaMemcpyAsync(static_cast<uint8_t *>(host_buffer) + sizeof(h), ctx->ws + ctx->L.rule0, h.state_bytes,
                            cudaMemcpyDeviceToHost, stream));
    EG_CUDA(cudaStreamSynchronize(stream));
    return EGERIA_OK;
}

egeria_status egeria_plasticity_import(egeria_ctx *ctx, void *cuda_stream, const void *host_buffer, size_t buffer_bytes) {
    if (!ctx || !host_buffer || buffer_bytes < sizeof(StateHeader)) return EGERIA_ERR_INVALID_ARG;
    StateHeader h;
    memcpy(&h, host_buffer, sizeof(h));
    const uint32_t rule_bits = ctx->flags & (EGERIA_FLAG_SIGNED_SLOPE | EGERIA_FLAG_AUTO_T | EGERIA_FLAG_FRONTMOST);
    if (h.magic != kStateMagic || h.M != ctx->M || h.W_cap != ctx->W_cap || h.flags != rule_bits ||
        h.state_bytes != ctx->L.rule_end - ctx->L.rule0)
        return EGERIA_ERR_INVALID_ARG;
    if (buffer_bytes < sizeof(h) + h.state_bytes) return EGERIA_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    ctx->last_stream = stream;
    EG_CUDA(cudaMemcpyAsync(ctx->ws + ctx->L.rule0, static_cast<const uint8_t *>(host_buffer) + sizeof(h), h.state_bytes,
                            cudaMemcpyHostToDevice, stream));
    EG_CUDA(cudaStreamSynchronize(stream));  // the buffer may be pageable: it is free again on return
    ctx->lr = h.lr;
    ctx->lr_checked = h.lr_checked;
    ctx->rule_evals = h.rule_evals;
    return EGERIA_OK;
}

egeria_status egeria_debug_dump_gram(egeria_ctx *ctx, void *cuda_stream, int module, float *Gt_norm,
                                     float *Gr_norm) {
    if (!ctx || !Gt_norm || !Gr_norm || module < 0 || module >= ctx->M) return EGERIA_ERR_INVALID_ARG;
    if (!(ctx->flags & EGERIA_FLAG_KEEP_GRAMS)) return EGERIA_ERR_WORKSPACE;
    if (ctx->plan_b < 2) return EGERIA_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t bb = (size_t)ctx->plan_b * ctx->plan_b;
    const float *keep = ctx->at<float>(ctx->L.keep);
    EG_CUDA(cudaMemcpyAsync(Gt_norm, keep + (size_t)(2 * module) * bb, bb * sizeof(float), cudaMemcpyDeviceToDevice,
                            stream));
    EG_CUDA(cudaMemcpyAsync(Gr_norm, keep + (size_t)(2 * module + 1) * bb, bb * sizeof(float),
                            cudaMemcpyDeviceToDevice, stream));
    return EGERIA_OK;
}

egeria_status egeria_gram_kernel_time(egeria_ctx *ctx, double *total_ms, int64_t *n_calls) {
    if (!ctx || !total_ms || !n_calls) return EGERIA_ERR_INVALID_ARG;
    if (!(ctx->flags & EGERIA_FLAG_TIME_GRAM)) return EGERIA_ERR_INVALID_ARG;
    double sum = 0.0;
    for (size_t i = 0; i + 1 < ctx->ev_used; i += 2) {
        EG_CUDA(cudaEventSynchronize(ctx->ev_pool[i + 1]));
        float ms = 0.f;
        EG_CUDA(cudaEventElapsedTime(&ms, ctx->ev_pool[i], ctx->ev_pool[i + 1]));
        sum += ms;
    }
    *total_ms = sum;
    *n_calls = (int64_t)(ctx->ev_used / 2);
    ctx->ev_used = 0;
    return EGERIA_OK;
}

egeria_status egeria_debug_stall_next(egeria_ctx *ctx, int kind) {
    if (!ctx || kind < 0 || kind > 2) return EGERIA_ERR_INVALID_ARG;
    ctx->stall_next = (uint32_t)kind;
    return EGERIA_OK;
}

int egeria_build_is_checked(void) { return kCheckedBuild ? 1 : 0; }

egeria_status egeria_debug_check_record(egeria_ctx *ctx, int32_t *out_record) {
    if (!ctx || !out_record) return EGERIA_ERR_INVALID_ARG;
    EG_CUDA(cudaStreamSynchronize(ctx->last_stream));
    EG_CUDA(cudaMemcpy(out_record, ctx->ws + ctx->L.status + sizeof(int32_t), 5 * sizeof(int32_t), cudaMemcpyDeviceToHost));
    EG_CUDA(cudaMemset(ctx->ws + ctx->L.status + sizeof(int32_t), 0, 5 * sizeof(int32_t)));  // the next failure is recorded afresh
    return EGERIA_OK;
}

egeria_status egeria_device_status(egeria_ctx *ctx) {
    if (!ctx) return EGERIA_ERR_INVALID_ARG;
    EG_CUDA(cudaStreamSynchronize(ctx->last_stream));
    int32_t word = 0;
    EG_CUDA(cudaMemcpy(&word, ctx->ws + ctx->L.status, sizeof(word), cudaMemcpyDeviceToHost));
    if (word != 0) {
        // a kernel that gave up leaves its progress counters and tickets half-way: start afresh
        EG_CUDA(cudaMemset(ctx->ws + ctx->L.fin_ctr, 0, (size_t)2 * ctx->M * sizeof(FinCounters)));
        EG_CUDA(cudaMemset(ctx->ws + ctx->L.tickets, 0, (size_t)ctx->M * sizeof(int32_t)));
        // ... and partial rows that were written and never read: every slot empty again
        EG_CUDA(cudaMemset(ctx->ws + ctx->L.slots, 0xff, ctx->L.slot_bytes_cap));
        ctx->slots_dirty = false;
        ctx->set_dirty[0] = ctx->set_dirty[1] = 0;
        EG_CUDA(cudaMemset(ctx->ws + ctx->L.status, 0, sizeof(int32_t)));
    }
    if (word == kStatusTimeout) return EGERIA_ERR_TIMEOUT;
    if (word == kStatusCheck) return EGERIA_ERR_CHECK;  // (what failed: egeria_debug_check_record)
    return word == 0 ? EGERIA_OK : EGERIA_ERR_CUDA;
}

}  // extern "C"

// =====================================================================================
// Allocation-free single-module evaluation (egeria_sp_loss_static).
//
// All scratch of this entry point is the fixed array below, which is part of the library
// image: every GPU that loads the library carries these 6 MiB until the process exits.
// Nothing here calls cudaMalloc, cudaFree or any routine that allocates device memory.
// =====================================================================================
namespace egeria {

constexpr int kStaticMaxB = 128;                   // largest b of the allocation-free entry point
constexpr int kStaticCtas = 32;                    // CTAs the feature axis is split over
constexpr size_t kStaticScratchBytes = 6u << 20;   // 6 MiB
constexpr int kStaticMaxDevices = 64;
constexpr size_t kStaticTableBytes = 4096;         // host image of the tables at the start of the array

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

struct StaticLayout {
    size_t tmaps, modules, units, cta_begin_tc, cta_begin_simt, sides, rowloss, ticket, slots, total;
};

static StaticLayout static_layout() {
    StaticLayout L;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        const size_t o = off;
        off = align_up(off + bytes, 256);
        return o;
    };
    L.tmaps = take(2 * sizeof(CUtensorMap));
    L.modules = take(sizeof(ModulePtrs));
    L.units = take((size_t)max_units(1, kSingle1, kStaticCtas) * sizeof(Unit));
    L.cta_begin_tc = take((kStaticCtas + 1) * sizeof(int32_t));
    L.cta_begin_simt = take((kStaticCtas + 1) * sizeof(int32_t));
    L.sides = take(2 * sizeof(SideInfo));
    L.rowloss = take(kMaxB * sizeof(double));
    L.ticket = take(8 * sizeof(int32_t) + 2 * sizeof(FinCounters));  // [0] finalisation ticket, [1] status word (+ the checked build's record),
                                                                     // then two sets of progress counters
    L.slots = take((size_t)max_units(1, kSingle1, kStaticCtas) * slot_floats_of_mode(kSingle1) * sizeof(float));
    L.total = off;
    return L;
}

// Per-device set-up state.  g_static_scratch is a host-side stand-in for the symbol, not a
// device address: the address a kernel may use comes from cudaGetSymbolAddress, asked once
// per device with that device current.
struct StaticDevice {
    unsigned char *scratch = nullptr;
    EncodeTiledFn encode = nullptr;
};
static StaticDevice g_static_dev[kStaticMaxDevices];

static egeria_status static_setup(int dev, StaticDevice **out) {
    if (dev < 0 || dev >= kStaticMaxDevices) return EGERIA_ERR_UNSUPPORTED_DEVICE;
    StaticDevice &sd = g_static_dev[dev];
    if (!sd.scratch) {
        cudaDeviceProp prop;
        EG_CUDA(cudaGetDeviceProperties(&prop, dev));
        if (prop.major != 10) return EGERIA_ERR_UNSUPPORTED_DEVICE;
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return EGERIA_ERR_CUDA;
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess || !fn)
            return EGERIA_ERR_CUDA;
        EG_CUDA(set_tc_attrs());
        sd.encode = reinterpret_cast<EncodeTiledFn>(fn);
        sd.scratch = static_cast<unsigned char *>(ptr);
    }
    *out = &sd;
    return EGERIA_OK;
}

}  // namespace egeria

extern "C" egeria_status egeria_sp_loss_static(void *cuda_stream, const void *At, const void *Ar, int b, int64_t d,
                                               float *out_loss) {
    if (!At || !Ar || !out_loss || b < 2) return EGERIA_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(At) | reinterpret_cast<uintptr_t>(Ar)) & 1) return EGERIA_ERR_INVALID_ARG;
    if (b > kStaticMaxB) return EGERIA_ERR_UNSUPPORTED_SHAPE;  // beyond the fixed scratch
    if (d < 1 || d > (int64_t)0x7fffffff - 2 * kKBlock) return EGERIA_ERR_UNSUPPORTED_SHAPE;
    const StaticLayout L = static_layout();
    static_assert(kStaticScratchBytes >= (5u << 20), "scratch array too small for its layout");
    if (L.total > kStaticScratchBytes) return EGERIA_ERR_WORKSPACE;

    int dev = 0;
    EG_CUDA(cudaGetDevice(&dev));
    StaticDevice *sd = nullptr;
    egeria_status s = static_setup(dev, &sd);
    if (s != EGERIA_OK) return s;
    unsigned char *ws = sd->scratch;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // The call copies from host memory that dies when it returns; captured into a graph, those
    // copies would read dead memory at replay.  Refuse rather than record them.
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    EG_CUDA(cudaStreamIsCapturing(stream, &capturing));
    if (capturing != cudaStreamCaptureStatusNone) return EGERIA_ERR_INVALID_ARG;

    const uint8_t tc_ok = (reinterpret_cast<uintptr_t>(At) % 16 == 0) && (reinterpret_cast<uintptr_t>(Ar) % 16 == 0) &&
                          (d % 8 == 0);
    Plan P;
    build_plan(1, &d, b, kStaticCtas, &tc_ok, P, nullptr, kEpiWarps, false, false);  // every row from the cursor
    if ((int64_t)P.units.size() > max_units(1, kSingle1, kStaticCtas)) return EGERIA_ERR_WORKSPACE;

    CUtensorMap maps[2];
    memset(maps, 0, sizeof(maps));
    if (tc_ok) {
        const int box_rows = pitch_of_mode(P.mode);
        const void *bases[2] = {At, Ar};
        for (int side = 0; side < 2; ++side) {
            cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)b};
            cuuint64_t strides[1] = {(cuuint64_t)d * 2};
            cuuint32_t box[2] = {(cuuint32_t)kKBlock, (cuuint32_t)box_rows};
            cuuint32_t estr[2] = {1, 1};
            if (sd->encode(&maps[side], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(bases[side]), dims,
                           strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
                return EGERIA_ERR_CUDA;
        }
    }
    // The array keeps whatever the previous call left: the ticket, the status word and the
    // progress counters must start at zero; everything else is overwritten before it is read.
    // The tables the kernels read (tensor maps, pointers, units, ranges, slot ranges) lie next to
    // each other at the start of the array and go up in ONE copy from one host image.  The image is
    // ordinary (pageable) memory: the runtime stages such a copy before it returns, so the image
    // may die with this call.
    unsigned char image[kStaticTableBytes];
    if (L.rowloss > sizeof(image)) return EGERIA_ERR_WORKSPACE;
    memset(image, 0, L.rowloss);
    const ModulePtrs mod{At, Ar, d};
    memcpy(image + L.tmaps, maps, sizeof(maps));
    memcpy(image + L.modules, &mod, sizeof(mod));
    memcpy(image + L.units, P.units.data(), P.units.size() * sizeof(Unit));
    memcpy(image + L.cta_begin_tc, P.cta_begin_tc.data(), P.cta_begin_tc.size() * sizeof(int32_t));
    memcpy(image + L.cta_begin_simt, P.cta_begin_simt.data(), P.cta_begin_simt.size() * sizeof(int32_t));
    memcpy(image + L.sides, P.sides.data(), P.sides.size() * sizeof(SideInfo));
    EG_CUDA(cudaMemsetAsync(ws + L.ticket, 0, 8 * sizeof(int32_t) + 2 * sizeof(FinCounters), stream));
    EG_CUDA(cudaMemcpyAsync(ws, image, L.rowloss, cudaMemcpyHostToDevice, stream));
    // A kernel that gives up (a bounded wait ran out) writes no loss: leave a NaN there for that case.
    EG_CUDA(cudaMemsetAsync(out_loss, 0xff, sizeof(float), stream));

    const int64_t slot_floats = slot_floats_of_mode(P.mode);
    int32_t *ticket = reinterpret_cast<int32_t *>(ws + L.ticket);
    FinCommon fc;
    fc.slots = reinterpret_cast<float *>(ws + L.slots);
    fc.slot_floats = slot_floats;
    fc.sentinel = 0u;  // counters and fences say when a partial is complete: the scratch needs no preparation
    fc.wait_limit_ns = kWaitLimitNs;
    fc.status = ticket + 1;
    fc.slots_floats = (int64_t)max_units(1, kSingle1, kStaticCtas) * slot_floats_of_mode(kSingle1);
    fc.chunk_doubles = 0;
    fc.sides = reinterpret_cast<const SideInfo *>(ws + L.sides);
    fc.b = b;
    fc.out_losses = out_loss;
    fc.rowloss = reinterpret_cast<double *>(ws + L.rowloss);
    fc.keep = nullptr;
    fc.chunk_sums = nullptr;
    fc.fuse_step = 0;
    fc.lr = NAN;
    fc.rule_flags = 0;
    fc.rule_serial = 0;
    fc.M = 1;
    fc.st = SlopeState{};
    fc.out_slopes = nullptr;
    fc.out_mask = nullptr;
    if (P.n_units_tc > 0) {
        TcParams tp;
        tp.tmaps = reinterpret_cast<const CUtensorMap *>(ws + L.tmaps);
        tp.units = reinterpret_cast<const Unit *>(ws + L.units);
        tp.cta_begin = reinterpret_cast<const int32_t *>(ws + L.cta_begin_tc);
        tp.cta_help = nullptr;
        tp.front_word = nullptr;
        tp.cta_stride = 0;
        tp.first_task = nullptr;
        tp.first_stride = 0;
        tp.empty_ptr = nullptr;
        tp.empty_n = 0;
        tp.empty_floats = 0;
        tp.n_units = P.n_units_tc;
        tp.slots = reinterpret_cast<float *>(ws + L.slots);
        tp.status = ticket + 1;
        tp.ctr = reinterpret_cast<FinCounters *>(ticket + 8);
        tp.ctr_next = tp.ctr + 1;
        tp.log = nullptr;
        tp.serial = 0;
        tp.early_inputs = 0;
        tp.test_stall = 0;
        tp.wait_limit_ns = kWaitLimitNs;
        tp.M = 1;
        tp.n_active = 1;
        tp.fin = fc;
        if (launch_tc_mode(P.mode, kStaticCtas, stream, tp) != cudaSuccess) return EGERIA_ERR_CUDA;
    } else {
        SimtParams sp;
        sp.modules = reinterpret_cast<const ModulePtrs *>(ws + L.modules);
        sp.units = reinterpret_cast<const Unit *>(ws + L.units);
        sp.cta_begin = reinterpret_cast<const int32_t *>(ws + L.cta_begin_simt);
        sp.slots = reinterpret_cast<float *>(ws + L.slots);
        sp.slot_floats = slot_floats;
        sp.b = b;
        sp.mode = P.mode;
        gram_simt_kernel<<<kStaticCtas, kSimtThreads, 0, stream>>>(sp);
        if (cudaGetLastError() != cudaSuccess) return EGERIA_ERR_CUDA;
        FinParams fp;
        fp.c = fc;
        fp.tickets = ticket;
        if (launch_finalize(fp, 1, b, stream) != cudaSuccess) return EGERIA_ERR_CUDA;
    }
    return EGERIA_OK;
}

extern "C" egeria_status egeria_sp_loss_static_status(void) {
    int dev = 0;
    EG_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kStaticMaxDevices || !g_static_dev[dev].scratch) return EGERIA_OK;  // nothing ran here yet
    const StaticLayout L = static_layout();
    int32_t word = 0;
    EG_CUDA(cudaMemcpy(&word, g_static_dev[dev].scratch + L.ticket + sizeof(int32_t), sizeof(word),
                       cudaMemcpyDeviceToHost));
    if (word == kStatusTimeout) return EGERIA_ERR_TIMEOUT;
    return word == 0 ? EGERIA_OK : EGERIA_ERR_CUDA;
}
