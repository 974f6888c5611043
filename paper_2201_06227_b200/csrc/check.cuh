// Index checks of the checked build (-DEGERIA_CHECKED; the second library the build script makes).
// The memory-checking tools are not available where this library is developed, so the kernels can
// check themselves: every index that comes from a table in memory (unit table, slot ranges, first
// tasks, cursors) and every offset into a slot, the staging area, the chunk scratch or tensor
// memory is compared with its bound before it is used.  A failed check records what it saw once
// (first failure wins), raises kStatusCheck in the status word and makes the caller SKIP the
// access; nothing traps.  In the ordinary build eg_check() is the constant true and costs nothing.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace egeria {

constexpr int kStatusCheck = 7;  // == EGERIA_ERR_CHECK; above kStatusTimeout, so that atomicMax keeps it

// What failed (status word 1).
enum CheckCode : int32_t {
    kCheckUnitRange = 1,   // a CTA's range of the unit table
    kCheckUnit = 2,        // a unit's module, slot or block range
    kCheckTmem = 3,        // tensor-memory column range of a drained chunk
    kCheckSlotStore = 4,   // where a drained chunk goes in its slot
    kCheckFirstTask = 5,   // a planned first task
    kCheckTask = 6,        // a task from a module's cursor
    kCheckFetch = 7,       // partial rows fetched into a warp's stage
    kCheckChunkSum = 8,    // chunk-sum scratch of the two-level finish
    kCheckStage = 9,       // pipeline stage index
    kCheckEmpty = 10,      // the range of slots a launch empties
};

#ifdef EGERIA_CHECKED
constexpr bool kCheckedBuild = true;
#else
constexpr bool kCheckedBuild = false;
#endif

// status[0] status word, [1] code of the first failed check, [2..3] the offending value, [4] block, [5] thread
__device__ __forceinline__ bool eg_check(bool ok, int32_t *status, int32_t code, long long value) {
#ifdef EGERIA_CHECKED
    if (!ok) {
        if (atomicCAS(status + 1, 0, code) == 0) {
            status[2] = (int32_t)(value & 0xffffffffll);
            status[3] = (int32_t)(value >> 32);
            status[4] = (int32_t)blockIdx.x;
            status[5] = (int32_t)threadIdx.x;
        }
        atomicMax(status, kStatusCheck);
    }
    return ok;
#else
    (void)ok;
    (void)status;
    (void)code;
    (void)value;
    return true;
#endif
}

}  // namespace egeria
