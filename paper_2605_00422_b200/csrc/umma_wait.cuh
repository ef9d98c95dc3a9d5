// Bounded waits on mbarriers for the tcgen05 kernels: every wait gives up after a fixed number of polls, records where
// in the workspace status words and raises the CTA's abort flag, so that a kernel whose producer never arrives ends by
// itself and the host can read what happened.
#pragma once

#include "umma_ptx.cuh"

namespace bwla {

using namespace ptx;

constexpr uint32_t kParkNs = 4000;          // longest a single poll of a barrier may park its thread
constexpr uint32_t kWaitLimit = 1u << 15;   // polls per wait before giving up (about a tenth of a second when nothing arrives)

__device__ __forceinline__ void give_up(uint32_t* status, volatile int* abort_flag, uint32_t where) {
    if (status) {
        atomicExch(status, 1u);
        status[1] = where;
        status[2] = blockIdx.x | (blockIdx.y << 16);
    }
    *abort_flag = 1;
}

__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    // Each poll may park the thread for up to kParkNs while the phase is open: a warp that spun on the barrier would
    // take issue slots from the expander warps that share its scheduler.
    // a phase that is already complete is seen by the non-blocking probe in a fraction of the time try_wait takes
    if (mbar_test_wait(bar, parity)) return true;
    for (uint32_t i = 0; i < kWaitLimit; ++i) {
        if (mbar_try_wait_parked(bar, parity, kParkNs)) return true;
        if (*abort_flag) return false;
    }
    return false;
}

// A whole warp waits on a barrier and leaves the call converged, as the .sync.aligned tcgen05 instructions that follow
// such a wait require (lanes that each ran their own polling loop may come out of it at different times, and a
// warp-wide tensor-memory store issued by part of a warp lands late): every lane polls, the warp goes on when all saw
// the phase complete.
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    if (__all_sync(0xFFFFFFFFu, mbar_test_wait(bar, parity))) return true;
    for (uint32_t i = 0; i < kWaitLimit; ++i) {
        const bool done = mbar_try_wait_parked(bar, parity, kParkNs);
        if (__all_sync(0xFFFFFFFFu, done)) return true;
        if (*abort_flag) return false;
    }
    return false;
}

}  // namespace bwla
