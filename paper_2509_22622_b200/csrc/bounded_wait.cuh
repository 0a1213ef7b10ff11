// Bounded waits on mbarriers: no kernel of the library spins without a limit.
//
// A role that waits longer than the limit claims the status words of the aux
// block (first come, first served), records who it was and what it waited for,
// and raises the CTA's abort flag; every other wait of the CTA then returns false
// as well, the roles drain to the kernel's common exit, and the host finds the
// record with ll_cache_device_status.
#pragma once

#include "ll_internal.h"
#include "ptx.cuh"

namespace ll {

constexpr uint64_t kWaitLimitNs = 2000000000ull;    // 2 s

struct WaitCtx {
    volatile int *abort_flag;     // in shared memory: 0 = running, 1 = a wait of this CTA ran out
    uint32_t *status;             // the aux block's status words
    int role;                     // who is waiting (the warp index)
};

// Returns false when the CTA is aborting.
__device__ __forceinline__ bool wait_slow(uint32_t bar, uint32_t parity, const WaitCtx &ctx, int bar_id, int iter,
                                          uint64_t limit_ns = kWaitLimitNs)
{
    using namespace ptx;
    const uint64_t t0 = globaltimer_ns();
    uint32_t spins = 0;
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++spins & 63u) == 0) {
            if (*ctx.abort_flag) return false;
            if (globaltimer_ns() - t0 > limit_ns) {
                *ctx.abort_flag = 1;
                if (atomicCAS(ctx.status, 0u, (uint32_t)kStatusTimeout) == 0u) {
                    ctx.status[1] = (uint32_t)ctx.role;
                    ctx.status[2] = (uint32_t)bar_id;
                    ctx.status[3] = (uint32_t)iter;
                    ctx.status[4] = blockIdx.x; ctx.status[5] = blockIdx.y; ctx.status[6] = blockIdx.z;
                    __threadfence();
                }
                return false;
            }
        }
    }
}

__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, const WaitCtx &ctx, int bar_id, int iter,
                                         uint64_t limit_ns = kWaitLimitNs)
{
    if (ptx::mbar_try_wait(bar, parity)) return true;
    return wait_slow(bar, parity, ctx, bar_id, iter, limit_ns);
}

}  // namespace ll
