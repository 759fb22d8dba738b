// Bounded mbarrier waits shared by the warp-specialised (TMA / tcgen05) kernels.
#pragma once
#include "molora.h"
#include "sm100_ptx.cuh"

namespace molora {

constexpr long long kTimeoutCycles = 2000000000LL;   // ~1 s at B200 clocks

// Bounded wait on an mbarrier phase.  Falls through once the CTA has aborted.
__device__ __forceinline__ void wait_bar(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t* dev_status,
                                         long long limit = kTimeoutCycles)
{
    if (ptx::mbar_try_wait(bar, parity)) return;
    if (*abort_flag) return;
    const long long t0 = clock64();
    while (!ptx::mbar_try_wait(bar, parity)) {
        if (*abort_flag) return;
        if (clock64() - t0 > limit) {
            *abort_flag = 1;
            if (dev_status != nullptr) atomicOr(dev_status, MOLORA_DEV_TIMEOUT);
            return;
        }
    }
}

// Same, for a barrier that CTAs of the cluster arrive on remotely (acquire at cluster scope).
__device__ __forceinline__ void wait_bar_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                                 uint32_t* dev_status)
{
    if (ptx::mbar_try_wait_cluster(bar, parity)) return;
    if (*abort_flag) return;
    const long long t0 = clock64();
    while (!ptx::mbar_try_wait_cluster(bar, parity)) {
        if (*abort_flag) return;
        if (clock64() - t0 > kTimeoutCycles) {
            *abort_flag = 1;
            if (dev_status != nullptr) atomicOr(dev_status, MOLORA_DEV_TIMEOUT);
            return;
        }
    }
}

}  // namespace molora
