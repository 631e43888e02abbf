// Self-test of the failure path: one CTA waits, with the library's own bounded wait, on an
// mbarrier that nobody ever arrives on.  The wait runs out after `limit_cycles`, the CTA
// records the time-out in the handle's status word exactly as the compute kernels do, and
// returns normally.  No TMA, no tensor memory, no MMA: nothing is in flight when it gives up.
#pragma once

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace optiml {

constexpr int kSelftestWaitSite = 7;          // "wait site" reported by this kernel
constexpr long long kSelftestMaxCycles = 2000000000ll;   // about a second: the longest wait a caller may ask for

__global__ void __launch_bounds__(32, 1) selftest_timeout_kernel(long long limit_cycles, int* __restrict__ status) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        ptx::mbar_init(&bar, 1);
        ptx::fence_mbar_init();
    }
    __syncwarp();
    ptx::griddep_wait();        // (no early trigger: whatever follows in the stream starts when this kernel is over)
    if (threadIdx.x == 0) {
        // phase 0 never completes: there is no arrival and no expected byte count
        if (!ptx::mbar_wait_limit(&bar, 0, limit_cycles)) report_timeout(status, kSelftestWaitSite);
    }
}

}  // namespace optiml
