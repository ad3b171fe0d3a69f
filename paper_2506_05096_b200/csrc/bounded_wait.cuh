// Warp-uniform election and the bounded mbarrier wait shared by the tcgen05 kernels.
#pragma once

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace astraea {

constexpr uint64_t kWaitLimitNs = 1000000000ull; // bounded waits: one second

__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile("{\n\t.reg .pred px;\n\telect.sync _|px, 0xffffffff;\n\tselp.u32 %0, 1, 0, px;\n\t}" : "=r"(pred));
    return pred != 0;
}

// Bounded mbarrier wait.  Gives up after the limit, or at once when another wait of this CTA
// already gave up; the caller carries on (its results are void, the error word says so).
__device__ __forceinline__ void wait_bar(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *err_word,
                                         uint64_t limit_ns = kWaitLimitNs) {
    using namespace ptx;
    if (mbar_try_wait(bar, parity)) return;
    if (*abort_flag) return;
    const uint64_t t0 = globaltimer_ns();
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 255u) == 0) {
            if (*abort_flag) return;
            if (globaltimer_ns() - t0 > limit_ns) {
                *abort_flag = 1;
                atomicExch(err_word, kErrTimeout);
                return;
            }
        }
    }
}

}  // namespace astraea
