// Self-test of the failure path every kernel of the library shares: a bounded mbarrier wait that runs out.
// One warp initialises a barrier that expects one arrival, nobody ever arrives, and the warp waits on it with the
// library's own wait routine (both its polling and its parked form) under a limit of about a millisecond instead of about
// a second.  The wait must give up, raise HF_DEV_TIMEOUT_FLAG with the caller's `where` code and return false; the kernel
// then leaves in the ordinary way, so the context stays usable.  Nothing here can hang: the limit is a clock comparison.
#pragma once
#include "tc5_common.cuh"

constexpr long long SELFTEST_WAIT_CYCLES = 2000000LL;     // ~1 ms

__global__ void __launch_bounds__(32) k_selftest_wait(int* dev_status, int where, int* result) {
    using namespace tc5;
    __shared__ __align__(8) uint64_t bar_mem;
    __shared__ int abort_word;
    const uint32_t bar = smem_u32(&bar_mem);
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    __syncwarp();
    volatile int* abort_flag = &abort_word;
    bool a = true, b = true;
    if (threadIdx.x == 0) a = mbar_wait<true, SELFTEST_WAIT_CYCLES>(bar, 0, abort_flag, dev_status, where);   // runs out, raises the flag
    __syncwarp();
    if (threadIdx.x == 1) b = mbar_wait<false, SELFTEST_WAIT_CYCLES>(bar, 0, abort_flag, dev_status, where + 1);   // sees the abort word
    __syncwarp();
    if (threadIdx.x < 2) result[threadIdx.x] = threadIdx.x == 0 ? (int)a : (int)b;
}
