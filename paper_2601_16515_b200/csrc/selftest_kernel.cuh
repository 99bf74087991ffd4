// Diagnostic kernel behind salad_selftest_bounded_wait: one thread waits, with a 2 ms limit, on an
// mbarrier that nothing ever arrives on, and reports the expiry the way the compute kernels do
// (status word = SALAD_ERR_TIMEOUT).  It exercises the bounded wait and the status path without any
// fault: the kernel returns normally.
#pragma once
#include "ptx.cuh"

namespace salad {

__global__ void __launch_bounds__(32) bounded_wait_selftest_kernel(int32_t* __restrict__ status,
                                                                   unsigned long long* __restrict__ waited_ns) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        fence_mbar_init();
        const uint64_t t0 = global_timer_ns();
        const bool ok = mbar_wait(smem_u32(&bar), 0, &abort_flag, 2000000ull);
        if (waited_ns) *waited_ns = global_timer_ns() - t0;
        *status = ok ? 0 : SALAD_ERR_TIMEOUT;
    }
}

}  // namespace salad
