// Self-test of the kernels' failure path.  Every wait in the library's kernels is bounded: a wait that runs out
// raises a CTA-wide flag, the other waiters leave at their next poll, all roles meet at the common teardown (which
// frees tensor memory), and PSA_ERR_TIMEOUT reaches the host through the device status word.  In a correct run no
// wait ever expires, so this file holds a miniature kernel with the same skeleton whose barrier nobody completes:
// the expiry path then runs on purpose, with a limit of microseconds instead of seconds.  Nothing traps, nothing
// spins without a bound, and the context stays usable.
#include "psa_internal.h"
#include "sm100.cuh"

namespace psa {

namespace {

__global__ void __launch_bounds__(128, 1) wait_expiry_kernel(DeviceCounters* dc, unsigned long long limit_ns) {
    __shared__ uint64_t never_bar;       // initialised for one arrival that is never made
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_flag;
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(&never_bar, 1);
        fence_mbar_init();
    }
    if (warp == 1) { tmem_alloc(&tmem_base_s, 32); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;
    volatile int* abortp = &abort_flag;
    // warp 0 gives up after `limit_ns`; the other warps would wait sixteen times longer and must leave through the
    // flag instead (they check it every 64 polls)
    const bool ok = mbar_wait(&never_bar, 0, abortp, warp == 0 ? limit_ns : 16 * limit_ns);
    // roles stay uniform after a failed wait: the vote every production role takes before acting on `ok`
    const bool all_ok = named_bar_all(ok, 1, 128);
    if (all_ok && threadIdx.x == 0) atomicAdd(&dc->proj_macs, 1ull);   // unreachable unless the wait succeeded
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag) atomicExch(&dc->status, (int)PSA_ERR_TIMEOUT);
    if (warp == 1) tmem_dealloc(tmem, 32);
}

}  // namespace

cudaError_t launch_wait_expiry(DeviceCounters* dc, unsigned limit_us, cudaStream_t stream) {
    wait_expiry_kernel<<<1, 128, 0, stream>>>(dc, 1000ull * limit_us);
    return cudaGetLastError();
}

}  // namespace psa
