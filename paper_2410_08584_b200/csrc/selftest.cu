// Self-test of the bounded device waits.  Every wait inside the tensor-core kernels
// (on an mbarrier that a TMA copy, an async copy group or a tcgen05.commit completes)
// goes through ptx::mbar_wait, which gives up after a fixed number of polls, raises the
// CTA's abort flag and lets every role unwind to the common exit, where the flag becomes
// ZIPVL_DEV_TIMEOUT in the caller's status word.  Nothing in the library can make such a
// wait run out on purpose, so this file holds a kernel that can: one CTA whose warps wait,
// with a caller-chosen poll limit, on a barrier nobody ever arrives at, next to a second
// barrier that does complete.  It exercises the same wait, the same flag and the same
// exit path as the real kernels and touches no tensor memory.
#include "common.cuh"
#include "tc_ptx.cuh"

namespace zipvl {
namespace {

using namespace ptx;

__global__ void __launch_bounds__(128)
wait_timeout_kernel(uint32_t poll_limit, int32_t *__restrict__ progress, int32_t *status_word) {
    __shared__ uint64_t never, always;
    __shared__ int abort_flag_s;
    volatile int *abort_flag = &abort_flag_s;
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&never), 1);     // no thread arrives here
        mbar_init(smem_u32(&always), 1);
        abort_flag_s = 0;
        fence_barrier_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) mbar_arrive(smem_u32(&always));
    // warp 0 waits on the barrier that completes: must succeed whatever the limit
    // warps 1-3 wait on the one that never does: the first to exhaust its polls raises the
    // flag, the others see it at their next look and leave too
    bool ok;
    if (warp == 0) ok = mbar_wait(smem_u32(&always), 0, abort_flag, poll_limit);
    else ok = mbar_wait(smem_u32(&never), 0, abort_flag, poll_limit);
    if (progress && (threadIdx.x & 31) == 0) progress[warp] = ok ? 1 : 0;
    __syncthreads();                        // the common exit of every role
    if (threadIdx.x == 0 && *abort_flag) report(status_word, ZIPVL_DEV_TIMEOUT);
}

}  // namespace
}  // namespace zipvl

extern "C" zipvl_status zipvl_selftest_wait_timeout(int32_t poll_limit, int32_t *progress,
                                                    int32_t *status_word, void *stream) {
    using namespace zipvl;
    if (poll_limit < 1 || poll_limit > (1 << 20))
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_selftest_wait_timeout: poll_limit = %d not in [1, 2^20]",
                    poll_limit);
    if (!status_word) return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_selftest_wait_timeout: status_word is NULL");
    wait_timeout_kernel<<<1, 128, 0, (cudaStream_t)stream>>>((uint32_t)poll_limit, progress, status_word);
    count_launches(1);
    return check_launch("zipvl_selftest_wait_timeout");
}
