// Self-test of the bounded-wait protocol every pipelined kernel of this library uses (mbarrier waits that give up after a
// time limit, raise the CTA's abort flag, store DM_ERR_TIMEOUT in the device status word, and let every role drain and
// return with its TMEM freed).  Nothing here faults or hangs: the wait is on a barrier that nothing ever arrives at, and it
// ends by its own time limit.
#include "dm_internal.h"
#include "tc_ptx.cuh"

namespace dm {
namespace {

using namespace tc;

// Warp 0 waits (time limit limit_ns) on a barrier nobody arrives at: it must give up, raise the abort flag and store the status.
// Warp 1 holds 32 TMEM columns and waits on a second barrier with the library's regular 2 s limit: it must leave early because
// of the abort flag, then free its TMEM.  out[0] = 1 if warp 0's wait returned "aborted", out[1] = 1 if warp 1's did,
// out[2] = nanoseconds warp 1 waited.
__global__ void __launch_bounds__(64, 1) wait_timeout_kernel(int *status, unsigned long long limit_ns, unsigned long long *out) {
    __shared__ uint64_t bars[2];
    __shared__ uint32_t tmem_base;
    __shared__ int abort_word;
    volatile int *abort_flag = &abort_word;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        mbar_init(&bars[0], 1);
        mbar_init(&bars[1], 1);
        abort_word = 0;
        mbar_fence_init();
    }
    if (warp == 1) tmem_alloc(&tmem_base, 32);
    fence_before();
    __syncthreads();
    fence_after();
    if (warp == 0) {
        const bool done = mbar_wait_limit(&bars[0], 0, abort_flag, status, limit_ns);
        if (lane == 0) out[0] = done ? 0ull : 1ull;
    } else {
        const uint64_t t0 = globaltimer_ns();
        const bool done = mbar_wait(&bars[1], 0, abort_flag, status);
        if (lane == 0) { out[1] = done ? 0ull : 1ull; out[2] = globaltimer_ns() - t0; }
    }
    fence_before();
    __syncthreads();
    if (warp == 1) {
        fence_after();
        tmem_dealloc(tmem_base, 32);
    }
}

}  // namespace

cudaError_t selftest_wait_timeout(unsigned long long limit_ns, unsigned long long *out, cudaStream_t s) {
    int *status = device_status_ptr();
    if (!status) return cudaErrorUnknown;
    wait_timeout_kernel<<<1, 64, 0, s>>>(status, limit_ns, out);
    count_launch();
    return cudaGetLastError();
}

}  // namespace dm
