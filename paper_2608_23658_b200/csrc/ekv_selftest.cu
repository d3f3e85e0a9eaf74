// ekv_selftest_bounded_wait: exercises the error path of the kernels' bounded waits without a fault.
//
// Every wait inside the attention kernels (on a copy barrier, on another warp role) gives up after a
// time limit, latches EKV_ERR_TIMEOUT in the pool's status word and lets the kernel finish, so that the
// context stays usable.  In a healthy run that path never executes.  This call runs it on purpose and
// harmlessly: one warp waits, with the kernels' two wait routines one after the other (the one bounded by a clock,
// the one bounded by a number of polls), on a barrier that nothing ever arrives on.
#include "ekv_internal.h"
#include "ptx.cuh"

namespace ekv {

__global__ void bounded_wait_probe_kernel(unsigned *status, unsigned long long limit_ns, unsigned max_polls, unsigned long long *waited_ns) {
    __shared__ unsigned long long bar;
    __shared__ unsigned give_up_flag;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        mbar_fence_init();
        give_up_flag = 0u;
    }
    __syncthreads();
    const uint64_t t0 = global_timer_ns();
    // the wait bounded by a clock (decode, one-head prefill kernels) ...
    const bool completed = mbar_wait(b, 0, limit_ns);  // nobody arrives: returns false after limit_ns
    // ... and the one bounded by a number of polls (two-head prefill kernel): gives up and leaves its mark
    const bool completed2 = mbar_wait_polls(b, 0, smem_u32(&give_up_flag), max_polls);
    __syncthreads();
    if (threadIdx.x == 0) {
        if (!completed && !completed2 && give_up_flag == 2u) atomicOr(status, EKV_DEV_FLAG_TIMEOUT);
        if (waited_ns) *waited_ns = global_timer_ns() - t0;
    }
}

}  // namespace ekv

using namespace ekv;

extern "C" ekv_status_t ekv_selftest_bounded_wait(ekv_pool_t *pool, int32_t limit_us, uint64_t *waited_ns_device, void *stream) {
    ekv_status_t st = check_compute(pool, 0, "ekv_selftest_bounded_wait");
    if (st != EKV_OK) return st;
    if (limit_us < 1 || limit_us > 100000) {
        set_error("ekv_selftest_bounded_wait: limit_us %d outside [1, 100000]", limit_us);
        return EKV_ERR_INVALID;
    }
    // a failed poll sleeps about 1.5 us: limit_us microseconds are about limit_us * 2 / 3 polls
    bounded_wait_probe_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(pool->d_status, (unsigned long long)limit_us * 1000ull,
                                                                (unsigned)(limit_us * 2 / 3 + 1), (unsigned long long *)waited_ns_device);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "ekv_selftest_bounded_wait launch");
    return EKV_OK;
}
