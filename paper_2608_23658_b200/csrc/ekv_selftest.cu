// ekv_selftest_bounded_wait: exercises the error path of the kernels' bounded waits without a fault.
//
// Every wait inside the attention kernels (on a copy barrier, on another warp role) gives up after a
// time limit, latches EKV_ERR_TIMEOUT in the pool's status word and lets the kernel finish, so that the
// context stays usable.  In a healthy run that path never executes.  This call runs it on purpose and
// harmlessly: one CTA waits, with the same wait routine, on a barrier that nothing ever arrives on.
#include "ekv_internal.h"
#include "ptx.cuh"

namespace ekv {

__global__ void bounded_wait_probe_kernel(unsigned *status, unsigned long long limit_ns, unsigned long long *waited_ns) {
    __shared__ unsigned long long bar;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        mbar_fence_init();
    }
    __syncthreads();
    const uint64_t t0 = global_timer_ns();
    const bool completed = mbar_wait(b, 0, limit_ns);  // nobody arrives: returns false after limit_ns
    if (threadIdx.x == 0) {
        if (!completed) atomicOr(status, EKV_DEV_FLAG_TIMEOUT);
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
    bounded_wait_probe_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(pool->d_status, (unsigned long long)limit_us * 1000ull,
                                                                (unsigned long long *)waited_ns_device);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "ekv_selftest_bounded_wait launch");
    return EKV_OK;
}
