// Self-test of the bounded device-side wait used by the tensor-core kernels (no paper counterpart).
//
// Every barrier wait in those kernels gives up after a time limit, records LPDT_ERR_TIMEOUT in the
// caller's status word and lets the kernel return, so that a lost arrival can never hang the GPU.  In
// the production kernels the limit is two seconds and is never reached.  The entry point below runs
// the same wait routine on a barrier that nothing ever arrives at, with a caller-chosen short limit, so
// that the expiry path itself can be exercised: the kernel returns after `limit_ns` and the status
// word holds LPDT_ERR_TIMEOUT.
#include "tc_common.cuh"

namespace lpdt {

__global__ void bounded_wait_probe_kernel(unsigned long long limit_ns, int32_t *dev_status, int32_t *returned) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        tc::mbar_init(tc::smem_u32(&bar), 1);
        tc::mbar_fence_init();
    }
    __syncthreads();
    // phase 0 of the barrier completes only after one arrival; nobody arrives
    const bool done = tc::mbar_wait(tc::smem_u32(&bar), 0, &abort_flag, dev_status, limit_ns);
    __syncthreads();
    if (threadIdx.x == 0 && returned) *returned = done ? 1 : 2;      // 2 = the wait gave up
}

}  // namespace lpdt

extern "C" lpdt_status lpdt_selftest_bounded_wait(uint64_t limit_ns, int32_t *dev_status, int32_t *returned,
                                                  void *stream) {
    LPDT_CHECK_ARG(dev_status != nullptr);
    LPDT_CHECK_ARG(limit_ns >= 1000 && limit_ns <= 50ull * 1000 * 1000);      // 1 us .. 50 ms
    ++lpdt::g_launch_count;
    lpdt::bounded_wait_probe_kernel<<<1, 64, 0, lpdt::as_stream(stream)>>>((unsigned long long)limit_ns, dev_status,
                                                                          returned);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}
