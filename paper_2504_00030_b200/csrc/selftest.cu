// Self-test of the bounded device-side wait that every tensor-core kernel of the library uses.
//
// The kernels never spin without a limit: a wait that does not end within its cycle budget sets
// SV_DEV_TIMEOUT in the caller's status word and the block drains.  In normal operation no wait
// ever runs out, so this entry point exists to exercise that path: one thread block waits, with
// a short budget, on an mbarrier that nothing arrives at, and must come back with the status bit
// set and the context intact.  Nothing faults, traps or hangs.
#include "tc_ptx.cuh"

namespace sv {

__global__ void __launch_bounds__(128)
wait_expiry_kernel(uint32_t *status, int32_t *result, long long limit_cycles)
{
    pdl_enter();
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const bool ok = bounded_wait(smem_u32(&bar), 0, &abort_flag, status, limit_cycles);
    // every thread gave up (on its own budget or on the block's abort flag); report the outcome
    const int any_ok = __syncthreads_or(ok ? 1 : 0);
    if (threadIdx.x == 0) *result = any_ok;
}

}  // namespace sv

extern "C" sv_status sv_selftest_wait_expiry(uint32_t *device_status, int32_t *device_result,
                                             int64_t limit_cycles, void *stream)
{
    if (device_status == nullptr || device_result == nullptr) return SV_EINVAL;
    if (limit_cycles < 1 || limit_cycles > 2000000000LL) return SV_EINVAL;     // at most about a second
    return sv::launch_kernel(true, sv::wait_expiry_kernel, 1, 128, 0, (cudaStream_t)stream, device_status, device_result,
                          (long long)limit_cycles);
}
