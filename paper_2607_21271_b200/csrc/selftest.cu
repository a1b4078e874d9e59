// Self-test of the error path every tensor-core kernel of this library shares: a bounded mbarrier wait that runs out
// must end the kernel normally and leave a code in the plan's device status word (EQL_ERR_DEVICE_TIMEOUT on the host),
// with the context intact.  The kernel below waits, through the very helper the other kernels use, on a barrier that
// nothing ever arrives on.  Nothing traps, faults or spins without a limit.
#include "eql_internal.h"
#include "ptx_sm100.cuh"

namespace eql {
namespace {

__global__ void __launch_bounds__(32, 1) expire_one_wait_kernel(int* status) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        ptx::mbar_init(&bar, 1);
        abort_flag = 0;
        ptx::fence_mbar_init();
    }
    __syncwarp();
    if (threadIdx.x == 0) ptx::mbar_wait(&bar, 0, &abort_flag, status, 901);   // no arrival will ever come
    __syncwarp();
}

}  // namespace
}  // namespace eql

extern "C" {

eql_status_t eqlinear_plan_selftest_expired_wait(eqlinear_plan_t plan, void* stream) {
    if (eql_status_t ps = eql_check_plan(plan); ps != EQL_OK) return ps;
    eql::expire_one_wait_kernel<<<1, 32, 0, (cudaStream_t)stream>>>((int*)(plan->ws + plan->lay.status));
    return cudaGetLastError() == cudaSuccess ? EQL_OK : EQL_ERR_CUDA;
}

eql_status_t eqlinear_plan_clear_device_status(eqlinear_plan_t plan, void* stream) {
    if (eql_status_t ps = eql_check_plan(plan); ps != EQL_OK) return ps;
    return cudaMemsetAsync(plan->ws + plan->lay.status, 0, sizeof(int), (cudaStream_t)stream) == cudaSuccess ? EQL_OK
                                                                                                              : EQL_ERR_CUDA;
}

}  // extern "C"
