// Failure-path self-test: one warp waits on a barrier that nothing will ever signal, with a short
// limit, so that a test can watch the bounded wait give up - status word, abort flag, normal
// return - without hanging, trapping or faulting anything.
#include "pw_kernels.h"

namespace pw {
namespace {

__global__ void __launch_bounds__(32)
wait_selftest_kernel(DeviceStatus* status, long long limit, int* returned)
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        fence_barrier_init();
    }
    __syncwarp();
    const bool ok = mbar_wait(smem_u32(&bar), 0, &abort_flag, status, 990, limit);   // nobody arrives
    const bool any_ok = __any_sync(0xffffffffu, ok);
    if (threadIdx.x == 0) *returned = any_ok ? 2 : 1;       // 1: every lane's wait gave up and the kernel went on
}

}  // namespace

const char* launch_wait_selftest(DeviceStatus* status, long long limit, int* returned, cudaStream_t stream)
{
    wait_selftest_kernel<<<1, 32, 0, stream>>>(status, limit, returned);
    return cudaGetLastError() == cudaSuccess ? nullptr : "self-test launch failed";
}

}  // namespace pw
