// Self-test of the bounded device-side wait that every pipeline role of the tensor-core kernels uses.
//
// One small block initialises an mbarrier that nothing ever arrives on and waits on it through the same
// mbar_wait / mbar_wait_warp helpers as the kernels, with a short limit.  The wait runs out, the waiting
// thread records its code in the context's status word, the other warp sees the abort flag and leaves, and
// the kernel returns by itself: the path that reports HTS_ERR_TIMEOUT, exercised without any fault or hang.
#include "common.cuh"
#include "tc_ptx.cuh"

namespace hts {
using namespace tc;

namespace {

__global__ void __launch_bounds__(64)
wait_selftest_kernel(long long limit_ticks, int* status)
{
    __shared__ uint64_t never;
    __shared__ int abort_flag;
    volatile int* abortp = &abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&never, 1);
        abort_flag = 0;
        fence_barrier_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        mbar_wait(&never, 0, abortp, status, 90, limit_ticks);             // the wait that runs out
    } else if (threadIdx.x >= 32) {
        mbar_wait_warp(&never, 0, abortp, status, 91);                     // a second role: leaves on the abort flag
    }
    __syncthreads();
}

}  // namespace

hts_status launch_wait_selftest(long long limit_ticks, int* status, cudaStream_t s)
{
    wait_selftest_kernel<<<1, 64, 0, s>>>(limit_ticks, status);
    HTS_LAUNCH_CHECK("wait_selftest_kernel");
    return HTS_OK;
}

}  // namespace hts
