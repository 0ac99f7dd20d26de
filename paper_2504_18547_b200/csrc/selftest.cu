// Self-test of the bounded device-side wait: the mechanism every kernel of the library relies on
// to give up instead of hanging (a wait that exceeds its limit records VITINT_ERR_TIMEOUT in the
// device status word and the kernel returns).
#include "common.cuh"
#include "ptx.cuh"
#include "tile_ops.cuh"

namespace vitint {
namespace {

// One warp waits on an mbarrier phase that nothing ever completes, with the given cycle limit.
__global__ void __launch_bounds__(32) wait_timeout_kernel(long long limit_cycles, int* gave_up) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        ptx::mbar_init(ptx::smem_addr(&bar), 1);
        ptx::fence_mbar_init();
    }
    __syncwarp();
    const bool ok = mbar_wait(ptx::smem_addr(&bar), 0u, &abort_flag, limit_cycles);
    if (threadIdx.x == 0 && gave_up) *gave_up = ok ? 0 : 1;
}

}  // namespace
}  // namespace vitint

using namespace vitint;

extern "C" int vitint_selftest_wait_timeout(int64_t limit_cycles, int32_t* gave_up, void* stream) {
    if (limit_cycles <= 0 || limit_cycles > 2000000000ll) return VITINT_ERR_INVALID_ARG;
    wait_timeout_kernel<<<1, 32, 0, (cudaStream_t)stream>>>((long long)limit_cycles, gave_up);
    return cuda_status(cudaGetLastError());
}
