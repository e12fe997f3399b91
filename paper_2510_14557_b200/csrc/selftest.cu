// Self-test of the bounded device-side wait every GEMM kernel here is built on.
//
// One warp waits on an mbarrier that nothing ever arrives at, with a caller-chosen cycle
// limit; the wait must come back false and the kernel must report MXP_ERR_TIMEOUT through
// the status block and exit normally, leaving the context usable.  Nothing faults, traps or
// spins without bound: this is how the timeout path is exercised without breaking a GEMM.
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace mxp {
namespace {

__global__ void __launch_bounds__(32, 1) wait_selftest_kernel(StatusBlock* status, long long limit_cycles)
{
    __shared__ uint64_t bar;
    __shared__ uint32_t abort_flag;
    if (threadIdx.x == 0) {
        ptx::mbar_init(&bar, 1);
        abort_flag = 0u;
        ptx::fence_mbar_init();
    }
    __syncwarp();
    const bool ok = ptx::mbar_wait(&bar, 0, &abort_flag, limit_cycles);
    if (threadIdx.x == 0) {
        status->code = ok ? 0u : (uint32_t)MXP_ERR_TIMEOUT;
        status->where = 0x5E1Fu;
    }
}

}  // namespace

mxp_status launch_wait_selftest(void* workspace, int64_t limit_cycles, cudaStream_t stream)
{
    wait_selftest_kernel<<<1, 32, 0, stream>>>(static_cast<StatusBlock*>(workspace), (long long)limit_cycles);
    return cudaGetLastError() == cudaSuccess ? MXP_OK : MXP_ERR_CUDA;
}

}  // namespace mxp
