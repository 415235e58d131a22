// Self-test of the bounded device-side wait: one block waits, through the same routine and with the same limit
// as every pipeline wait of the library's kernels, on a barrier that nothing ever arrives at.  The wait runs out,
// raises the device timeout flag and the kernel returns in order: no copy is in flight, no tensor memory is held,
// the context stays usable.
#include "common.cuh"
#include "ptx.cuh"

namespace lrd {
namespace {

__global__ void __launch_bounds__(32, 1) wait_runs_out_kernel(unsigned int* timeout_flag) {
    __shared__ __align__(8) uint64_t never;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        ptx::mbar_init(ptx::smem_u32(&never), 1);
        ptx::fence_mbar_init();
    }
    __syncwarp();
    const ptx::AbortCtx ab{&abort_flag, timeout_flag};
    ptx::mbar_wait_uniform(ptx::smem_u32(&never), 0, ab);     // phase 0 never completes
}

}  // namespace

lrd_status_t selftest_wait_runs_out(cudaStream_t stream) {
    unsigned int* flag = device_timeout_flag();
    if (!flag) return LRD_ERR_CUDA;
    wait_runs_out_kernel<<<1, 32, 0, stream>>>(flag);
    count_launch();
    return cuda_ok(cudaGetLastError(), "launch of the wait self-test") ? LRD_OK : LRD_ERR_CUDA;
}

}  // namespace lrd
