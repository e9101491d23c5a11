// Self-test of the give-up path of the bounded waits.  See bpt_selftest_wait_timeout in include/bpt.h.
#include "bpt_internal.cuh"
#include "mma_tools.cuh"
#include "tc5_tools.cuh"

namespace bpt {
namespace {

// One thread waits, with a short limit, on an mbarrier that expects one arrival nobody makes: the wait
// is bounded by construction, so the kernel ends either way; it reports what the tensor-memory kernels
// report when one of their waits runs out.
__global__ void wait_timeout_kernel(int* status, long long limit_cycles, int arrive) {
    __shared__ uint64_t bar;
    const uint32_t bar_u = smem_u32(&bar);
    if (threadIdx.x == 0) {
        tc5::mbar_init(bar_u, 1);
        tc5::mbar_init_fence();
        if (arrive) tc5::mbar_arrive(bar_u);
        if (!tc5::mbar_wait(bar_u, 0, limit_cycles)) status[0] = (int)BPT_ERR_TIMEOUT;
    }
}

}  // namespace
}  // namespace bpt

extern "C" bpt_status bpt_selftest_wait_timeout(void* workspace, int64_t limit_cycles, int32_t arrive, void* cuda_stream) {
    if (!workspace || limit_cycles < 1 || limit_cycles > bpt::tc5::kWaitCycles) return BPT_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (cudaMemsetAsync(workspace, 0, 256, st) != cudaSuccess) return BPT_ERR_CUDA;
    bpt::wait_timeout_kernel<<<1, 32, 0, st>>>(static_cast<int*>(workspace), (long long)limit_cycles, arrive);
    return cudaGetLastError() == cudaSuccess ? BPT_OK : BPT_ERR_CUDA;
}
