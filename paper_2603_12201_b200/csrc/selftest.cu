// Self-test of the failure-detection path: a wait that can never be satisfied must give up after its
// cycle budget, record a status code and let the kernel return normally (no trap, no hang).
#include "kernels.h"
#include "ptx_sm100.cuh"

namespace idxc {
namespace {

__global__ void __launch_bounds__(32)
selftest_bounded_wait_kernel(unsigned int* status, long long budget_cycles) {
    __shared__ uint64_t bar;
    __shared__ uint32_t abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);          // one arrival expected; nobody ever arrives
        abort_flag = 0u;
        fence_mbar_init();
    }
    __syncwarp();
    if (threadIdx.x == 0) {
        const bool ok = mbar_wait(smem_u32(&bar), 0u, &abort_flag, budget_cycles);
        if (!ok) {
            abort_flag = 1u;
            atomicCAS(status, 0u, static_cast<unsigned int>(DEV_TIMEOUT_SELFTEST));
        }
    }
}

}  // namespace

cudaError_t launch_selftest_bounded_wait(unsigned int* status, long long budget_cycles, cudaStream_t stream) {
    selftest_bounded_wait_kernel<<<1, 32, 0, stream>>>(status, budget_cycles);
    return cudaGetLastError();
}

}  // namespace idxc
