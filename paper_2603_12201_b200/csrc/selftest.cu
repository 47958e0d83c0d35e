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

// Measures how fast the prefill scorer's epilogue can read accumulators out of tensor memory, with nothing else
// running: the same CTA shape (one per SM, 8 reading warps, two per tensor-memory lane quarter) and the same loads
// (tcgen05.ld 16x256b.x4, eight per 128 x 256 accumulator and warp), `iters` accumulators per warp. The loaded words
// are folded into one register so that the loads cannot be dropped; `sink` only ever receives them if that fold
// equals a value no read-out produces in practice. Tensor memory is read as it stands (never written here).
__global__ void __launch_bounds__(320, 1)
selftest_tmem_readout_kernel(uint32_t iters, uint32_t* sink) {
    __shared__ uint32_t tmem_base_slot;
    const int warp = threadIdx.x >> 5;
    if (warp == 1) {
        tmem_alloc(smem_u32(&tmem_base_slot), 512);
        tmem_relinquish_alloc_permit();
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    tcgen05_fence_after_sync();
    const uint32_t tmem_base = tmem_base_slot;
    if (warp >= 2) {
        const int ew = warp - 2;
        const int quarter = warp & 3;            // the tensor-memory lane quarter this warp may read
        const int colhalf = ew >> 2;             // which 128 of an accumulator's 256 columns
        uint32_t fold = 0;
        for (uint32_t it = 0; it < iters; ++it) {
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                                   static_cast<uint32_t>((it & 1u) * 256 + colhalf * 128);
            uint32_t ra[16], rb[16];
            tmem_ld_16x256b_x4(taddr, ra);
            tmem_ld_wait(ra);
#pragma unroll
            for (int n = 0; n < 8; ++n) {        // n = lane half (16 lanes) * 4 + 32-column chunk, double-buffered like the epilogue
                uint32_t (&cur)[16] = (n & 1) ? rb : ra;
                uint32_t (&nxt)[16] = (n & 1) ? ra : rb;
                if (n + 1 < 8) tmem_ld_16x256b_x4(taddr + (static_cast<uint32_t>(((n + 1) / 4) * 16) << 16) + ((n + 1) % 4) * 32, nxt);
#pragma unroll
                for (int i = 0; i < 16; ++i) fold ^= cur[i];
                if (n + 1 < 8) tmem_ld_wait(nxt);
            }
        }
        if (fold == 0x9E3779B9u && iters == 0xFFFFFFFFu) *sink = fold;
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tcgen05_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
}

}  // namespace

cudaError_t launch_selftest_tmem_readout(uint32_t iters, uint32_t* sink, int sm_count, cudaStream_t stream) {
    selftest_tmem_readout_kernel<<<sm_count, 320, 0, stream>>>(iters, sink);
    return cudaGetLastError();
}

cudaError_t launch_selftest_bounded_wait(unsigned int* status, long long budget_cycles, cudaStream_t stream) {
    selftest_bounded_wait_kernel<<<1, 32, 0, stream>>>(status, budget_cycles);
    return cudaGetLastError();
}

}  // namespace idxc
