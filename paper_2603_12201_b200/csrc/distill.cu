// Forward value of the multi-layer distillation loss of training-aware IndexCache (Eq. 1):
//     L_multi = sum_{j=0..m} 1/(m+1) sum_t KL( p_t^(l+j) || Softmax(I_t) )
// over the causal positions s <= t of every row, or (sparse-training form) over the row's selected top-k
// positions with p renormalised over them. One 256-thread CTA per row; the dense form reads the scores and every
// target exactly once, in one sweep. HBM-bound: 4 * (1 + n_targets) bytes per (t, s) pair. exp / log and the
// per-thread sums in fp32, block sums in fp64.
#include "../../include/idxc.h"
#include "kernels.h"

namespace idxc {
namespace {

constexpr int DK_THREADS = 256;
constexpr int DK_MAX_TARGETS = 16;

struct DistillTargets {
    const float* p[DK_MAX_TARGETS];
};

__device__ __forceinline__ double block_sum_f64(double v, double* sh) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
    __syncthreads();
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < DK_THREADS / 32; ++w) t += sh[w];
    return t;
}

// NT: targets handled by one dense sweep (1, 2 or 4: their sums live in registers); more targets take one sweep per
// group of NT, the scores of the later sweeps coming from the L2.
template <int NT>
__global__ void __launch_bounds__(DK_THREADS)
distill_kl_kernel(const float* __restrict__ scores, int64_t ld, int64_t rows, int64_t first_len, int64_t len_step,
                  DistillTargets tg, int n_targets, const int32_t* __restrict__ topk, int k_top, double* __restrict__ loss_out,
                  float* __restrict__ row_out) {
    __shared__ double sh[DK_THREADS / 32];
    __shared__ float sh_m[DK_THREADS / 32];
    for (int64_t r = blockIdx.x; r < rows; r += gridDim.x) {
        const float* I = scores + r * ld;
        const int32_t* T = topk ? topk + r * k_top : nullptr;
        int64_t n = first_len + r * len_step;
        n = n < 0 ? 0 : (n > ld ? ld : n);
        const int count = T ? k_top : static_cast<int>(n);
        double row_loss = 0.0;
        if (!T) {
            // ---- dense causal row, ONE sweep over the scores and all targets (128-bit loads). With lse = log sum exp(x):
            //   KL(p || softmax(x)) = sum p log p - sum p x + lse * sum p,
            // so a thread keeps the online (m, l) pair of the soft-max plus, per target, C = sum p log p,
            // D = sum p (x - m) against its own running maximum m (when m moves to m', D += (m - m') * S) and S = sum p;
            // the block then brings every thread to the row maximum and adds up. No second pass over the scores.
            const int nvec = static_cast<int>(n >> 2);
            const float4* I4 = reinterpret_cast<const float4*>(I);
            for (int j0 = 0; j0 < n_targets; j0 += NT) {
            const int nt = n_targets - j0 < NT ? n_targets - j0 : NT;     // targets of this sweep
            float m = -INFINITY, l = 0.f;
            float C[NT], D[NT], S[NT];
#pragma unroll
            for (int j = 0; j < NT; ++j) C[j] = D[j] = S[j] = 0.f;
            auto raise = [&](float x) {                    // the running maximum moves up to x
                l *= __expf(m - x);                        // exp(-inf) = 0 for the first element
                if (m > -INFINITY) {
#pragma unroll
                    for (int j = 0; j < NT; ++j)
                        if (j < nt) D[j] += (m - x) * S[j];
                }
                m = x;
            };
            auto push4 = [&](const float4& x, const float4* pv) {
                const float xm = fmaxf(fmaxf(x.x, x.y), fmaxf(x.z, x.w));
                if (xm > m) raise(xm);
                const float d0 = x.x - m, d1 = x.y - m, d2 = x.z - m, d3 = x.w - m;
                l += (__expf(d0) + __expf(d1)) + (__expf(d2) + __expf(d3));
#pragma unroll
                for (int j = 0; j < NT; ++j) {
                    if (j < nt) {
                        const float4 q = pv[j];
                        if (q.x > 0.f) { C[j] += q.x * __logf(q.x); D[j] += q.x * d0; S[j] += q.x; }
                        if (q.y > 0.f) { C[j] += q.y * __logf(q.y); D[j] += q.y * d1; S[j] += q.y; }
                        if (q.z > 0.f) { C[j] += q.z * __logf(q.z); D[j] += q.z * d2; S[j] += q.z; }
                        if (q.w > 0.f) { C[j] += q.w * __logf(q.w); D[j] += q.w * d3; S[j] += q.w; }
                    }
                }
            };
            for (int v = threadIdx.x; v < nvec; v += DK_THREADS) {
                float4 pv[NT];
#pragma unroll
                for (int j = 0; j < NT; ++j)
                    if (j < nt) pv[j] = __ldg(reinterpret_cast<const float4*>(tg.p[j0 + j] + r * ld) + v);
                push4(__ldg(I4 + v), pv);
            }
            for (int i = 4 * nvec + threadIdx.x; i < n; i += DK_THREADS) {       // at most 3 elements of the row
                const float x = __ldg(I + i);
                if (x > m) raise(x);
                const float d = x - m;
                l += __expf(d);
#pragma unroll
                for (int j = 0; j < NT; ++j) {
                    if (j < nt) {
                        const float q = __ldg(tg.p[j0 + j] + r * ld + i);
                        if (q > 0.f) { C[j] += q * __logf(q); D[j] += q * d; S[j] += q; }
                    }
                }
            }
            // row maximum, then every thread's sums relative to it
            float bm = m;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) bm = fmaxf(bm, __shfl_xor_sync(0xFFFFFFFFu, bm, o));
            __syncthreads();
            if ((threadIdx.x & 31) == 0) sh_m[threadIdx.x >> 5] = bm;
            __syncthreads();
#pragma unroll
            for (int w = 0; w < DK_THREADS / 32; ++w) bm = fmaxf(bm, sh_m[w]);
            const double se = block_sum_f64(l > 0.f ? static_cast<double>(l * __expf(m - bm)) : 0.0, sh);
            const double lse_rel = log(se);                                       // lse - bm
#pragma unroll
            for (int j = 0; j < NT; ++j) {
                if (j >= nt) break;                        // block-uniform
                // sum p log p - sum p (x - bm) + (lse - bm) * sum p
                const double dj = m > -INFINITY ? static_cast<double>(D[j]) + static_cast<double>(m - bm) * static_cast<double>(S[j]) : 0.0;
                const double part = static_cast<double>(C[j]) - dj + lse_rel * static_cast<double>(S[j]);
                row_loss += block_sum_f64(part, sh);
            }
            }
        } else {
            // ---- sparse-training form: the row's selected positions only
            float m = -INFINITY;
            for (int i = threadIdx.x; i < count; i += DK_THREADS) {
                const int s = T[i];
                if (s >= 0) m = fmaxf(m, __ldg(I + s));
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
            __syncthreads();
            if ((threadIdx.x & 31) == 0) sh_m[threadIdx.x >> 5] = m;
            __syncthreads();
#pragma unroll
            for (int w = 0; w < DK_THREADS / 32; ++w) m = fmaxf(m, sh_m[w]);
            double se = 0.0;
            for (int i = threadIdx.x; i < count; i += DK_THREADS) {
                const int s = T[i];
                if (s >= 0) se += static_cast<double>(__expf(__ldg(I + s) - m));
            }
            se = block_sum_f64(se, sh);
            const float lse = m + logf(static_cast<float>(se));
            for (int j = 0; j < n_targets; ++j) {
                const float* P = tg.p[j] + r * ld;
                double tot = 0.0;                      // renormalise the target over the selected positions
                for (int i = threadIdx.x; i < count; i += DK_THREADS) {
                    const int s = T[i];
                    if (s >= 0) tot += static_cast<double>(__ldg(P + s));
                }
                tot = block_sum_f64(tot, sh);
                const float norm = tot > 0.0 ? static_cast<float>(1.0 / tot) : 1.f;
                double acc = 0.0;
                for (int i = threadIdx.x; i < count; i += DK_THREADS) {
                    const int s = T[i];
                    if (s < 0) continue;
                    const float p = __ldg(P + s) * norm;
                    if (p > 0.f) acc += static_cast<double>(p) * static_cast<double>(logf(p) - (__ldg(I + s) - lse));
                }
                row_loss += block_sum_f64(acc, sh);
            }
        }
        row_loss /= n_targets;
        if (threadIdx.x == 0) {
            if (row_out) row_out[r] = static_cast<float>(row_loss);
            atomicAdd(loss_out, row_loss);
        }
    }
}

}  // namespace
}  // namespace idxc

using namespace idxc;

extern "C" idxc_status idxc_distill_kl(const float* scores, int64_t ld, int64_t rows, int64_t first_len, int64_t len_step,
                                       const float* const* targets, int n_targets, const int32_t* topk, int k_top,
                                       double* loss_out, float* row_loss_out, void* cuda_stream) {
    if (rows < 0 || ld < 0 || first_len < 0 || len_step < 0 || n_targets < 1 || n_targets > DK_MAX_TARGETS) return IDXC_ERR_INVALID_ARG;
    if (topk && (k_top < 1 || k_top > IDXC_MAX_K_TOP)) return IDXC_ERR_INVALID_ARG;
    if (!scores || !targets || !loss_out) return IDXC_ERR_INVALID_ARG;
    if (!topk && ((ld & 3) || (reinterpret_cast<uintptr_t>(scores) & 15))) return IDXC_ERR_INVALID_ARG;   // 128-bit row loads
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemsetAsync(loss_out, 0, sizeof(double), stream) != cudaSuccess) return IDXC_ERR_CUDA;
    if (rows == 0) return IDXC_OK;
    DistillTargets tg{};
    for (int j = 0; j < n_targets; ++j) {
        if (!targets[j] || (!topk && (reinterpret_cast<uintptr_t>(targets[j]) & 15))) return IDXC_ERR_INVALID_ARG;
        tg.p[j] = targets[j];
    }
    const unsigned grid = static_cast<unsigned>(rows < (1 << 20) ? rows : (1 << 20));
    auto launch = [&](auto kernel) {
        kernel<<<grid, DK_THREADS, 0, stream>>>(scores, ld, rows, first_len, len_step, tg, n_targets, topk, k_top, loss_out, row_loss_out);
    };
    if (n_targets <= 1) launch(distill_kl_kernel<1>);
    else if (n_targets <= 2) launch(distill_kl_kernel<2>);
    else launch(distill_kl_kernel<4>);
    return cudaGetLastError() == cudaSuccess ? IDXC_OK : IDXC_ERR_CUDA;
}
