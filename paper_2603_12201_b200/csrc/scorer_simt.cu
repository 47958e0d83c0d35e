// Plain CUDA-core indexer scorer: one thread per (query row, key) pair.
// I[t,s] = sum_h w[t,h] * max(q[t,h,:] . k[s,:], 0)  (Sec. 2.1). Not a fast path: it exists
// as a debugging aid (IDXC_FLAG_SIMT_SCORER) to separate tensor-core descriptor problems
// from everything else. fp32 accumulation in head-then-dimension order.
#include <cuda_bf16.h>
#include <cuda_fp8.h>

#include "kernels.h"

namespace idxc {
namespace {

template <bool FP8>
__device__ __forceinline__ float load_elem(const void* base, int64_t idx) {
    if constexpr (FP8) {
        __nv_fp8_e4m3 v;
        v.__x = static_cast<const unsigned char*>(base)[idx];
        return static_cast<float>(v);
    } else {
        return __bfloat162float(static_cast<const __nv_bfloat16*>(base)[idx]);
    }
}

template <bool FP8>
__global__ void __launch_bounds__(128)
score_simt_kernel(ScoreArgs a) {
    const int64_t r = blockIdx.y;
    const int64_t s = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    int64_t n_keys, k_row0;
    if (a.lens) {
        n_keys = a.lens[r];
        k_row0 = a.k_offsets[r];
    } else {
        n_keys = a.q_begin + r + 1;
        k_row0 = 0;
    }
    if (s >= n_keys || s >= a.ld) return;
    const int64_t krow = k_row0 + s;
    float I = 0.f;
    for (int h = 0; h < a.H; ++h) {
        float x = 0.f;
        const int64_t qb = (r * a.H + h) * a.d;
        for (int i = 0; i < a.d; ++i) x = fmaf(load_elem<FP8>(a.q, qb + i), load_elem<FP8>(a.k, krow * a.d + i), x);
        I = fmaf(fmaxf(x, 0.f), a.w[r * a.H + h], I);
    }
    if constexpr (FP8) I *= a.q_scale[r] * a.k_scale[krow];
    a.scores[r * a.ld + s] = I;
}

// Causal mask for callers that read whole rows (IDXC_FLAG_FILL_MASKED): row r of `scores` gets -inf in columns
// q_begin + r + 1 .. n_cols - 1. One CTA per row, 4-byte stores up to the next 16-byte boundary, then 16-byte stores.
__global__ void __launch_bounds__(256)
fill_masked_kernel(float* __restrict__ scores, int64_t ld, int64_t q_begin, int64_t n_cols) {
    const int64_t r = blockIdx.x;
    float* row = scores + r * ld;
    const int64_t c0 = q_begin + r + 1;
    if (c0 >= n_cols) return;
    const int64_t a0 = (c0 + 3) & ~int64_t(3);                 // rows start 16-byte aligned and ld is a multiple of 4
    const int64_t a1 = n_cols & ~int64_t(3);
    const float ninf = -INFINITY;
    if (a0 >= a1) {
        for (int64_t c = c0 + threadIdx.x; c < n_cols; c += blockDim.x) row[c] = ninf;
        return;
    }
    for (int64_t c = c0 + threadIdx.x; c < a0; c += blockDim.x) row[c] = ninf;
    const float4 v = make_float4(ninf, ninf, ninf, ninf);
    for (int64_t c = a0 + 4 * static_cast<int64_t>(threadIdx.x); c < a1; c += 4 * static_cast<int64_t>(blockDim.x))
        *reinterpret_cast<float4*>(row + c) = v;
    for (int64_t c = a1 + threadIdx.x; c < n_cols; c += blockDim.x) row[c] = ninf;
}

}  // namespace

cudaError_t launch_fill_masked(float* scores, int64_t ld, int64_t q_begin, int64_t n_rows, int64_t n_cols, cudaStream_t stream) {
    for (int64_t r0 = 0; r0 < n_rows; r0 += (int64_t(1) << 30)) {
        const int64_t nr = n_rows - r0 < (int64_t(1) << 30) ? n_rows - r0 : (int64_t(1) << 30);
        fill_masked_kernel<<<static_cast<unsigned>(nr), 256, 0, stream>>>(scores + r0 * ld, ld, q_begin + r0, n_cols);
        if (cudaError_t e = cudaGetLastError(); e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t preload_score_simt() {
    cudaFuncAttributes fa;
    if (cudaError_t e = cudaFuncGetAttributes(&fa, reinterpret_cast<const void*>(score_simt_kernel<false>)); e != cudaSuccess) return e;
    return cudaFuncGetAttributes(&fa, reinterpret_cast<const void*>(score_simt_kernel<true>));
}

cudaError_t launch_score_simt(const ScoreArgs& a, cudaStream_t stream) {
    if (a.n_rows <= 0) return cudaSuccess;
    const int64_t max_keys = a.lens ? a.max_len : a.q_begin + a.n_rows;
    if (max_keys <= 0) return cudaSuccess;
    // grid.y is limited to 65535 rows per launch
    for (int64_t r0 = 0; r0 < a.n_rows; r0 += 65535) {
        ScoreArgs b = a;
        const int64_t nr = a.n_rows - r0 < 65535 ? a.n_rows - r0 : 65535;
        b.q = static_cast<const char*>(a.q) + r0 * a.H * a.d * (a.fp8 ? 1 : 2);
        b.w = a.w + r0 * a.H;
        if (a.q_scale) b.q_scale = a.q_scale + r0;
        if (a.k_offsets) { b.k_offsets = a.k_offsets + r0; b.lens = a.lens + r0; }
        b.q_begin = a.q_begin + r0;
        b.n_rows = nr;
        b.scores = a.scores + r0 * a.ld;
        const int64_t mk = a.lens ? a.max_len : b.q_begin + nr;
        dim3 grid(static_cast<unsigned>((mk + 127) / 128), static_cast<unsigned>(nr));
        if (a.fp8) score_simt_kernel<true><<<grid, 128, 0, stream>>>(b);
        else score_simt_kernel<false><<<grid, 128, 0, stream>>>(b);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace idxc
