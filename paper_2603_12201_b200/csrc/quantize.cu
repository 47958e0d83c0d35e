// Per-token FP8 quantiser with optional K-cache append: the step in front of the indexer (Sec. 2.1:
// the lightning indexer runs in FP8 arithmetic). For token r:
//     scale[r]   = max(max_i |x[r,i]|, 1e-12) / 448            (fp32, IEEE division)
//     code[r,i]  = e4m3(x[r,i] / scale[r])                     (round to nearest even, saturating)
// written at row dst_rows[r] of the outputs when dst_rows is given (appending freshly projected keys
// to a paged or contiguous indexer K cache), else at row r. HBM-bound: 2 bytes read and 1 byte written
// per element. Rows of up to 256 elements are handled by a group of row_elems/8 lanes of one warp
// (one 128-bit load per lane, shuffle max); longer rows by one 256-thread CTA that keeps the row in
// registers between the max and the conversion, so the input is read once.
#include <cuda_bf16.h>
#include <cuda_fp8.h>

#include "kernels.h"

namespace idxc {
namespace {

constexpr float kE4m3Max = 448.0f;

struct Vec8 {            // 8 bf16 values as loaded by one 128-bit load
    uint4 raw;
    __device__ __forceinline__ float get(int i) const {
        const uint32_t w = i < 2 ? raw.x : (i < 4 ? raw.y : (i < 6 ? raw.z : raw.w));
        return __uint_as_float((i & 1) ? (w & 0xFFFF0000u) : (w << 16));
    }
};

// x / scale, correctly rounded, from the correctly rounded reciprocal r of the row's scale: the product x * r is within
// two units of the quotient and one residual step (both FMAs exact in their product) lands on the nearest float. Checked
// against the IEEE division for EVERY pair of a bf16 maximum and a bf16 value not above it, both signs: the e4m3 codes
// agree everywhere (the floats differ only where x is so small that the residual underflows, all of which are code 0).
// Written with the residual's sign flipped so that a zero keeps its sign. A division costs about three times as many
// instructions, and with eight of them per 128-bit load the kernel was bound by its instruction issue, not by HBM.
__device__ __forceinline__ float div_by_scale(float x, float scale, float r) {
    const float q = x * r;
    const float e = __fmaf_rn(q, scale, -x);
    return __fmaf_rn(-e, r, q);
}

template <bool EXACT_DIV>
__device__ __forceinline__ uint2 quantize8_impl(const Vec8& v, float scale, float r) {
    uint32_t lo = 0, hi = 0;
#pragma unroll
    for (int p = 0; p < 4; ++p) {
        const float x0 = v.get(2 * p), x1 = v.get(2 * p + 1);
        const float2 y = EXACT_DIV ? make_float2(__fdiv_rn(x0, scale), __fdiv_rn(x1, scale))
                                   : make_float2(div_by_scale(x0, scale, r), div_by_scale(x1, scale, r));
        const uint32_t two = __nv_cvt_float2_to_fp8x2(y, __NV_SATFINITE, __NV_E4M3);   // .x in the low byte
        if (p < 2) lo |= two << (16 * p);
        else hi |= two << (16 * (p - 2));
    }
    return make_uint2(lo, hi);
}

__device__ __forceinline__ uint2 quantize8(const Vec8& v, float scale) {
    if (scale <= 3.0e38f) return quantize8_impl<false>(v, scale, __frcp_rn(scale));
    return quantize8_impl<true>(v, scale, 0.f);        // an infinite maximum: plain divisions (x / inf = 0)
}

// G lanes per token (G = row_elems / 8 in {8, 16, 32}); a CTA of 256 threads handles 4 * 256 / G tokens,
// every thread one 128-bit vector of four different tokens (four loads in flight).
template <int G>
__global__ void __launch_bounds__(256)
quantize_small_rows_kernel(const uint4* __restrict__ x, int64_t n_tokens, uint2* __restrict__ codes, float* __restrict__ scale,
                           const int64_t* __restrict__ dst_rows) {
    constexpr int TPC = 256 / G;                       // tokens per CTA and pass
    const int lane_in_group = threadIdx.x % G;
    const int64_t token0 = static_cast<int64_t>(blockIdx.x) * (4 * TPC) + threadIdx.x / G;
    Vec8 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int64_t token = token0 + u * TPC;
        v[u].raw = token < n_tokens ? __ldg(x + token * G + lane_in_group) : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int64_t token = token0 + u * TPC;
        float amax = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(v[u].get(i)));
#pragma unroll
        for (int o = G / 2; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, o));
        if (token >= n_tokens) continue;
        const float sc = __fdiv_rn(fmaxf(amax, 1e-12f), kE4m3Max);
        const int64_t dst = dst_rows ? dst_rows[token] : token;
        codes[dst * G + lane_in_group] = quantize8(v[u], sc);
        if (lane_in_group == 0) scale[dst] = sc;
    }
}

// One CTA per token; V = 128-bit vectors per thread (row_elems <= 256 * 8 * V).
template <int V>
__global__ void __launch_bounds__(256)
quantize_long_rows_kernel(const uint4* __restrict__ x, int64_t n_tokens, int vecs_per_row, uint2* __restrict__ codes,
                          float* __restrict__ scale, const int64_t* __restrict__ dst_rows) {
    __shared__ float warp_max[2][8];
    int par = 0;
    for (int64_t token = blockIdx.x; token < n_tokens; token += gridDim.x, par ^= 1) {
        Vec8 v[V];
        float amax = 0.f;
#pragma unroll
        for (int j = 0; j < V; ++j) {
            const int vi = j * 256 + threadIdx.x;
            v[j].raw = vi < vecs_per_row ? __ldg(x + token * vecs_per_row + vi) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
            for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(v[j].get(i)));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, o));
        if ((threadIdx.x & 31) == 0) warp_max[par][threadIdx.x >> 5] = amax;
        __syncthreads();                                  // the other buffer is free again after the next barrier
#pragma unroll
        for (int w = 0; w < 8; ++w) amax = fmaxf(amax, warp_max[par][w]);
        const float sc = __fdiv_rn(fmaxf(amax, 1e-12f), kE4m3Max);
        const int64_t dst = dst_rows ? dst_rows[token] : token;
#pragma unroll
        for (int j = 0; j < V; ++j) {
            const int vi = j * 256 + threadIdx.x;
            if (vi < vecs_per_row) codes[dst * vecs_per_row + vi] = quantize8(v[j], sc);
        }
        if (threadIdx.x == 0) scale[dst] = sc;
    }
}

}  // namespace

cudaError_t launch_quantize_e4m3(const void* x, int64_t n_tokens, int row_elems, void* codes, float* scale,
                                 const int64_t* dst_rows, cudaStream_t stream) {
    if (n_tokens <= 0) return cudaSuccess;
    const uint4* xv = static_cast<const uint4*>(x);
    uint2* cv = static_cast<uint2*>(codes);
    const int vecs = row_elems / 8;
    if (row_elems == 64 || row_elems == 128 || row_elems == 256) {
        const int64_t tokens_per_cta = 4 * (256 / vecs);
        const unsigned grid = static_cast<unsigned>((n_tokens + tokens_per_cta - 1) / tokens_per_cta);
        if (vecs == 8) quantize_small_rows_kernel<8><<<grid, 256, 0, stream>>>(xv, n_tokens, cv, scale, dst_rows);
        else if (vecs == 16) quantize_small_rows_kernel<16><<<grid, 256, 0, stream>>>(xv, n_tokens, cv, scale, dst_rows);
        else quantize_small_rows_kernel<32><<<grid, 256, 0, stream>>>(xv, n_tokens, cv, scale, dst_rows);
        return cudaGetLastError();
    }
    const unsigned grid = static_cast<unsigned>(n_tokens < (1 << 20) ? n_tokens : (1 << 20));
    const int v_needed = (vecs + 255) / 256;
    if (v_needed <= 1) quantize_long_rows_kernel<1><<<grid, 256, 0, stream>>>(xv, n_tokens, vecs, cv, scale, dst_rows);
    else if (v_needed <= 2) quantize_long_rows_kernel<2><<<grid, 256, 0, stream>>>(xv, n_tokens, vecs, cv, scale, dst_rows);
    else quantize_long_rows_kernel<4><<<grid, 256, 0, stream>>>(xv, n_tokens, vecs, cv, scale, dst_rows);
    return cudaGetLastError();
}

}  // namespace idxc
