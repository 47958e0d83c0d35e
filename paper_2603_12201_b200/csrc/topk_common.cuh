// Building blocks shared by the top-k kernels: order-preserving keys, block-wide prefix sums,
// histogram bucket selection, the 128-bit sweep over a warp's segment of a row, and the slow path
// for rows whose threshold bucket is crowded.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace idxc {
namespace topk {

constexpr int TK_BINS1 = 4096;   // top 12 key bits
constexpr int TK_BINS23 = 1024;  // 10-bit digits
constexpr int TK_UNROLL = 4;     // 128-bit loads in flight per lane in a sweep

template <int WARPS>
struct TopkSmem {
    uint32_t hist[TK_BINS1];
    uint32_t warp_sums[2][WARPS];
    uint32_t sel_bucket;
    uint32_t sel_above;
};

__device__ __forceinline__ uint32_t score_key(float x) {
    uint32_t u = __float_as_uint(x);
    if ((u << 1) == 0u) u = 0u;
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_to_score(uint32_t k) {
    return __uint_as_float((k & 0x80000000u) ? (k ^ 0x80000000u) : ~k);
}
// Top 12 bits of score_key(x).
__device__ __forceinline__ uint32_t score_digit1(float x) {
    const uint32_t d = __float_as_uint(x + 0.0f) >> 20;     // -0 + 0 = +0
    return (d & 0x800u) ? (d ^ 0xFFFu) : (d | 0x800u);
}

// Exclusive prefix sum of `v` over the block in thread order; `total` = block sum.
// `slot` alternates between calls so one barrier per call is enough.
template <int WARPS>
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, TopkSmem<WARPS>& sm, int& slot, uint32_t& total) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= o) inc += y;
    }
    if (lane == 31) sm.warp_sums[slot][wid] = inc;
    __syncthreads();
    uint32_t ws = lane < WARPS ? sm.warp_sums[slot][lane] : 0u;
    uint32_t winc = ws;
#pragma unroll
    for (int o = 1; o < WARPS; o <<= 1) {
        uint32_t y = __shfl_up_sync(0xFFFFFFFFu, winc, o);
        if (lane >= o) winc += y;
    }
    const uint32_t base = __shfl_sync(0xFFFFFFFFu, winc - ws, wid);
    total = __shfl_sync(0xFFFFFFFFu, winc, WARPS - 1);
    slot ^= 1;
    return base + inc - v;
}

// Calls f(score, index) for every element of the row (thread-strided), 128-bit loads.
template <int THREADS, typename F>
__device__ __forceinline__ void for_each_score(const float* __restrict__ src, int n, F f) {
    const int nvec = n >> 2;
    const float4* src4 = reinterpret_cast<const float4*>(src);
    for (int v = threadIdx.x; v < nvec; v += THREADS) {
        float4 x = __ldg(src4 + v);
        f(x.x, 4 * v);
        f(x.y, 4 * v + 1);
        f(x.z, 4 * v + 2);
        f(x.w, 4 * v + 3);
    }
    const int i = 4 * nvec + threadIdx.x;
    if (threadIdx.x < 4 && i < n) f(__ldg(src + i), i);
}

// Visits this warp's segment [seg_begin, seg_end) of a row of n scores in index order, one
// 128-score block per step (lane l holds the 4 scores at block_base + 4l). U steps are loaded
// before any is processed, so U 128-bit loads per lane are in flight. f(x, base) gets the lane's
// float4 and the index of its first score; scores at index >= n are padding (the row pitch is a
// multiple of 4, so the load itself stays inside the row) and must be ignored by f.
template <int U, typename F>
__device__ __forceinline__ void sweep_segment(const float* __restrict__ src, int n, int seg_begin, int seg_end, int lane, F f) {
    for (int cb = seg_begin; cb < seg_end; cb += 128 * U) {
        float4 x[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int base = cb + 128 * u + 4 * lane;
            x[u] = (cb + 128 * u < seg_end && base < n) ? __ldg(reinterpret_cast<const float4*>(src + base))
                                                        : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (cb + 128 * u < seg_end) f(x[u], cb + 128 * u + 4 * lane);
        }
    }
}

// hist[0..NB) holds counts per digit value. Finds the digit value `bucket` holding the
// need-th largest element (1-based): above < need <= above + hist[bucket], where `above`
// counts the elements in larger buckets. Requires sum(hist) >= need. Ends with a barrier.
template <int NB, int THREADS>
__device__ __forceinline__ void select_bucket(TopkSmem<THREADS / 32>& sm, uint32_t need, int& slot, uint32_t& bucket,
                                              uint32_t& above) {
    constexpr int PER = NB / THREADS;
    uint32_t loc[PER];
    uint32_t sum = 0;
    const int top = NB - static_cast<int>(threadIdx.x) * PER;       // one past my largest bin
    if constexpr (PER % 4 == 0) {
#pragma unroll
        for (int j4 = 0; j4 < PER / 4; ++j4) {
            const uint4 v = *reinterpret_cast<const uint4*>(&sm.hist[top - 4 * (j4 + 1)]);
            loc[4 * j4 + 0] = v.w; loc[4 * j4 + 1] = v.z; loc[4 * j4 + 2] = v.y; loc[4 * j4 + 3] = v.x;   // descending bins
            sum += v.x + v.y + v.z + v.w;
        }
    } else {
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            loc[j] = sm.hist[top - 1 - j];
            sum += loc[j];
        }
    }
    uint32_t total;
    uint32_t run = block_excl_scan(sum, sm, slot, total);
    if (run < need && need <= run + sum) {
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            if (need <= run + loc[j]) {
                sm.sel_bucket = static_cast<uint32_t>(top - 1 - j);
                sm.sel_above = run;
                break;
            }
            run += loc[j];
        }
    }
    __syncthreads();
    bucket = sm.sel_bucket;
    above = sm.sel_above;
}

template <int THREADS>
__device__ __forceinline__ void zero_hist(TopkSmem<THREADS / 32>& sm, int nb) {
    uint4* h4 = reinterpret_cast<uint4*>(sm.hist);
    for (int i = threadIdx.x; i < nb / 4; i += THREADS) h4[i] = make_uint4(0u, 0u, 0u, 0u);
}


// Digits 2 and 3 (10 + 10 bits) of a radix select over the low 20 key bits of c1 candidates that
// share the top 12 bits. need = rank of the wanted candidate among them (1-based, from the top).
// Returns the low 20 bits of its key, how many candidates equal to it are to be taken (need_eq >= 1)
// and how many there are (m_eq). Uses hist[0..1023]; every thread of the block must call it.
template <int THREADS>
__device__ __forceinline__ void candidate_select(TopkSmem<THREADS / 32>& sm, const uint32_t* cand_key, uint32_t c1, uint32_t need,
                                                 int& slot, uint32_t& t_low, uint32_t& need_eq, uint32_t& m_eq) {
    uint32_t b2, b3, above;
    zero_hist<THREADS>(sm, TK_BINS23);
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < c1; i += THREADS) atomicAdd(&sm.hist[cand_key[i] >> 10], 1u);
    __syncthreads();
    select_bucket<TK_BINS23, THREADS>(sm, need, slot, b2, above);
    need -= above;
    zero_hist<THREADS>(sm, TK_BINS23);
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < c1; i += THREADS) {
        const uint32_t c = cand_key[i];
        if ((c >> 10) == b2) atomicAdd(&sm.hist[c & 1023u], 1u);
    }
    __syncthreads();
    select_bucket<TK_BINS23, THREADS>(sm, need, slot, b3, above);
    need -= above;
    t_low = (b2 << 10) | b3;
    need_eq = need;
    m_eq = sm.hist[b3];
}

// Slow path of the select for a row whose threshold bucket b1 (top 12 key bits) is crowded or
// which is too long for the selection map: digits 2 and 3 are histogrammed over the whole row,
// then the row is swept in index order with block-wide prefix sums. need = rank inside bucket b1.
template <int THREADS>
__device__ __forceinline__ void slow_path(TopkSmem<THREADS / 32>& sm, const float* __restrict__ src, int n, uint32_t b1,
                                          uint32_t need, uint32_t k, int32_t* __restrict__ out_row, int& slot) {
    uint32_t b2, b3, above;
    __syncthreads();
    zero_hist<THREADS>(sm, TK_BINS23);
    __syncthreads();
    for_each_score<THREADS>(src, n, [&](float x, int) {
        const uint32_t key = score_key(x);
        if ((key >> 20) == b1) atomicAdd(&sm.hist[(key >> 10) & 1023u], 1u);
    });
    __syncthreads();
    select_bucket<TK_BINS23, THREADS>(sm, need, slot, b2, above);
    need -= above;
    zero_hist<THREADS>(sm, TK_BINS23);
    __syncthreads();
    const uint32_t p2 = (b1 << 10) | b2;
    for_each_score<THREADS>(src, n, [&](float x, int) {
        const uint32_t key = score_key(x);
        if ((key >> 10) == p2) atomicAdd(&sm.hist[key & 1023u], 1u);
    });
    __syncthreads();
    select_bucket<TK_BINS23, THREADS>(sm, need, slot, b3, above);
    need -= above;
    const uint32_t T = (p2 << 10) | b3;   // key of the k-th largest score
    const uint32_t need_eq = need;
    const uint32_t n_gt = k - need_eq;
    uint32_t gt_base = 0, eq_base = 0;
    for (int v0 = 0; 4 * v0 < n; v0 += THREADS) {
        const int base = 4 * (v0 + static_cast<int>(threadIdx.x));
        float x[4] = {0.f, 0.f, 0.f, 0.f};
        if (base < n) {
            const float4 v4 = __ldg(reinterpret_cast<const float4*>(src + base));
            x[0] = v4.x; x[1] = v4.y; x[2] = v4.z; x[3] = v4.w;
        }
        uint32_t key[4];
        uint32_t cg = 0, ce = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const bool valid = base + e < n;
            key[e] = valid ? score_key(x[e]) : 0u;
            if (valid) { cg += key[e] > T; ce += key[e] == T; }
        }
        uint32_t tot_g, tot_e;
        const uint32_t ex_g = block_excl_scan(cg, sm, slot, tot_g);
        const uint32_t ex_e = block_excl_scan(ce, sm, slot, tot_e);
        uint32_t my_gt = gt_base + ex_g;
        uint32_t my_eq = eq_base + ex_e;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (base + e >= n) continue;
            if (key[e] > T) {
                out_row[my_gt + (my_eq < need_eq ? my_eq : need_eq)] = base + e;
                ++my_gt;
            } else if (key[e] == T) {
                if (my_eq < need_eq) out_row[my_gt + my_eq] = base + e;
                ++my_eq;
            }
        }
        gt_base += tot_g;
        eq_base += tot_e;
        if (gt_base == n_gt && eq_base >= need_eq) break;   // all k found (uniform across the block)
    }
}

}  // namespace topk
}  // namespace idxc
