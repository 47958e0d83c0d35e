// Building blocks shared by the top-k kernels: order-preserving keys, block-wide prefix sums,
// histogram bucket selection, the 128-bit sweep over a warp's segment of a row, and the slow path
// for rows whose threshold bucket is crowded.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace idxc {
namespace topk {

constexpr int TK_UNROLL = 4;     // 128-bit loads in flight per lane in a sweep

// The 32 key bits are consumed in three digits, most significant first: D1 bits (11 or 12), then LOW - 10 bits,
// then 10 bits, LOW = 32 - D1. BINS = the largest histogram a kernel needs (1 << D1).
template <int WARPS, int BINS>
struct TopkSmem {
    uint32_t hist[BINS];
    uint32_t warp_sums[2][WARPS];
    uint32_t sel_bucket;
    uint32_t sel_above;
    uint32_t sel_bucket2;
    uint32_t sel_above2;
};

__device__ __forceinline__ uint32_t score_key(float x) {
    uint32_t u = __float_as_uint(x);
    if ((u << 1) == 0u) u = 0u;
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_to_score(uint32_t k) {
    return __uint_as_float((k & 0x80000000u) ? (k ^ 0x80000000u) : ~k);
}
// Top D1 bits of score_key(x).
template <int D1>
__device__ __forceinline__ uint32_t score_digit1(float x) {
    constexpr uint32_t kSign = 1u << (D1 - 1), kAll = (1u << D1) - 1u;
    const uint32_t d = __float_as_uint(x + 0.0f) >> (32 - D1);     // -0 + 0 = +0
    return (d & kSign) ? (d ^ kAll) : (d | kSign);
}
// True when first-digit bucket b holds no finite score (infinities and NaN patterns sit in the lowest and highest
// buckets): float comparisons against such a bucket's bounds do not order like the keys.
template <int D1>
__device__ __forceinline__ bool bucket_is_finite(uint32_t b) {
    constexpr uint32_t kNonFinite = 1u << (D1 - 9);                 // buckets whose exponent field is all ones, per sign
    return b >= kNonFinite && b < (1u << D1) - kNonFinite;
}

// Exclusive prefix sum of `v` over the block in thread order; `total` = block sum.
// `slot` alternates between calls so one barrier per call is enough.
template <int WARPS, typename SM>
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, SM& sm, int& slot, uint32_t& total) {
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
template <int NB, int THREADS, typename SM>
__device__ __forceinline__ void select_bucket(SM& sm, uint32_t need, int& slot, uint32_t& bucket,
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
    uint32_t run = block_excl_scan<THREADS / 32>(sum, sm, slot, total);
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

// The same for two ranks at once (need_a <= need_b, both in 1..sum(hist)): one scan serves both.
template <int NB, int THREADS, typename SM>
__device__ __forceinline__ void select_two_buckets(SM& sm, uint32_t need_a, uint32_t need_b, int& slot, uint32_t& bucket_a,
                                                   uint32_t& above_a, uint32_t& bucket_b, uint32_t& above_b) {
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
    const uint32_t run0 = block_excl_scan<THREADS / 32>(sum, sm, slot, total);
    if (run0 < need_a && need_a <= run0 + sum) {
        uint32_t run = run0;
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            if (need_a <= run + loc[j]) { sm.sel_bucket = static_cast<uint32_t>(top - 1 - j); sm.sel_above = run; break; }
            run += loc[j];
        }
    }
    if (run0 < need_b && need_b <= run0 + sum) {
        uint32_t run = run0;
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            if (need_b <= run + loc[j]) { sm.sel_bucket2 = static_cast<uint32_t>(top - 1 - j); sm.sel_above2 = run; break; }
            run += loc[j];
        }
    }
    __syncthreads();
    bucket_a = sm.sel_bucket; above_a = sm.sel_above;
    bucket_b = sm.sel_bucket2; above_b = sm.sel_above2;
}

template <int THREADS, typename SM>
__device__ __forceinline__ void zero_hist(SM& sm, int nb) {
    uint4* h4 = reinterpret_cast<uint4*>(sm.hist);
    for (int i = threadIdx.x; i < nb / 4; i += THREADS) h4[i] = make_uint4(0u, 0u, 0u, 0u);
}


// Digits 2 and 3 (LOW - 10 and 10 bits) of a radix select over the low LOW key bits of c1 candidates that
// share the top 32 - LOW bits. need = rank of the wanted candidate among them (1-based, from the top).
// Returns the low LOW bits of its key, how many candidates equal to it are to be taken (need_eq >= 1)
// and how many there are (m_eq). Uses hist[0 .. 1 << (LOW - 10)); every thread of the block must call it.
template <int THREADS, int LOW, typename SM>
__device__ __forceinline__ void candidate_select(SM& sm, const uint32_t* cand_key, uint32_t c1, uint32_t need,
                                                 int& slot, uint32_t& t_low, uint32_t& need_eq, uint32_t& m_eq) {
    constexpr int BINS2 = 1 << (LOW - 10), BINS3 = 1024;
    uint32_t b2, b3, above;
    zero_hist<THREADS>(sm, BINS2);
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < c1; i += THREADS) atomicAdd(&sm.hist[(cand_key[i] >> 10) & (BINS2 - 1)], 1u);
    __syncthreads();
    select_bucket<BINS2, THREADS>(sm, need, slot, b2, above);
    need -= above;
    zero_hist<THREADS>(sm, BINS3);
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < c1; i += THREADS) {
        const uint32_t c = cand_key[i];
        if ((c >> 10) == b2) atomicAdd(&sm.hist[c & 1023u], 1u);
    }
    __syncthreads();
    select_bucket<BINS3, THREADS>(sm, need, slot, b3, above);
    need -= above;
    t_low = (b2 << 10) | b3;
    need_eq = need;
    m_eq = sm.hist[b3];
}

// Slow path of the select for a row whose threshold bucket b1 (top D1 key bits) is crowded, holds non-finite
// values, or which is too long for the selection map: digits 2 and 3 are histogrammed over the whole row,
// then the row is swept in index order with block-wide prefix sums. need = rank inside bucket b1. Everything
// here compares keys, so infinities order like any other score.
template <int THREADS, int D1, typename SM>
__device__ __forceinline__ void slow_path(SM& sm, const float* __restrict__ src, int n, uint32_t b1,
                                          uint32_t need, uint32_t k, int32_t* __restrict__ out_row, int& slot) {
    constexpr int LOW = 32 - D1, BINS2 = 1 << (LOW - 10), BINS3 = 1024;
    uint32_t b2, b3, above;
    __syncthreads();
    zero_hist<THREADS>(sm, BINS2);
    __syncthreads();
    for_each_score<THREADS>(src, n, [&](float x, int) {
        const uint32_t key = score_key(x);
        if ((key >> LOW) == b1) atomicAdd(&sm.hist[(key >> 10) & (BINS2 - 1)], 1u);
    });
    __syncthreads();
    select_bucket<BINS2, THREADS>(sm, need, slot, b2, above);
    need -= above;
    zero_hist<THREADS>(sm, BINS3);
    __syncthreads();
    const uint32_t p2 = (b1 << (LOW - 10)) | b2;
    for_each_score<THREADS>(src, n, [&](float x, int) {
        const uint32_t key = score_key(x);
        if ((key >> 10) == p2) atomicAdd(&sm.hist[key & 1023u], 1u);
    });
    __syncthreads();
    select_bucket<BINS3, THREADS>(sm, need, slot, b3, above);
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
        const uint32_t ex_g = block_excl_scan<THREADS / 32>(cg, sm, slot, tot_g);
        const uint32_t ex_e = block_excl_scan<THREADS / 32>(ce, sm, slot, tot_e);
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

// Radix select over a LIST of c full 32-bit keys (11 + 11 + 10 bits): finds the key T of the need-th largest entry
// (1-based), how many entries equal to T are to be taken (need_eq >= 1) and how many there are (m_eq).
// Uses hist[0..2047]; every thread of the block must call it.
template <int THREADS, typename SM>
__device__ __forceinline__ void list_select32(SM& sm, const uint32_t* key, uint32_t c, uint32_t need, int& slot,
                                              uint32_t& T, uint32_t& need_eq, uint32_t& m_eq) {
    uint32_t b, above;
    zero_hist<THREADS>(sm, 2048);
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < c; i += THREADS) atomicAdd(&sm.hist[key[i] >> 21], 1u);
    __syncthreads();
    select_bucket<2048, THREADS>(sm, need, slot, b, above);
    need -= above;
    uint32_t prefix = b;                                    // top 11 bits
    zero_hist<THREADS>(sm, 2048);
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < c; i += THREADS) {
        const uint32_t x = key[i];
        if ((x >> 21) == prefix) atomicAdd(&sm.hist[(x >> 10) & 2047u], 1u);
    }
    __syncthreads();
    select_bucket<2048, THREADS>(sm, need, slot, b, above);
    need -= above;
    prefix = (prefix << 11) | b;                            // top 22 bits
    zero_hist<THREADS>(sm, 1024);
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < c; i += THREADS) {
        const uint32_t x = key[i];
        if ((x >> 10) == prefix) atomicAdd(&sm.hist[x & 1023u], 1u);
    }
    __syncthreads();
    select_bucket<1024, THREADS>(sm, need, slot, b, above);
    need -= above;
    T = (prefix << 10) | b;
    need_eq = need;
    m_eq = sm.hist[b];
}

// The whole select on keys alone, three digits over the row (11 + 11 + 10 bits): the path of last resort for rows
// whose scores the faster paths cannot separate (constant rows, heavy ties, infinities, rows longer than the map).
template <int THREADS, typename SM>
__device__ __forceinline__ void slow_path_full(SM& sm, const float* __restrict__ src, int n, uint32_t k,
                                               int32_t* __restrict__ out_row, int& slot) {
    uint32_t b1, above;
    __syncthreads();
    zero_hist<THREADS>(sm, 2048);
    __syncthreads();
    for_each_score<THREADS>(src, n, [&](float x, int) { atomicAdd(&sm.hist[score_key(x) >> 21], 1u); });
    __syncthreads();
    select_bucket<2048, THREADS>(sm, k, slot, b1, above);
    slow_path<THREADS, 11>(sm, src, n, b1, k - above, k, out_row, slot);
}

}  // namespace topk
}  // namespace idxc
