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

// ---------------------------------------------------------------------------------------------------------------
// Building blocks of the one-sweep select: a sample of the row fixes two pivot scores that bracket the k-th largest.

__device__ __forceinline__ void flag_selected(uint32_t* sel_map, uint32_t idx) {
    atomicOr(&sel_map[idx >> 4], 1u << (8u * ((idx >> 2) & 3u) + (idx & 3u)));
}
// 0xFFFFFFFF if a >= b else 0 (false for NaN)
__device__ __forceinline__ uint32_t ge_mask(float a, float b) {
    uint32_t r;
    asm("set.ge.u32.f32 %0, %1, %2;" : "=r"(r) : "f"(a), "f"(b));
    return r;
}
// z with P(N(0,1) > z) = p, to about 1e-3 (Abramowitz & Stegun 26.2.23), clamped to [-2.5, 2.5]
__device__ __forceinline__ float upper_quantile_z(float p) {
    const bool upper = p <= 0.5f;
    const float q = fminf(fmaxf(upper ? p : 1.f - p, 1e-6f), 0.5f);
    const float t2 = -2.f * __logf(q);
    const float t = t2 * rsqrtf(t2);
    const float zz = t - __fdividef(2.515517f + t * (0.802853f + t * 0.010328f), 1.f + t * (1.432788f + t * (0.189269f + t * 0.001308f)));
    return fminf(fmaxf(upper ? zz : -zz, -2.5f), 2.5f);
}
// bits 0-3, 8-11, 16-19, 24-27 of m (a map word's nibbles of one kind) as one 16-bit mask: bit j <-> position 16 w + j
__device__ __forceinline__ uint32_t squeeze_nibbles(uint32_t m) {
    return (m & 0xFu) | ((m >> 4) & 0xF0u) | ((m >> 8) & 0xF00u) | ((m >> 12) & 0xF000u);
}
// exclusive prefix sum of v over the lanes of a warp; total = the warp's sum
__device__ __forceinline__ uint32_t warp_excl_scan(uint32_t v, int lane, uint32_t& total) {
    uint32_t inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= o) inc += y;
    }
    total = __shfl_sync(0xFFFFFFFFu, inc, 31);
    return inc - v;
}

constexpr float TK_MARGIN_SIGMAS = 3.5f;          // half-width of the bracket in standard deviations of the sampled rank

struct SampleSmem {
    float part_sum[32], part_sq[32];
    uint32_t part_cnt[32];
};

// What the sample yields. Scores map monotonically to bins floor(x * scale + offset); lo_x and hi_x are the pivot scores
// (x >= hi_x: certainly among the k largest; lo_x <= x < hi_x: candidate; below lo_x: certainly not), either may be
// infinite. [y_lo, y_hi) is the band in bin units, for the finer bins the candidates are sorted into.
struct Pivots {
    float scale, offset, lo_x, hi_x, y_lo, fscale;
    bool usable;
    template <int BINS>
    __device__ __forceinline__ uint32_t fine_bin(float x) const {
        const int b = __float2int_rd((__fmaf_rn(x, scale, offset) - y_lo) * fscale);
        return static_cast<uint32_t>(min(max(b, 0), BINS - 1));
    }
};

// Samples the row (n scores at src, n > k_top): every warp of the block reads S blocks of 128 scores spread evenly over
// its share n / WARPS of the row (2048 scores per 32768 of the row over the whole block, at least U blocks per warp; the
// whole row when it is short), the block computes their mean and spread, histograms them in BINS monotone bins laid
// around where the k-th largest score should lie, and takes as pivots the bin edges next to the sample's scores of rank
// r -+ (TK_MARGIN_SIGMAS standard deviations of that rank under sampling without replacement), r = k * sample / n.
// Every thread of the block must call it; it uses sm.hist[0..BINS) and ends after a barrier. A block that calls it
// with the same row gets the same pivots whatever its place in a cluster. usable = false: the sample is constant or not
// finite (the caller selects on keys alone).
template <int THREADS, int BINS, typename SM, typename RS>
__device__ __forceinline__ Pivots sample_pivots(SM& sm, RS& rs, const float* __restrict__ src, int n, int k_top, int& slot) {
    constexpr int WARPS = THREADS / 32;
    constexpr int U = TK_UNROLL;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int seg = (((n + WARPS - 1) / WARPS) + 127) & ~127;
    const int seg_begin = wid * seg < n ? wid * seg : n;
    const int seg_end = seg_begin + seg < n ? seg_begin + seg : n;
    const int seg_blocks = seg >> 7;
    int S = (16 * ((n + 32767) >> 15) + WARPS - 1) / WARPS;
    S = S < U ? U : S;
    S = S > seg_blocks ? seg_blocks : S;
    const int stride = (seg_blocks / S) << 7;
    // The lane's part of sample block j: four scores from index base on (base >= seg_end: none)
    auto sample_base = [&](int j) -> int { return j < S ? seg_begin + j * stride + 4 * lane : seg_end; };
    auto sample_load = [&](int base) -> float4 {
        return base < seg_end ? __ldg(reinterpret_cast<const float4*>(src + base)) : make_float4(0.f, 0.f, 0.f, 0.f);
    };
    // calls f(float4, index of its first score) for the lane's part of every sample block after the first U
    auto for_rest = [&](auto f) {
        for (int j0 = U; j0 < S; j0 += U) {
            float4 x[U];
#pragma unroll
            for (int u = 0; u < U; ++u) x[u] = sample_load(sample_base(j0 + u));
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int base = sample_base(j0 + u);
                if (base < seg_end) f(x[u], base);
            }
        }
    };
    // the first U blocks (all of the sample unless the row is longer than 32768 scores per 16 blocks of the block's
    // warps) stay in registers for both passes
    float4 x0[U];
    int base0[U];
#pragma unroll
    for (int u = 0; u < U; ++u) { base0[u] = sample_base(u); x0[u] = sample_load(base0[u]); }
    Pivots pv;
    // ---- mean and spread
    zero_hist<THREADS>(sm, BINS);
    {
        float s1 = 0.f, s2 = 0.f;
        uint32_t m = 0;
        auto add = [&](const float4& x, int base) {
            if (base + 3 < n) {                                   // all but the last load of a row
                s1 += (x.x + x.y) + (x.z + x.w);
                s2 = fmaf(x.x, x.x, fmaf(x.y, x.y, fmaf(x.z, x.z, fmaf(x.w, x.w, s2))));
                m += 4u;
            } else {
                const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (base + e < n) { s1 += xs[e]; s2 = fmaf(xs[e], xs[e], s2); ++m; }
            }
        };
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (base0[u] < seg_end) add(x0[u], base0[u]);
        for_rest(add);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            s1 += __shfl_xor_sync(0xFFFFFFFFu, s1, o);
            s2 += __shfl_xor_sync(0xFFFFFFFFu, s2, o);
            m += __shfl_xor_sync(0xFFFFFFFFu, m, o);
        }
        if (lane == 0) { rs.part_sum[wid] = s1; rs.part_sq[wid] = s2; rs.part_cnt[wid] = m; }
    }
    __syncthreads();
    uint32_t m_sample = 0;
    {
        float s1 = 0.f, s2 = 0.f;
#pragma unroll
        for (int w = 0; w < WARPS; ++w) { s1 += rs.part_sum[w]; s2 += rs.part_sq[w]; m_sample += rs.part_cnt[w]; }
        const float inv_m = __fdividef(1.f, static_cast<float>(m_sample));
        const float mean = s1 * inv_m;
        const float var = fmaxf(s2 * inv_m - mean * mean, 0.f);
        const float sd = var * rsqrtf(fmaxf(var, 1e-37f));
        // where the k-th largest of n draws of such a distribution is expected, in standard deviations from the mean
        // (a rough inverse normal distribution is enough: it only centres the bins)
        const float z = upper_quantile_z(__fdividef(static_cast<float>(k_top), static_cast<float>(n)));
        const float half = 1.5f * sd;                         // the bins span [centre - half, centre + half)
        pv.scale = __fdividef(0.5f * BINS, half);
        pv.offset = -(mean + z * sd - half) * pv.scale;
        // a constant sample, or one with infinities, gives no usable map
        pv.usable = sd > 0.f && fabsf(pv.scale) < 3.0e38f && fabsf(pv.offset) < 3.0e38f;
    }
    if (!pv.usable) return pv;                                // the same for every thread
    // ---- histogram of the sample
    {
        auto count = [&](const float4& x, int base) {
            const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if (base + e < n) {
                    const int b = __float2int_rd(__fmaf_rn(xs[e], pv.scale, pv.offset));     // NaN -> 0; saturates
                    atomicAdd(&sm.hist[min(max(b, 0), BINS - 1)], 1u);
                }
            }
        };
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (base0[u] < seg_end) count(x0[u], base0[u]);
        for_rest(count);
    }
    __syncthreads();
    // ---- rank of the k-th largest of the row inside the sample, and its standard deviation under sampling without replacement
    const float mf = static_cast<float>(m_sample), nf = static_cast<float>(n);
    const float p = __fdividef(static_cast<float>(k_top), nf);
    const float r = mf * p;
    const float var_r = fmaxf(mf * p * (1.f - p) * __fdividef(nf - mf, fmaxf(nf - 1.f, 1.f)), 0.f);
    const float sd_r = var_r * rsqrtf(fmaxf(var_r, 1e-37f));
    const bool whole = m_sample == static_cast<uint32_t>(n);          // the sample is the row: ranks are exact
    const float margin = whole ? 0.f : TK_MARGIN_SIGMAS * sd_r + 2.f;
    const int r_hi = whole ? k_top : static_cast<int>(floorf(r - margin));  // sample ranks below r_hi: certainly selected
    const int r_lo = whole ? k_top : static_cast<int>(ceilf(r + margin));   // sample ranks above r_lo: certainly not
    const bool has_hi = r_hi >= 1;
    const bool has_lo = r_lo <= static_cast<int>(m_sample);
    uint32_t hi_bin, lo_bin, ab_hi, ab_lo;
    select_two_buckets<BINS, THREADS>(sm, has_hi ? r_hi : 1, has_lo ? r_lo : m_sample, slot, hi_bin, ab_hi, lo_bin, ab_lo);
    // the pivots as scores: the upper edge of bin hi_bin and the lower edge of bin lo_bin (any bracket will do, so the
    // rounding of these divisions does not matter); an end bin has no edge on its outer side
    const float inv_scale = __fdividef(1.f, pv.scale);
    const bool open_lo = !has_lo || lo_bin == 0u, open_hi = !has_hi || hi_bin == BINS - 1;
    pv.lo_x = open_lo ? -INFINITY : (static_cast<float>(lo_bin) - pv.offset) * inv_scale;
    pv.hi_x = open_hi ? INFINITY : (static_cast<float>(hi_bin + 1u) - pv.offset) * inv_scale;
    pv.y_lo = open_lo ? 0.f : static_cast<float>(lo_bin);
    const float y_hi = open_hi ? static_cast<float>(BINS) : static_cast<float>(hi_bin + 1u);
    pv.fscale = __fdividef(static_cast<float>(BINS), y_hi - pv.y_lo);
    return pv;
}

// Flags of four consecutive scores: bit e (low nibble) = at or above the upper pivot, bit 4 + e = between the pivots.
__device__ __forceinline__ uint32_t flag4(const float4& v, float lo_x, float hi_x) {
    const float x[4] = {v.x, v.y, v.z, v.w};
    uint32_t sel = 0, ge_lo = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        sel |= ge_mask(x[e], hi_x) & (1u << e);
        ge_lo |= ge_mask(x[e], lo_x) & (16u << e);
    }
    return sel | (ge_lo & ~(sel << 4));
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
