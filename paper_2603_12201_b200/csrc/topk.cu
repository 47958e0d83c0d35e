// Row-wise top-k select (Sec. 3 "Notation": T_t = Top-k(I_t)).
//
// One 512-thread CTA per row; each of its 16 warps owns one contiguous segment of the row.
// The k-th largest score is found exactly by a radix select on order-preserving 32-bit keys
// (12 + 10 + 10 bits, most significant first), in two sweeps over the row:
//   sweep 1 (the HBM read)  4096-bin shared-memory histogram of the top 12 key bits; a suffix
//                           scan finds the threshold bucket b1 holding the k-th largest score;
//   sweep 2 (L2)            scores above bucket b1 are certainly selected: their positions are
//                           marked in a shared-memory selection map (4 flag bits per byte, one
//                           byte per 128-bit load). Scores inside bucket b1 (typically < 1 % of the
//                           row) are kept with their index; digits 2 and 3 run on those only and
//                           give the exact threshold T, after which the kept scores above T, and
//                           the lowest-index ones equal to T until k are reached, are marked too.
//   emission                a block-wide prefix popcount over the map ranks every marked position,
//                           so the indices come out ascending, with a deterministic tie-break and no
//                           atomics on the output.
// Sweep 2 compares floats against the bucket bounds, which orders exactly like the keys
// (-0 == +0). If the threshold bucket holds more scores than the shared buffer (many near-equal
// scores, e.g. a constant row), or the row is longer than the selection map, the remaining digits
// are histogrammed over the whole row and the emission uses block-wide prefix sums over the row
// instead; same result, slower.
#include "kernels.h"

namespace idxc {
namespace {

constexpr int TK_THREADS = 512;
constexpr int TK_WARPS = TK_THREADS / 32;
constexpr int TK_BINS1 = 4096;   // top 12 bits
constexpr int TK_BINS23 = 1024;  // next 10 and last 10 bits
constexpr int TK_CAP = 4096;     // candidate keys kept in shared memory
constexpr int TK_UNROLL = 8;     // 128-bit loads in flight per lane in each sweep

struct TopkSmem {
    uint32_t hist[TK_BINS1];
    uint32_t warp_sums[2][TK_WARPS];
    uint32_t sel_bucket;
    uint32_t sel_above;
    uint32_t cand_count;
};
// Dynamic shared memory: cand_low[TK_CAP] (low 20 key bits of the kept scores), cand_idx[TK_CAP]
// (their positions), then the selection map (one byte per 4 scores).
constexpr int TK_DYN_FIXED_BYTES = 2 * TK_CAP * 4;
constexpr int TK_MAP_MAX_BYTES = 128 * 1024;      // rows up to 524288 scores use the map

// Larger float <=> larger key; -0 and +0 share a key.
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
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, TopkSmem& sm, int& slot, uint32_t& total) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= o) inc += y;
    }
    if (lane == 31) sm.warp_sums[slot][wid] = inc;
    __syncthreads();
    uint32_t ws = lane < TK_WARPS ? sm.warp_sums[slot][lane] : 0u;
    uint32_t winc = ws;
#pragma unroll
    for (int o = 1; o < TK_WARPS; o <<= 1) {
        uint32_t y = __shfl_up_sync(0xFFFFFFFFu, winc, o);
        if (lane >= o) winc += y;
    }
    uint32_t base = __shfl_sync(0xFFFFFFFFu, winc - ws, wid);
    total = __shfl_sync(0xFFFFFFFFu, winc, TK_WARPS - 1);
    slot ^= 1;
    return base + inc - v;
}

// Calls f(score, index) for every element of the row, 128-bit loads where possible.
template <typename F>
__device__ __forceinline__ void for_each_score(const float* __restrict__ src, int n, F f) {
    const int nvec = n >> 2;
    const float4* src4 = reinterpret_cast<const float4*>(src);
    for (int v = threadIdx.x; v < nvec; v += TK_THREADS) {
        float4 x = __ldg(src4 + v);
        f(x.x, 4 * v);
        f(x.y, 4 * v + 1);
        f(x.z, 4 * v + 2);
        f(x.w, 4 * v + 3);
    }
    const int i = 4 * nvec + threadIdx.x;
    if (threadIdx.x < 4 && i < n) f(__ldg(src + i), i);
}

// Visits this warp's segment [seg_begin, seg_end) of a row of n scores in index order, 128
// scores per step (lane l holds the 4 scores at step_base + 4l). U steps are loaded before any
// is processed, so U 128-bit loads per lane are in flight. f(x, base) gets the lane's float4
// and the index of its first score; scores at index >= n are padding (the row pitch is a
// multiple of 4, so the load itself stays inside the row) and must be ignored by f.
// The step condition is warp-uniform, so f may use warp collectives.
template <int U, typename F>
__device__ __forceinline__ void sweep_segment(const float* __restrict__ src, int n, int seg_begin, int seg_end, int lane, F f) {
    for (int cb = seg_begin; cb < seg_end; cb += 128 * U) {
        float4 x[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int base = cb + 128 * u + 4 * lane;
            x[u] = base < n ? __ldg(reinterpret_cast<const float4*>(src + base)) : make_float4(0.f, 0.f, 0.f, 0.f);
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
template <int NB>
__device__ __forceinline__ void select_bucket(TopkSmem& sm, uint32_t need, int& slot, uint32_t& bucket, uint32_t& above) {
    constexpr int PER = NB / TK_THREADS;
    uint32_t loc[PER];
    uint32_t sum = 0;
    const int top = NB - 1 - static_cast<int>(threadIdx.x) * PER;   // my largest bin
#pragma unroll
    for (int j = 0; j < PER; ++j) {
        loc[j] = sm.hist[top - j];
        sum += loc[j];
    }
    uint32_t total;
    uint32_t run = block_excl_scan(sum, sm, slot, total);
    if (run < need && need <= run + sum) {
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            if (need <= run + loc[j]) {
                sm.sel_bucket = static_cast<uint32_t>(top - j);
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

__device__ __forceinline__ void zero_hist(TopkSmem& sm, int nb) {
    for (int i = threadIdx.x; i < nb; i += TK_THREADS) sm.hist[i] = 0u;
}

__global__ void __launch_bounds__(TK_THREADS, 2)
topk_rows_kernel(const float* __restrict__ scores, int64_t ld, int64_t n_rows, int64_t first_len, int64_t len_step,
                 const int32_t* __restrict__ lens, int k_top, int32_t* __restrict__ out, int map_scores) {
    __shared__ TopkSmem sm;
    extern __shared__ uint32_t dyn[];
    uint32_t* cand_low = dyn;
    uint32_t* cand_idx = dyn + TK_CAP;
    uint32_t* sel_map = dyn + 2 * TK_CAP;                        // map_scores / 16 words
    uint8_t* sel_bytes = reinterpret_cast<uint8_t*>(sel_map);
    int slot = 0;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    // longest rows first when lengths grow with the row number
    for (int64_t blk = blockIdx.x; blk < n_rows; blk += gridDim.x) {
        const int64_t row = n_rows - 1 - blk;
        int64_t len = lens ? static_cast<int64_t>(lens[row]) : first_len + row * len_step;
        len = len < 0 ? 0 : (len > ld ? ld : len);
        const int n = static_cast<int>(len);
        int32_t* out_row = out + row * static_cast<int64_t>(k_top);
        if (n <= k_top) {   // fewer candidates than k: all of them, then padding
            for (int j = threadIdx.x; j < k_top; j += TK_THREADS) out_row[j] = j < n ? j : -1;
            continue;
        }
        const float* src = scores + row * ld;
        // this warp's segment: a multiple of 128 scores, so every lane loads aligned float4s
        const int seg = (((n + TK_WARPS - 1) / TK_WARPS) + 127) & ~127;
        const int seg_begin = wid * seg < n ? wid * seg : n;
        const int seg_end = seg_begin + seg < n ? seg_begin + seg : n;

        // ---- sweep 1: histogram of digit 1 (key bits 31..20) over the whole row
        __syncthreads();   // previous row's readers of sm are done
        zero_hist(sm, TK_BINS1);
        if (threadIdx.x == 0) sm.cand_count = 0u;
        __syncthreads();
        sweep_segment<TK_UNROLL>(src, n, seg_begin, seg_end, lane, [&](const float4& x, int base) {
            if (base + 3 < n) {
                atomicAdd(&sm.hist[score_digit1(x.x)], 1u);
                atomicAdd(&sm.hist[score_digit1(x.y)], 1u);
                atomicAdd(&sm.hist[score_digit1(x.z)], 1u);
                atomicAdd(&sm.hist[score_digit1(x.w)], 1u);
            } else {
                const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (base + e < n) atomicAdd(&sm.hist[score_digit1(xs[e])], 1u);
            }
        });
        __syncthreads();
        uint32_t b1, above1;
        select_bucket<TK_BINS1>(sm, static_cast<uint32_t>(k_top), slot, b1, above1);
        const uint32_t c1 = sm.hist[b1];
        uint32_t need = static_cast<uint32_t>(k_top) - above1;   // rank inside bucket b1, 1-based
        uint32_t b2, above2, b3, above3;
        __syncthreads();   // everyone has read hist[b1]

        if (c1 <= static_cast<uint32_t>(TK_CAP) && n <= map_scores) {
            // ---- sweep 2: mark the scores above bucket b1, keep the scores inside it
            const float lo = key_to_score(b1 << 20);                       // smallest score of bucket b1
            const bool has_above = b1 < TK_BINS1 - 1;
            const float hi = key_to_score(has_above ? ((b1 + 1) << 20) : 0xFFFFFFFFu);   // smallest score above it
            sweep_segment<TK_UNROLL>(src, n, seg_begin, seg_end, lane, [&](const float4& x4, int base) {
                const float x[4] = {x4.x, x4.y, x4.z, x4.w};
                uint32_t nib = 0;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (base + e >= n || !(x[e] >= lo)) continue;
                    if (has_above && x[e] >= hi) {
                        nib |= 1u << e;
                    } else {
                        const uint32_t slot_i = atomicAdd(&sm.cand_count, 1u);
                        if (slot_i < TK_CAP) {
                            cand_low[slot_i] = score_key(x[e]) & 0xFFFFFu;
                            cand_idx[slot_i] = static_cast<uint32_t>(base + e);
                        }
                    }
                }
                sel_bytes[base >> 2] = static_cast<uint8_t>(nib);      // lanes past the end of the row write 0
            });
            zero_hist(sm, TK_BINS23);
            __syncthreads();
            // ---- digits 2 and 3 on the kept scores
            for (uint32_t i = threadIdx.x; i < c1; i += TK_THREADS) atomicAdd(&sm.hist[(cand_low[i] >> 10) & 1023u], 1u);
            __syncthreads();
            select_bucket<TK_BINS23>(sm, need, slot, b2, above2);
            need -= above2;
            zero_hist(sm, TK_BINS23);
            __syncthreads();
            for (uint32_t i = threadIdx.x; i < c1; i += TK_THREADS) {
                const uint32_t c = cand_low[i];
                if ((c >> 10) == b2) atomicAdd(&sm.hist[c & 1023u], 1u);
            }
            __syncthreads();
            select_bucket<TK_BINS23>(sm, need, slot, b3, above3);
            need -= above3;
            const uint32_t t_low = (b2 << 10) | b3;              // low 20 key bits of the k-th largest score
            const uint32_t need_eq = need;                       // how many scores equal to it are taken (>= 1)
            const uint32_t m_eq = sm.hist[b3];                   // how many there are
            // ---- mark the kept scores that are selected
            for (uint32_t i = threadIdx.x; i < c1; i += TK_THREADS) {
                const uint32_t low = cand_low[i];
                bool take = low > t_low;
                if (low == t_low) {
                    take = true;
                    if (m_eq != need_eq) {                       // ties compete: the lowest positions win
                        uint32_t before = 0;
                        for (uint32_t i2 = 0; i2 < c1; ++i2) before += (cand_low[i2] == t_low) & (cand_idx[i2] < cand_idx[i]);
                        take = before < need_eq;
                    }
                }
                if (take) {
                    const uint32_t idx = cand_idx[i];
                    atomicOr(&sel_map[idx >> 4], 1u << (8u * ((idx >> 2) & 3u) + (idx & 3u)));
                }
            }
            __syncthreads();
            // ---- emission: rank the marked positions by a prefix popcount over the map
            const int words = (n + 15) >> 4;
            const int wpt = (words + TK_THREADS - 1) / TK_THREADS;
            const int w0 = static_cast<int>(threadIdx.x) * wpt < words ? static_cast<int>(threadIdx.x) * wpt : words;
            const int w1 = w0 + wpt < words ? w0 + wpt : words;
            uint32_t cnt = 0;
            for (int w = w0; w < w1; ++w) cnt += __popc(sel_map[w]);
            uint32_t total;
            uint32_t rank = block_excl_scan(cnt, sm, slot, total);
            for (int w = w0; w < w1; ++w) {
                uint32_t m = sel_map[w];
                while (m) {
                    const int b = __ffs(m) - 1;
                    m &= m - 1;
                    if (rank < static_cast<uint32_t>(k_top)) out_row[rank] = 16 * w + 4 * (b >> 3) + (b & 7);
                    ++rank;
                }
            }
            continue;
        }

        // ---- crowded threshold bucket: digits 2 and 3 over the row, block-scan emission
        zero_hist(sm, TK_BINS23);
        __syncthreads();
        for_each_score(src, n, [&](float x, int) {
            const uint32_t key = score_key(x);
            if ((key >> 20) == b1) atomicAdd(&sm.hist[(key >> 10) & 1023u], 1u);
        });
        __syncthreads();
        select_bucket<TK_BINS23>(sm, need, slot, b2, above2);
        need -= above2;
        zero_hist(sm, TK_BINS23);
        __syncthreads();
        const uint32_t p2 = (b1 << 10) | b2;
        for_each_score(src, n, [&](float x, int) {
            const uint32_t key = score_key(x);
            if ((key >> 10) == p2) atomicAdd(&sm.hist[key & 1023u], 1u);
        });
        __syncthreads();
        select_bucket<TK_BINS23>(sm, need, slot, b3, above3);
        need -= above3;
        const uint32_t T = (b1 << 20) | (b2 << 10) | b3;   // key of the k-th largest score
        const uint32_t need_eq = need;
        const uint32_t n_gt = static_cast<uint32_t>(k_top) - need_eq;
        uint32_t gt_base = 0, eq_base = 0;
        for (int v0 = 0; 4 * v0 < n; v0 += TK_THREADS) {
            const int base = 4 * (v0 + static_cast<int>(threadIdx.x));
            float x[4] = {0.f, 0.f, 0.f, 0.f};
            bool valid[4];
            if (base < n) {
                const float4 v4 = __ldg(reinterpret_cast<const float4*>(src + base));
                x[0] = v4.x; x[1] = v4.y; x[2] = v4.z; x[3] = v4.w;
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) valid[e] = base + e < n;
            uint32_t key[4];
            uint32_t cg = 0, ce = 0;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                key[e] = valid[e] ? score_key(x[e]) : 0u;
                if (valid[e]) { cg += key[e] > T; ce += key[e] == T; }
            }
            uint32_t total;
            const uint32_t excl = block_excl_scan(cg | (ce << 16), sm, slot, total);
            uint32_t my_gt = gt_base + (excl & 0xFFFFu);
            uint32_t my_eq = eq_base + (excl >> 16);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if (!valid[e]) continue;
                if (key[e] > T) {
                    out_row[my_gt + (my_eq < need_eq ? my_eq : need_eq)] = base + e;
                    ++my_gt;
                } else if (key[e] == T) {
                    if (my_eq < need_eq) out_row[my_gt + my_eq] = base + e;
                    ++my_eq;
                }
            }
            gt_base += total & 0xFFFFu;
            eq_base += total >> 16;
            if (gt_base == n_gt && eq_base >= need_eq) break;   // all k found (uniform across the block)
        }
    }
}

}  // namespace

cudaError_t launch_topk_rows(const float* scores, int64_t ld, int64_t n_rows, int64_t first_len, int64_t len_step,
                             const int32_t* lens, int k_top, int32_t* out, cudaStream_t stream) {
    if (n_rows <= 0) return cudaSuccess;
    // the selection map covers the longest row of this launch, rounded up to a whole sweep step
    int64_t longest = lens ? ld : first_len + (n_rows - 1) * len_step;
    if (longest > ld) longest = ld;
    if (longest < 0) longest = 0;
    int64_t map_bytes = (longest + 127) / 128 * 32;
    if (map_bytes > TK_MAP_MAX_BYTES) map_bytes = TK_MAP_MAX_BYTES;
    const int dyn_bytes = TK_DYN_FIXED_BYTES + static_cast<int>(map_bytes);
    static int attr_bytes = 0;
    if (dyn_bytes > attr_bytes) {
        cudaError_t e = cudaFuncSetAttribute(topk_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             TK_DYN_FIXED_BYTES + TK_MAP_MAX_BYTES);
        if (e != cudaSuccess) return e;
        attr_bytes = TK_DYN_FIXED_BYTES + TK_MAP_MAX_BYTES;
    }
    const int64_t max_grid = 1 << 20;
    const unsigned grid = static_cast<unsigned>(n_rows < max_grid ? n_rows : max_grid);
    topk_rows_kernel<<<grid, TK_THREADS, dyn_bytes, stream>>>(scores, ld, n_rows, first_len, len_step, lens, k_top, out,
                                                              static_cast<int>(map_bytes * 4));
    return cudaGetLastError();
}

}  // namespace idxc
