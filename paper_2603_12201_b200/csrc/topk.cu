// Row-wise top-k select (Sec. 3 "Notation": T_t = Top-k(I_t)).
//
// One CTA per row. The k-th largest score is found exactly by a radix select on
// order-preserving 32-bit keys (12 + 10 + 10 bits, most significant first) with
// shared-memory histograms; after the first digit only the few keys that fall in
// the threshold bucket are kept (in shared memory) for the remaining digits.
// The row is then swept once more in index order: every key above the threshold is
// taken, keys equal to it are taken lowest index first until k are found, and an
// ordered compaction (warp shuffles + block prefix sums) writes the indices in
// ascending order. The row is read from HBM once (histogram sweep) and twice more
// through L2.
#include "kernels.h"

namespace idxc {
namespace {

constexpr int TK_THREADS = 512;
constexpr int TK_WARPS = TK_THREADS / 32;
constexpr int TK_BINS1 = 4096;   // top 12 bits
constexpr int TK_BINS23 = 1024;  // next 10 and last 10 bits
constexpr int TK_CAP = 4096;     // candidate keys kept in shared memory

struct TopkSmem {
    uint32_t hist[TK_BINS1];
    uint32_t cand[TK_CAP];
    uint32_t warp_sums[2][TK_WARPS];
    uint32_t sel_bucket;
    uint32_t sel_above;
    uint32_t cand_count;
};

// Larger float <=> larger key; -0 and +0 share a key.
__device__ __forceinline__ uint32_t score_key(float x) {
    uint32_t u = __float_as_uint(x);
    if ((u << 1) == 0u) u = 0u;
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
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

// Calls f(key, index) for every element of the row, 128-bit loads where possible.
template <typename F>
__device__ __forceinline__ void for_each_key(const float* __restrict__ src, int n, F f) {
    const int nvec = n >> 2;
    const float4* src4 = reinterpret_cast<const float4*>(src);
    for (int v = threadIdx.x; v < nvec; v += TK_THREADS) {
        float4 x = __ldg(src4 + v);
        f(score_key(x.x), 4 * v);
        f(score_key(x.y), 4 * v + 1);
        f(score_key(x.z), 4 * v + 2);
        f(score_key(x.w), 4 * v + 3);
    }
    const int i = 4 * nvec + threadIdx.x;
    if (threadIdx.x < 4 && i < n) f(score_key(__ldg(src + i)), i);
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

__global__ void __launch_bounds__(TK_THREADS)
topk_rows_kernel(const float* __restrict__ scores, int64_t ld, int64_t n_rows, int64_t first_len, int64_t len_step,
                 const int32_t* __restrict__ lens, int k_top, int32_t* __restrict__ out) {
    __shared__ TopkSmem sm;
    int slot = 0;
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

        // ---- digit 1 (bits 31..20): histogram over the whole row
        __syncthreads();   // previous row's readers of sm are done
        zero_hist(sm, TK_BINS1);
        if (threadIdx.x == 0) sm.cand_count = 0u;
        __syncthreads();
        for_each_key(src, n, [&](uint32_t key, int) { atomicAdd(&sm.hist[key >> 20], 1u); });
        __syncthreads();
        uint32_t b1, above1;
        select_bucket<TK_BINS1>(sm, static_cast<uint32_t>(k_top), slot, b1, above1);
        const uint32_t c1 = sm.hist[b1];
        uint32_t need = static_cast<uint32_t>(k_top) - above1;   // rank inside bucket b1, 1-based
        uint32_t b2, above2, b3, above3;
        __syncthreads();   // everyone has read hist[b1]

        if (c1 <= static_cast<uint32_t>(TK_CAP)) {
            // ---- keep the threshold bucket's keys in shared memory; digits 2 and 3 on those only
            for_each_key(src, n, [&](uint32_t key, int) {
                if ((key >> 20) == b1) sm.cand[atomicAdd(&sm.cand_count, 1u)] = key;
            });
            zero_hist(sm, TK_BINS23);
            __syncthreads();
            for (uint32_t i = threadIdx.x; i < c1; i += TK_THREADS) atomicAdd(&sm.hist[(sm.cand[i] >> 10) & 1023u], 1u);
            __syncthreads();
            select_bucket<TK_BINS23>(sm, need, slot, b2, above2);
            need -= above2;
            zero_hist(sm, TK_BINS23);
            __syncthreads();
            for (uint32_t i = threadIdx.x; i < c1; i += TK_THREADS) {
                uint32_t key = sm.cand[i];
                if (((key >> 10) & 1023u) == b2) atomicAdd(&sm.hist[key & 1023u], 1u);
            }
            __syncthreads();
            select_bucket<TK_BINS23>(sm, need, slot, b3, above3);
            need -= above3;
        } else {
            // ---- crowded threshold bucket (many near-equal scores): digits 2 and 3 over the row
            zero_hist(sm, TK_BINS23);
            __syncthreads();
            for_each_key(src, n, [&](uint32_t key, int) {
                if ((key >> 20) == b1) atomicAdd(&sm.hist[(key >> 10) & 1023u], 1u);
            });
            __syncthreads();
            select_bucket<TK_BINS23>(sm, need, slot, b2, above2);
            need -= above2;
            zero_hist(sm, TK_BINS23);
            __syncthreads();
            const uint32_t p2 = (b1 << 10) | b2;
            for_each_key(src, n, [&](uint32_t key, int) {
                if ((key >> 10) == p2) atomicAdd(&sm.hist[key & 1023u], 1u);
            });
            __syncthreads();
            select_bucket<TK_BINS23>(sm, need, slot, b3, above3);
            need -= above3;
        }
        const uint32_t T = (b1 << 20) | (b2 << 10) | b3;   // key of the k-th largest score
        const uint32_t need_eq = need;                      // how many keys equal to T are taken (>= 1)
        const uint32_t n_gt = static_cast<uint32_t>(k_top) - need_eq;

        // ---- ordered emission
        uint32_t gt_base = 0, eq_base = 0;
        const int nvec = n >> 2;
        const float4* src4 = reinterpret_cast<const float4*>(src);
        for (int v0 = 0; 4 * v0 < n; v0 += TK_THREADS) {
            const int v = v0 + threadIdx.x;
            uint32_t key[4];
            bool valid[4] = {false, false, false, false};
            if (v < nvec) {
                float4 x = __ldg(src4 + v);
                key[0] = score_key(x.x); key[1] = score_key(x.y); key[2] = score_key(x.z); key[3] = score_key(x.w);
                valid[0] = valid[1] = valid[2] = valid[3] = true;
            } else if (v == nvec) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (4 * v + j < n) { key[j] = score_key(__ldg(src + 4 * v + j)); valid[j] = true; }
                }
            }
            uint32_t cg = 0, ce = 0;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (valid[j]) { cg += key[j] > T; ce += key[j] == T; }
            }
            uint32_t total;
            const uint32_t excl = block_excl_scan(cg | (ce << 16), sm, slot, total);
            uint32_t my_gt = gt_base + (excl & 0xFFFFu);
            uint32_t my_eq = eq_base + (excl >> 16);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (!valid[j]) continue;
                if (key[j] > T) {
                    out_row[my_gt + (my_eq < need_eq ? my_eq : need_eq)] = 4 * v + j;
                    ++my_gt;
                } else if (key[j] == T) {
                    if (my_eq < need_eq) out_row[my_gt + my_eq] = 4 * v + j;
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
    const int64_t max_grid = 1 << 20;
    const unsigned grid = static_cast<unsigned>(n_rows < max_grid ? n_rows : max_grid);
    topk_rows_kernel<<<grid, TK_THREADS, 0, stream>>>(scores, ld, n_rows, first_len, len_step, lens, k_top, out);
    return cudaGetLastError();
}

}  // namespace idxc
