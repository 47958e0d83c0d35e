// Second half of the streaming top-k of the prefill indexer (Sec. 2.1: the per-query top-k of the index scores).
//
// The scorer in streaming mode (scorer_tc.cu) leaves, per query row t, a list of (score, key index) pairs: the scores
// of a strided sample of the row's key tiles that reach the row's threshold tau, and every later score that is not
// below tau. tau is a sample quantile chosen so that, with high probability, at least k_top scores of the row reach
// it. This kernel checks that for every row with its own exact count:
//   * the list did not overflow and at least min(k_top, t + 1) of its entries are >= tau: every score that was
//     dropped is < tau, so the row's k_top largest scores are all in the list, and their exact selection (largest
//     score first, lowest key index among equal scores: the same order as the ordinary select) is the row's answer;
//   * otherwise the row is flagged, and the caller computes it by the ordinary path (full scores, ordinary select).
// One CTA per block of rows_per_item rows (the scorer's work item), so that the CTA can also say whether any row of
// the block was flagged: the scorer's second run visits only flagged blocks.
//
// Selection: the list (a sample part and 128 short per-thread lists) is read from global memory once and its keys
// (order-preserving 32-bit images of the scores) packed into shared memory; histogram passes over the packed keys, with
// 2048 bins laid over [smallest, largest] and narrowed to the bin of the wanted rank, find that rank's key; the chosen
// key indices are set in a bitmap over the row's positions and read out in ascending order.
#include "kernels.h"
#include "topk_common.cuh"

namespace idxc {
using namespace topk;
namespace {

constexpr int FS_THREADS = 256;
constexpr int FS_WARPS = FS_THREADS / 32;
constexpr int FS_EQ_MAX = 256;                           // entries equal to the threshold key ranked by direct comparison
static_assert(FS_THREADS % kStreamLanes == 0, "whole threads per per-thread list");

constexpr int FS_DENSE_MAX = 6144;                        // list entries the shared-memory copy holds; longer lists are flagged

__global__ void __launch_bounds__(FS_THREADS)
finish_topk_stream_kernel(const uint2* __restrict__ cand, const uint32_t* __restrict__ sample_count,
                          const uint8_t* __restrict__ lane_count, const float* __restrict__ tau,
                          int64_t n_rows, int64_t q_begin, int rows_per_item, int k_top, int32_t* __restrict__ out,
                          uint8_t* __restrict__ row_fail, uint8_t* __restrict__ item_fail) {
    __shared__ __align__(16) TopkSmem<FS_WARPS, 2048> sm;
    __shared__ uint32_t dense_key[FS_DENSE_MAX];               // the list's keys, packed
    __shared__ uint16_t dense_slot[FS_DENSE_MAX];              // ... and the slot of the row's list each came from
    __shared__ uint32_t eq_idx[FS_EQ_MAX];
    __shared__ uint32_t list_off[kStreamLanes + 1];            // where per-thread list j starts in the packed copy
    __shared__ uint32_t eq_count, ge_count, over_count, key_lo, key_hi;
    extern __shared__ uint32_t bitmap[];                       // one bit per key position of the longest row of the launch
    const int tid = threadIdx.x;
    const int lane = tid & 31, wid = tid >> 5;
    constexpr int kListsPerWarp = kStreamLanes / FS_WARPS;
    int slot = 0;
    for (int64_t item = blockIdx.x; item * rows_per_item < n_rows; item += gridDim.x) {
        bool any_fail = false;
        for (int r = 0; r < rows_per_item; ++r) {
            const int64_t row = item * rows_per_item + r;
            if (row >= n_rows) break;
            const int n = static_cast<int>(q_begin + row + 1);                 // the row has scores 0 .. n - 1
            const uint32_t kk = static_cast<uint32_t>(k_top < n ? k_top : n);
            int32_t* out_row = out + row * static_cast<int64_t>(k_top);
            const uint32_t n_sample = sample_count[row];
            const float t_row = tau[row];
            const bool no_tau = t_row == -INFINITY;
            const uint32_t t_key = score_key(t_row);
            const uint2* lst = cand + row * static_cast<int64_t>(kStreamRowSlots);
            __syncthreads();                                   // the previous row's readers of the shared arrays are done
            if (tid == 0) { eq_count = 0u; ge_count = 0u; over_count = 0u; key_lo = 0xFFFFFFFFu; key_hi = 0u; }
            // ---- where every per-thread list goes in the packed copy: a prefix sum over the 128 list lengths
            uint32_t my_len = 0;
            if (tid < kStreamLanes) {
                my_len = lane_count[row * kStreamLanes + tid];
                if (my_len > static_cast<uint32_t>(kStreamLaneCap)) { atomicAdd(&over_count, 1u); my_len = kStreamLaneCap; }
            }
            uint32_t m;                                        // entries of the list
            const uint32_t off = block_excl_scan<FS_WARPS>(my_len, sm, slot, m) + n_sample;
            if (tid < kStreamLanes) list_off[tid] = off;
            m += n_sample;
            if (tid == 0) list_off[kStreamLanes] = m;
            __syncthreads();
            // flagged: a list overflowed or is longer than the packed copy (the same for every thread)
            if (over_count != 0u || n_sample > static_cast<uint32_t>(kStreamSampleCap) || m > static_cast<uint32_t>(FS_DENSE_MAX) || m < kk) {
                if (tid == 0) row_fail[row] = 1;
                any_fail = true;
                continue;
            }
            // ---- one pass over global memory: keys into the packed copy (the sample part thread by thread; the per-thread
            // lists a warp per list, a lane per position: a list is a contiguous run of slots), smallest and largest key,
            // entries >= tau
            uint32_t c_ge = 0, k_lo = 0xFFFFFFFFu, k_hi = 0u;
            auto take = [&](uint32_t dst, int slot_i) {
                const uint32_t key = score_key(__uint_as_float(__ldg(&lst[slot_i].x)));
                dense_key[dst] = key;
                dense_slot[dst] = static_cast<uint16_t>(slot_i);
                c_ge += no_tau || key >= t_key;
                k_lo = key < k_lo ? key : k_lo;
                k_hi = key > k_hi ? key : k_hi;
            };
            for (uint32_t i = tid; i < n_sample; i += FS_THREADS) take(i, static_cast<int>(i));
#pragma unroll 4
            for (int j = 0; j < kListsPerWarp; ++j) {
                const int list = wid * kListsPerWarp + j;
                const uint32_t o = list_off[list], len = list_off[list + 1] - o;
                for (uint32_t pos = lane; pos < len; pos += 32) take(o + pos, kStreamSampleCap + list * kStreamLaneCap + static_cast<int>(pos));
            }
            c_ge = __reduce_add_sync(0xFFFFFFFFu, c_ge);
            k_lo = __reduce_min_sync(0xFFFFFFFFu, k_lo);
            k_hi = __reduce_max_sync(0xFFFFFFFFu, k_hi);
            if (lane == 0) {
                if (c_ge != 0u) atomicAdd(&ge_count, c_ge);
                atomicMin(&key_lo, k_lo);
                atomicMax(&key_hi, k_hi);
            }
            __syncthreads();
            // flagged: fewer than kk entries reach tau (some score that was dropped could belong to the answer)
            if (ge_count < kk) {
                if (tid == 0) row_fail[row] = 1;
                any_fail = true;
                continue;
            }
            // ---- the key of rank kk. The keys of a list are close together (scores at or above one threshold), so the
            // top bits of the key would put them all into a few bins; the bins are laid over [smallest, largest] instead,
            // 2048 at a time, and narrowed to the bin that holds the rank until a bin is one key wide
            uint32_t need = kk;
            uint32_t base = key_lo;                            // the window of keys still in play starts here ...
            uint32_t window_bits = 32u - static_cast<uint32_t>(__clz(key_hi - key_lo));   // ... and is < 2^window_bits wide (0: one key)
            for (;;) {
                const uint32_t shift = window_bits > 11u ? window_bits - 11u : 0u;
                const uint32_t window_last = window_bits >= 32u ? 0xFFFFFFFFu : (1u << window_bits) - 1u;   // largest key - base in the window
                zero_hist<FS_THREADS>(sm, 2048);
                __syncthreads();
                for (uint32_t i = tid; i < m; i += FS_THREADS) {
                    const uint32_t key = dense_key[i];
                    if (key >= base && key - base <= window_last) atomicAdd(&sm.hist[(key - base) >> shift], 1u);
                }
                __syncthreads();
                uint32_t bin, above;
                select_bucket<2048, FS_THREADS>(sm, need, slot, bin, above);
                need -= above;
                base += bin << shift;
                if (shift == 0u) break;
                window_bits = shift;
            }
            const uint32_t T = base;                           // need = entries to take among those equal to T, >= 1
            // ---- bitmap of the chosen positions
            const int n_words = (n + 31) >> 5;
            for (int w = tid; w < n_words; w += FS_THREADS) bitmap[w] = 0u;
            __syncthreads();
            bool bad_index = false;
            for (uint32_t i = tid; i < m; i += FS_THREADS) {
                const uint32_t key = dense_key[i];
                if (key < T) continue;
                const uint32_t idx = __ldg(&lst[dense_slot[i]].y);
                if (idx >= static_cast<uint32_t>(n)) { bad_index = true; continue; }      // cannot happen with a list the scorer wrote
                if (key > T) {
                    atomicOr(&bitmap[idx >> 5], 1u << (idx & 31u));
                } else {
                    const uint32_t pos = atomicAdd(&eq_count, 1u);
                    if (pos < static_cast<uint32_t>(FS_EQ_MAX)) eq_idx[pos] = idx;
                }
            }
            const bool any_bad = __syncthreads_or(bad_index);
            const uint32_t n_eq = eq_count;
            if (any_bad || n_eq > static_cast<uint32_t>(FS_EQ_MAX)) {          // many equal scores at the threshold: the ordinary path
                if (tid == 0) row_fail[row] = 1;
                any_fail = true;
                continue;
            }
            for (uint32_t i = tid; i < n_eq; i += FS_THREADS) {               // among equal scores the lowest key indices win
                const uint32_t mine = eq_idx[i];
                uint32_t lower = 0;
                for (uint32_t j = 0; j < n_eq; ++j) lower += eq_idx[j] < mine;
                if (lower < need) atomicOr(&bitmap[mine >> 5], 1u << (mine & 31u));
            }
            __syncthreads();
            // ---- read-out in ascending position order: every thread owns a run of bitmap words
            const int wpt = (n_words + FS_THREADS - 1) / FS_THREADS;
            const int w0 = tid * wpt < n_words ? tid * wpt : n_words;
            const int w1 = w0 + wpt < n_words ? w0 + wpt : n_words;
            uint32_t c = 0;
            for (int w = w0; w < w1; ++w) c += __popc(bitmap[w]);
            uint32_t total;
            uint32_t pos = block_excl_scan<FS_WARPS>(c, sm, slot, total);
            for (int w = w0; w < w1; ++w) {
                uint32_t bw = bitmap[w];
                while (bw) {
                    const int bit = __ffs(bw) - 1;
                    bw &= bw - 1;
                    if (pos < kk) out_row[pos] = 32 * w + bit;
                    ++pos;
                }
            }
            for (uint32_t j = kk + tid; j < static_cast<uint32_t>(k_top); j += FS_THREADS) out_row[j] = -1;
            if (tid == 0) row_fail[row] = 0;
        }
        if (tid == 0) item_fail[item] = any_fail ? 1 : 0;
    }
}

}  // namespace

cudaError_t launch_finish_topk_stream(const StreamTopk& st, int64_t n_rows, int64_t q_begin, int rows_per_item, int32_t* out,
                                      uint8_t* row_fail, uint8_t* item_fail, cudaStream_t stream) {
    if (n_rows <= 0) return cudaSuccess;
    const int64_t n_items = (n_rows + rows_per_item - 1) / rows_per_item;
    const int64_t max_grid = 1 << 20;
    const unsigned grid = static_cast<unsigned>(n_items < max_grid ? n_items : max_grid);
    const int64_t longest = q_begin + n_rows;                  // keys of the last row
    if (longest > kStreamMaxKeys) return cudaErrorInvalidValue;
    const int map_bytes = static_cast<int>((longest + 31) / 32 * 4);
    if (cudaError_t e = ensure_max_dynamic_smem(reinterpret_cast<const void*>(finish_topk_stream_kernel), kStreamMaxKeys / 8); e != cudaSuccess) return e;
    finish_topk_stream_kernel<<<grid, FS_THREADS, map_bytes, stream>>>(st.cand, st.sample_count, st.lane_count, st.tau, n_rows, q_begin,
                                                                       rows_per_item, st.k_top, out, row_fail, item_fail);
    return cudaGetLastError();
}

}  // namespace idxc
