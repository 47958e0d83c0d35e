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
// Selection: the list's keys (order-preserving 32-bit images of the scores) sit in registers; three histogram passes
// (11 + 11 + 10 bits) find the key of the wanted rank; the chosen key indices are set in a bitmap over the row's
// positions and read out in ascending order.
#include "kernels.h"
#include "topk_common.cuh"

namespace idxc {
using namespace topk;
namespace {

constexpr int FS_THREADS = 256;
constexpr int FS_WARPS = FS_THREADS / 32;
constexpr int FS_SAMPLE_PER = kStreamSampleCap / FS_THREADS;                 // sample slots per thread
constexpr int FS_LIST_PER = kStreamLaneCap / (FS_THREADS / kStreamLanes);     // slots of a per-thread list that one thread covers
constexpr int FS_PER = FS_SAMPLE_PER + FS_LIST_PER;                           // entries a thread may hold
constexpr int FS_EQ_MAX = 256;                           // entries equal to the threshold key ranked by direct comparison
static_assert(kStreamSampleCap % FS_THREADS == 0 && FS_THREADS % kStreamLanes == 0 && kStreamLaneCap % (FS_THREADS / kStreamLanes) == 0,
              "list slots per thread");
static_assert(FS_PER <= 64, "one bit per slot of a thread");
// Entry e of thread tid: e < FS_SAMPLE_PER: slot tid + 256 e of the sample part; else position
// tid / 128 + 2 (e - FS_SAMPLE_PER) of per-thread list tid % 128 (lists are filled from position 0, so a thread's
// entries of a list end where the list does, and the whole block can stop at the longest list).
__device__ __forceinline__ int fs_slot(int tid, int e) {
    if (e < FS_SAMPLE_PER) return tid + FS_THREADS * e;
    return kStreamSampleCap + (tid % kStreamLanes) * kStreamLaneCap + tid / kStreamLanes + (FS_THREADS / kStreamLanes) * (e - FS_SAMPLE_PER);
}

__global__ void __launch_bounds__(FS_THREADS)
finish_topk_stream_kernel(const uint2* __restrict__ cand, const uint32_t* __restrict__ sample_count,
                          const uint8_t* __restrict__ lane_count, const float* __restrict__ tau,
                          int64_t n_rows, int64_t q_begin, int rows_per_item, int k_top, int32_t* __restrict__ out,
                          uint8_t* __restrict__ row_fail, uint8_t* __restrict__ item_fail) {
    __shared__ __align__(16) TopkSmem<FS_WARPS, 2048> sm;
    extern __shared__ uint32_t bitmap[];                       // one bit per key position of the longest row of the launch
    __shared__ uint32_t eq_idx[FS_EQ_MAX];
    __shared__ uint32_t lane_len[kStreamLanes];
    __shared__ uint32_t eq_count, ge_count, over_count, longest_list;
    const int tid = threadIdx.x;
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
            __syncthreads();                                   // the previous row's readers of the shared arrays are done
            if (tid == 0) { eq_count = 0u; ge_count = 0u; over_count = 0u; longest_list = 0u; }
            if (tid < kStreamLanes) lane_len[tid] = lane_count[row * kStreamLanes + tid];
            zero_hist<FS_THREADS>(sm, 2048);
            __syncthreads();
            // ---- the list's keys into registers; entries >= tau counted; first histogram
            uint32_t key[FS_PER];
            uint64_t have = 0;                                 // bit e: entry e of this thread exists
            uint32_t c_ge = 0;
            const uint2* lst = cand + row * static_cast<int64_t>(kStreamRowSlots);
            if (tid < kStreamLanes) {
                if (lane_len[tid] > static_cast<uint32_t>(kStreamLaneCap)) atomicAdd(&over_count, 1u);
                atomicMax(&longest_list, lane_len[tid] < static_cast<uint32_t>(kStreamLaneCap) ? lane_len[tid] : static_cast<uint32_t>(kStreamLaneCap));
            }
            __syncthreads();
            const uint32_t my_len = lane_len[tid % kStreamLanes];
            const int n_list_iter = static_cast<int>((longest_list + (FS_THREADS / kStreamLanes) - 1) / (FS_THREADS / kStreamLanes));
#pragma unroll
            for (int e = 0; e < FS_PER; ++e) {
                key[e] = 0u;
                if (e >= FS_SAMPLE_PER && e - FS_SAMPLE_PER >= n_list_iter) continue;                  // (the same for every thread)
                const bool there = e < FS_SAMPLE_PER ? static_cast<uint32_t>(tid + FS_THREADS * e) < n_sample
                                                     : static_cast<uint32_t>(tid / kStreamLanes + (FS_THREADS / kStreamLanes) * (e - FS_SAMPLE_PER)) < my_len;
                if (there) {
                    have |= 1ull << e;
                    key[e] = score_key(__uint_as_float(__ldg(&lst[fs_slot(tid, e)].x)));
                    c_ge += no_tau || key[e] >= t_key;
                    atomicAdd(&sm.hist[key[e] >> 21], 1u);
                }
            }
            c_ge = __reduce_add_sync(0xFFFFFFFFu, c_ge);
            if ((tid & 31) == 0 && c_ge != 0u) atomicAdd(&ge_count, c_ge);
            __syncthreads();
            // flagged: overflow, fewer than kk entries reach tau, or an index that cannot be a key of this row (the
            // same for every thread)
            if (over_count != 0u || n_sample > static_cast<uint32_t>(kStreamSampleCap) || ge_count < kk) {
                if (tid == 0) row_fail[row] = 1;
                any_fail = true;
                continue;
            }
            // ---- the key of rank kk: 11 + 11 + 10 bits
            uint32_t need = kk, b1, b2, b3, above;
            select_bucket<2048, FS_THREADS>(sm, need, slot, b1, above);
            need -= above;
            zero_hist<FS_THREADS>(sm, 2048);
            __syncthreads();
#pragma unroll
            for (int e = 0; e < FS_PER; ++e)
                if (((have >> e) & 1ull) && (key[e] >> 21) == b1) atomicAdd(&sm.hist[(key[e] >> 10) & 2047u], 1u);
            __syncthreads();
            select_bucket<2048, FS_THREADS>(sm, need, slot, b2, above);
            need -= above;
            zero_hist<FS_THREADS>(sm, 1024);
            __syncthreads();
            const uint32_t p2 = (b1 << 11) | b2;
#pragma unroll
            for (int e = 0; e < FS_PER; ++e)
                if (((have >> e) & 1ull) && (key[e] >> 10) == p2) atomicAdd(&sm.hist[key[e] & 1023u], 1u);
            __syncthreads();
            select_bucket<1024, FS_THREADS>(sm, need, slot, b3, above);
            need -= above;                                     // entries to take among those equal to the threshold key, >= 1
            const uint32_t T = (p2 << 10) | b3;
            // ---- bitmap of the chosen positions
            const int n_words = (n + 31) >> 5;
            for (int w = tid; w < n_words; w += FS_THREADS) bitmap[w] = 0u;
            __syncthreads();
            bool bad_index = false;
#pragma unroll
            for (int e = 0; e < FS_PER; ++e) {
                if (!((have >> e) & 1ull) || key[e] < T) continue;
                const uint32_t idx = __ldg(&lst[fs_slot(tid, e)].y);
                if (idx >= static_cast<uint32_t>(n)) { bad_index = true; continue; }      // cannot happen with a list the scorer wrote
                if (key[e] > T) {
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
                uint32_t b = bitmap[w];
                while (b) {
                    const int bit = __ffs(b) - 1;
                    b &= b - 1;
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
    finish_topk_stream_kernel<<<grid, FS_THREADS, map_bytes, stream>>>(st.cand, st.sample_count, st.lane_count, st.tau, n_rows, q_begin,
                                                                       rows_per_item, st.k_top, out, row_fail, item_fail);
    return cudaGetLastError();
}

}  // namespace idxc
