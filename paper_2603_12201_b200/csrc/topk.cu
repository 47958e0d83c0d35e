// Row-wise top-k select (Sec. 3 "Notation": T_t = Top-k(I_t)).
//
// One CTA per row, many rows in flight per SM (256 threads and <= 42 registers per thread when
// there are many rows; 1024 threads for a handful of rows). A few LONG rows (decode) go to the
// cluster kernel of topk_cluster.cu instead. Each warp
// owns one contiguous segment of the row. Scores are compared through order-preserving 32-bit
// keys (larger score <=> larger key, -0 == +0); the k-th largest is found exactly by a radix
// select, 12 + 10 + 10 key bits, most significant first:
//   sweep 1 (the HBM read)  4096-bin shared-memory histogram of the top 12 key bits; a suffix
//                           scan finds the threshold bucket b1 holding the k-th largest score.
//   sweep 2 (L2)            scores above bucket b1 are certainly selected, scores inside it
//                           (typically < 2 % of the row) are candidates: both are flagged in a
//                           shared-memory map (one byte per 128-bit load: low nibble "selected",
//                           high nibble "candidate").
//   candidates              gathered with key and position by walking the high nibbles (slots by
//                           prefix popcount, no atomics); digits 2 and 3 on those only give the
//                           exact threshold T; candidates above T, and the lowest-position ones
//                           equal to T until k are reached, are flagged as selected.
//   emission                a block-wide prefix popcount over the low nibbles ranks every selected
//                           position: ascending indices, deterministic tie-break, no atomics on
//                           the output.
// Sweep 2 compares floats against the bucket bounds, which orders exactly like the keys. If the
// threshold bucket holds more scores than the candidate buffer (many near-equal scores, e.g. a
// constant row), or the row is longer than the map, digits 2 and 3 are histogrammed over the whole
// row and the emission uses block-wide prefix sums over the row instead; same result, slower.
#include "kernels.h"
#include "topk_common.cuh"

namespace idxc {
using namespace topk;
namespace {

// The candidate buffers live in the upper three quarters of the 4096-bin histogram, which is
// only needed as a whole until the threshold bucket is known: 1536 keys + 1536 positions.
constexpr int TK_CAP = (TK_BINS1 - TK_BINS23) / 2;
constexpr int TK_MAP_MAX_BYTES = 128 * 1024;      // rows up to 524288 scores use the map

// CAP_DYN = 0: the candidate buffers alias the histogram (TK_CAP entries). CAP_DYN > 0: they hold
// CAP_DYN entries and live in dynamic shared memory behind the map (for launches with few, long rows,
// whose threshold bucket holds more scores).
template <int THREADS, int MIN_BLOCKS, int CAP_DYN>
__global__ void __launch_bounds__(THREADS, MIN_BLOCKS)
topk_rows_kernel(const float* __restrict__ scores, int64_t ld, int64_t n_rows, int64_t first_len, int64_t len_step,
                 const int32_t* __restrict__ lens, int k_top, int32_t* __restrict__ out, int map_scores) {
    constexpr int WARPS = THREADS / 32;
    __shared__ __align__(16) TopkSmem<WARPS> sm;
    extern __shared__ uint32_t sel_map[];                        // map_scores / 16 words
    uint8_t* sel_bytes = reinterpret_cast<uint8_t*>(sel_map);
    constexpr int CAP = CAP_DYN > 0 ? CAP_DYN : TK_CAP;
    uint32_t* cand_key = CAP_DYN > 0 ? sel_map + map_scores / 16 : sm.hist + TK_BINS23;   // aliased: valid once b1 is known
    uint32_t* cand_idx = cand_key + CAP;
    int slot = 0;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const uint32_t k = static_cast<uint32_t>(k_top);
    // longest rows first when lengths grow with the row number
    for (int64_t blk = blockIdx.x; blk < n_rows; blk += gridDim.x) {
        const int64_t row = n_rows - 1 - blk;
        int64_t len = lens ? static_cast<int64_t>(lens[row]) : first_len + row * len_step;
        len = len < 0 ? 0 : (len > ld ? ld : len);
        const int n = static_cast<int>(len);
        int32_t* out_row = out + row * static_cast<int64_t>(k_top);
        if (n <= k_top) {   // fewer candidates than k: all of them, then padding
            for (int j = threadIdx.x; j < k_top; j += THREADS) out_row[j] = j < n ? j : -1;
            continue;
        }
        const float* src = scores + row * ld;
        // this warp's segment: a multiple of 128 scores, so every lane loads aligned float4s
        const int seg = (((n + WARPS - 1) / WARPS) + 127) & ~127;
        const int seg_begin = wid * seg < n ? wid * seg : n;
        const int seg_end = seg_begin + seg < n ? seg_begin + seg : n;

        // ---- sweep 1: histogram of the top 12 key bits over the whole row
        __syncthreads();   // earlier readers of sm are done
        zero_hist<THREADS>(sm, TK_BINS1);
        __syncthreads();
        sweep_segment<TK_UNROLL>(src, n, seg_begin, seg_end, lane, [&](const float4& x, int base) {
            const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (base + e < n) atomicAdd(&sm.hist[score_digit1(xs[e])], 1u);
        });
        __syncthreads();
        uint32_t b1, above1;
        select_bucket<TK_BINS1, THREADS>(sm, k, slot, b1, above1);
        const uint32_t c1 = sm.hist[b1];
        uint32_t need = k - above1;          // rank inside bucket b1, 1-based
        __syncthreads();                     // everyone has read hist[b1]: the candidate buffers may now overwrite the bins

        if (c1 <= static_cast<uint32_t>(CAP) && n <= map_scores) {
            // ---- sweep 2: flag the scores above bucket b1 (selected) and inside it (candidates)
            const float lo = key_to_score(b1 << 20);                       // smallest score of bucket b1
            const bool has_above = b1 < TK_BINS1 - 1;
            const float hi = key_to_score(has_above ? ((b1 + 1) << 20) : 0xFFFFFFFFu);   // smallest score above it
            sweep_segment<TK_UNROLL>(src, n, seg_begin, seg_end, lane, [&](const float4& x4, int base) {
                const float x[4] = {x4.x, x4.y, x4.z, x4.w};
                uint32_t flags = 0;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (base + e >= n || !(x[e] >= lo)) continue;
                    flags |= (has_above && x[e] >= hi) ? (1u << e) : (16u << e);
                }
                sel_bytes[base >> 2] = static_cast<uint8_t>(flags);        // lanes past the end of the row write 0
            });
            __syncthreads();
            // ---- gather the candidates (high nibbles) with their keys; slots by prefix popcount
            const int words = (n + 15) >> 4;
            const int wpt = (words + THREADS - 1) / THREADS;
            const int w0 = static_cast<int>(threadIdx.x) * wpt < words ? static_cast<int>(threadIdx.x) * wpt : words;
            const int w1 = w0 + wpt < words ? w0 + wpt : words;
            {
                uint32_t cnt = 0;
                for (int w = w0; w < w1; ++w) cnt += __popc(sel_map[w] & 0xF0F0F0F0u);
                uint32_t total;
                uint32_t pos = block_excl_scan(cnt, sm, slot, total);
                for (int w = w0; w < w1; ++w) {
                    uint32_t m = sel_map[w] & 0xF0F0F0F0u;
                    while (m) {
                        const int b = __ffs(m) - 1;
                        m &= m - 1;
                        const int idx = 16 * w + 4 * (b >> 3) + (b & 7) - 4;
                        if (pos < static_cast<uint32_t>(CAP)) {
                            cand_key[pos] = score_key(__ldg(src + idx)) & 0xFFFFFu;
                            cand_idx[pos] = static_cast<uint32_t>(idx);
                        }
                        ++pos;
                    }
                }
            }
            // ---- digits 2 and 3 on the candidates
            uint32_t t_low, need_eq, m_eq;
            candidate_select<THREADS>(sm, cand_key, c1, need, slot, t_low, need_eq, m_eq);
            // ---- flag the selected candidates
            for (uint32_t i = threadIdx.x; i < c1; i += THREADS) {
                const uint32_t c = cand_key[i];
                bool take = c > t_low;
                if (c == t_low) {
                    take = true;
                    if (m_eq != need_eq) {                       // ties compete: the lowest positions win
                        uint32_t before = 0;
                        for (uint32_t i2 = 0; i2 < c1; ++i2) before += (cand_key[i2] == t_low) & (cand_idx[i2] < cand_idx[i]);
                        take = before < need_eq;
                    }
                }
                if (take) {
                    const uint32_t idx = cand_idx[i];
                    atomicOr(&sel_map[idx >> 4], 1u << (8u * ((idx >> 2) & 3u) + (idx & 3u)));
                }
            }
            __syncthreads();
            // ---- emission: rank the selected positions by a prefix popcount over the low nibbles
            uint32_t cnt = 0;
            for (int w = w0; w < w1; ++w) cnt += __popc(sel_map[w] & 0x0F0F0F0Fu);
            uint32_t total;
            uint32_t rank = block_excl_scan(cnt, sm, slot, total);
            for (int w = w0; w < w1; ++w) {
                uint32_t m = sel_map[w] & 0x0F0F0F0Fu;
                while (m) {
                    const int b = __ffs(m) - 1;
                    m &= m - 1;
                    if (rank < k) out_row[rank] = 16 * w + 4 * (b >> 3) + (b & 7);
                    ++rank;
                }
            }
            continue;
        }

        // ---- slow path: digits 2 and 3 over the whole row, then block-scan emission
        slow_path<THREADS>(sm, src, n, b1, need, k, out_row, slot);
    }
}

template <int THREADS, int MIN_BLOCKS, int CAP_DYN>
cudaError_t launch_instance(const float* scores, int64_t ld, int64_t n_rows, int64_t first_len, int64_t len_step,
                            const int32_t* lens, int k_top, int32_t* out, int map_bytes, cudaStream_t stream) {
    auto kern = topk_rows_kernel<THREADS, MIN_BLOCKS, CAP_DYN>;
    if (cudaError_t e = ensure_max_dynamic_smem(reinterpret_cast<const void*>(kern), TK_MAP_MAX_BYTES + 8 * CAP_DYN); e != cudaSuccess) return e;
    const int64_t max_grid = 1 << 20;
    const unsigned grid = static_cast<unsigned>(n_rows < max_grid ? n_rows : max_grid);
    kern<<<grid, THREADS, map_bytes + 8 * CAP_DYN, stream>>>(scores, ld, n_rows, first_len, len_step, lens, k_top, out, map_bytes * 4);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_topk_rows(const float* scores, int64_t ld, int64_t n_rows, int64_t first_len, int64_t len_step,
                             const int32_t* lens, int k_top, int32_t* out, cudaStream_t stream) {
    if (n_rows <= 0) return cudaSuccess;
    // the selection map covers the longest row of this launch, rounded up to a whole 128-score block
    int64_t longest = lens ? ld : first_len + (n_rows - 1) * len_step;
    if (longest > ld) longest = ld;
    if (longest < 0) longest = 0;
    if (topk_cluster_applicable(n_rows, longest))
        return launch_topk_rows_cluster(scores, ld, n_rows, first_len, len_step, lens, k_top, out, longest, stream);
    int64_t map_bytes = (longest + 127) / 128 * 32;
    if (map_bytes > TK_MAP_MAX_BYTES) map_bytes = TK_MAP_MAX_BYTES;
    // many rows: small CTAs, many per SM; few rows: more threads per row
    if (n_rows >= 1024)
        return launch_instance<256, 6, 0>(scores, ld, n_rows, first_len, len_step, lens, k_top, out, static_cast<int>(map_bytes), stream);
    return launch_instance<1024, 1, 8192>(scores, ld, n_rows, first_len, len_step, lens, k_top, out, static_cast<int>(map_bytes), stream);
}

}  // namespace idxc
