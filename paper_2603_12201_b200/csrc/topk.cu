// Row-wise top-k select (Sec. 3 "Notation": T_t = Top-k(I_t)).
//
// One CTA per row, many rows in flight per SM (128 threads when there are many rows; 1024 threads for a
// handful of rows). A few LONG rows (decode) go to the cluster kernel of topk_cluster.cu instead. Each warp
// owns one contiguous segment of the row. The exact top-k comes out of ONE sweep over the row:
//   sample      a sixteenth of the row or more (128-score blocks spread over every warp's segment; the whole row
//               when it is short) gives a mean and a spread, which fix a monotone map score -> bin
//               floor(x * scale + offset), clamped to [0, 1023], with the bins laid around where the k-th largest
//               score should lie. A histogram of the sample in these bins gives two pivot scores that bracket the
//               k-th largest score of the whole row: bin edges next to the sample's scores of rank
//               r -+ (3.5 standard deviations of that rank under sampling), r = k * sample / n.
//   sweep       (the HBM read) every score at or above the upper pivot is certainly selected, the scores between
//               the pivots (a few per cent of the row) are candidates: both are flagged in a shared-memory map (one
//               byte per 128-bit load: low nibble "selected", high nibble "candidate") and counted.
//   check       with A scores above and C candidates the bracket held iff A < k <= A + C. It then remains to take
//               the k - A largest candidates.
//   candidates  gathered into a list by walking the map; one histogram of the list in 1024 finer bins across the band
//               leaves a handful of scores in the bin of the wanted rank; those are ranked by direct comparison of
//               their order-preserving 32-bit keys (larger key first, lower position first among equal keys).
//               Selected candidates are flagged in the map.
//   emission    warp-wide prefix popcounts over the map rank every selected position: ascending indices,
//               deterministic tie-break, no atomics on the output.
// The result never depends on the sample: the pivots only decide how many scores become candidates, the counts are
// exact, and when the bracket does not hold (a few rows in ten thousand for independent scores; constant rows,
// heavy ties, infinities, or scores that drift along the row) or a list overflows, the row is selected on keys
// alone by three histogram passes over the row; same result, slower. Rows longer than the map take that path too.
#include "kernels.h"
#include "topk_common.cuh"

namespace idxc {
using namespace topk;
namespace {

constexpr int TK_BINS = 1024;
constexpr int TK_MAP_MAX_BYTES = 128 * 1024;      // rows up to 524288 scores use the map
constexpr int TK_SMALL = 128;                     // scores ranked by direct comparison at most
constexpr int TK_PREFETCH = 16384;                // bytes of a warp's segment asked for ahead of the sweep

struct alignas(16) TopkRowSmem : SampleSmem {
    uint32_t part_a[32], part_c[32];
    uint32_t cand_count;
    uint32_t small_count;
    uint32_t small_key[TK_SMALL];
    uint32_t small_idx[TK_SMALL];
};

// CAP candidates (fine bin, position) in dynamic shared memory behind the map.
template <int THREADS, int MIN_BLOCKS, int CAP>
__global__ void __launch_bounds__(THREADS, MIN_BLOCKS)
topk_rows_kernel(const float* __restrict__ scores, int64_t ld, int64_t n_rows, int64_t first_len, int64_t len_step,
                 const int32_t* __restrict__ lens, int k_top, int32_t* __restrict__ out, int map_scores,
                 const uint8_t* __restrict__ row_mask) {
    constexpr int WARPS = THREADS / 32;
    constexpr int U = TK_UNROLL;
    __shared__ __align__(16) TopkSmem<WARPS, 2048> sm;           // 2048 bins: the keys-only path needs them
    __shared__ TopkRowSmem rs;
    extern __shared__ uint32_t sel_map[];                        // map_scores / 16 words, then the candidates
    uint8_t* sel_bytes = reinterpret_cast<uint8_t*>(sel_map);
    uint32_t* cand_fb = sel_map + map_scores / 16;               // a candidate's fine bin ...
    uint32_t* cand_idx = cand_fb + CAP;                          // ... and position
    int32_t* stage = reinterpret_cast<int32_t*>(cand_fb);        // the selected indices of a row before they are stored (the candidates are done with by then)
    static_assert(2 * CAP >= 2048, "the staging area holds k_top indices");
    int slot = 0;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const uint32_t k = static_cast<uint32_t>(k_top);
    // longest rows first when lengths grow with the row number
    for (int64_t blk = blockIdx.x; blk < n_rows; blk += gridDim.x) {
        const int64_t row = n_rows - 1 - blk;
        if (row_mask != nullptr && row_mask[row] == 0) continue;
        int64_t len = lens ? static_cast<int64_t>(lens[row]) : first_len + row * len_step;
        len = len < 0 ? 0 : (len > ld ? ld : len);
        const int n = static_cast<int>(len);
        int32_t* out_row = out + row * static_cast<int64_t>(k_top);
        if (n <= k_top) {   // fewer candidates than k: all of them, then padding
            for (int j = threadIdx.x; j < k_top; j += THREADS) out_row[j] = j < n ? j : -1;
            continue;
        }
        const float* src = scores + row * ld;
        if (n > map_scores) {                                    // longer than the map: keys alone
            slow_path_full<THREADS>(sm, src, n, k, out_row, slot);
            continue;
        }
        // this warp's segment: a multiple of 128 scores, so every lane loads aligned float4s
        const int seg = (((n + WARPS - 1) / WARPS) + 127) & ~127;
        const int seg_begin = wid * seg < n ? wid * seg : n;
        const int seg_end = seg_begin + seg < n ? seg_begin + seg : n;
        // ask the L2 for the head of this warp's segment now: the sweep comes after the sample, its histogram and two
        // scans, and then finds its first scores on the chip (5 % of the kernel's time on rows of 12K..40K scores, which
        // this covers whole; asking for all of a longer row, at once or as the sweep advances, measured slower: the rows
        // of the resident blocks then no longer fit the L2 together)
        {
            const int seg_bytes = ((seg_end - seg_begin) * 4) & ~15;
            if (lane == 0 && seg_bytes > 0)
                asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src + seg_begin), "r"(static_cast<uint32_t>(seg_bytes < TK_PREFETCH ? seg_bytes : TK_PREFETCH)) : "memory");
        }
        // ---- the sample and the two pivot scores around the k-th largest (the same code serves the cluster kernel)
        __syncthreads();   // earlier readers of sm, rs and the map are done
        if (threadIdx.x == 0) { rs.cand_count = 0u; rs.small_count = 0u; }
        const Pivots pv = sample_pivots<THREADS, TK_BINS>(sm, rs, src, n, k_top, slot);
        if (!pv.usable) {                                        // the same for every thread
            slow_path_full<THREADS>(sm, src, n, k, out_row, slot);
            continue;
        }
        const float lo_x = pv.lo_x, hi_x = pv.hi_x;

        // ---- the sweep: flag the scores at or above the upper pivot and those between the pivots
        {
            // whole steps of U blocks that lie inside the segment and the row need no bounds checks
            const int full_end = seg_begin + ((seg_end & ~3) - seg_begin) / (128 * U) * (128 * U);
            const float* p = src + seg_begin + 4 * lane;
            uint8_t* mb = sel_bytes + (seg_begin >> 2) + lane;
            int cb = seg_begin;
            for (; cb < full_end; cb += 128 * U, p += 128 * U, mb += 32 * U) {
                float4 x4[U];
#pragma unroll
                for (int u = 0; u < U; ++u) x4[u] = __ldg(reinterpret_cast<const float4*>(p + 128 * u));
#pragma unroll
                for (int u = 0; u < U; ++u) mb[32 * u] = static_cast<uint8_t>(flag4(x4[u], lo_x, hi_x));
            }
            for (; cb < seg_end; cb += 128) {                           // the ragged rest, one block at a time
                const int base = cb + 4 * lane;
                uint32_t flags = 0;
                if (base < n) {
                    flags = flag4(__ldg(reinterpret_cast<const float4*>(src + base)), lo_x, hi_x);
                    const int left = n - base;                          // scores of this 128-bit load inside the row
                    if (left < 4) flags &= (0x11u << left) - 0x11u;
                }
                sel_bytes[base >> 2] = static_cast<uint8_t>(flags);    // lanes past the end of the row write 0
            }
        }
        __syncwarp();
        // A = scores above the band, C = scores inside it: counted from this warp's part of the map, summed over the block
        const int w_begin = seg_begin >> 4, w_end = seg_begin < seg_end ? (seg_end + 15) >> 4 : w_begin;
        {
            uint32_t n_sel = 0, n_cand = 0;
            for (int w = w_begin + lane; w < w_end; w += 32) {
                const uint32_t m = sel_map[w];
                n_sel += __popc(m & 0x0F0F0F0Fu);
                n_cand += __popc(m & 0xF0F0F0F0u);
            }
            n_sel = __reduce_add_sync(0xFFFFFFFFu, n_sel);
            n_cand = __reduce_add_sync(0xFFFFFFFFu, n_cand);
            if (lane == 0) { rs.part_a[wid] = n_sel; rs.part_c[wid] = n_cand; }
        }
        __syncthreads();
        uint32_t A = 0, C = 0;
#pragma unroll
        for (int w = 0; w < WARPS; ++w) { A += rs.part_a[w]; C += rs.part_c[w]; }
        if (!(A < k && k - A <= C && C <= static_cast<uint32_t>(CAP))) { // the bracket did not hold, or the list would overflow
            slow_path_full<THREADS>(sm, src, n, k, out_row, slot);
            continue;
        }
        const uint32_t need = k - A;                                    // candidates to take, 1..C
        // ---- gather the candidates: each warp walks the map words of its segment, 32 words at a time
        zero_hist<THREADS>(sm, TK_BINS);
        // every lane owns a run of consecutive map words of its warp's segment
        const int wpl = (w_end - w_begin + 31) >> 5;
        const int lw0 = w_begin + lane * wpl < w_end ? w_begin + lane * wpl : w_end;
        const int lw1 = lw0 + wpl < w_end ? lw0 + wpl : w_end;
        {
            uint32_t c = 0;
            for (int w = lw0; w < lw1; ++w) c += __popc(sel_map[w] & 0xF0F0F0F0u);
            uint32_t total;
            uint32_t pos = warp_excl_scan(c, lane, total);
            uint32_t basepos = 0;
            if (lane == 0 && total != 0u) basepos = atomicAdd(&rs.cand_count, total);
            pos += __shfl_sync(0xFFFFFFFFu, basepos, 0);
            for (int w = lw0; w < lw1; ++w) {
                uint32_t m = squeeze_nibbles(sel_map[w] >> 4);
                const uint32_t idx0 = 16u * static_cast<uint32_t>(w);
                while (m) {
                    const uint32_t b = __ffs(m) - 1;
                    m &= m - 1;
                    if (pos < static_cast<uint32_t>(CAP)) cand_idx[pos] = idx0 + b;
                    ++pos;
                }
            }
        }
        __syncthreads();
        // ---- candidates: finer bins across the band
        auto fine_bin = [&](float x) -> uint32_t { return pv.fine_bin<TK_BINS>(x); };
        for (uint32_t i = threadIdx.x; i < C; i += THREADS) {             // independent loads (L2), all in flight together
            const uint32_t fb = fine_bin(__ldg(src + cand_idx[i]));
            cand_fb[i] = fb;
            atomicAdd(&sm.hist[fb], 1u);
        }
        __syncthreads();
        uint32_t fb1, above_f;
        select_bucket<TK_BINS, THREADS>(sm, need, slot, fb1, above_f);
        const uint32_t m1 = sm.hist[fb1];
        if (m1 > static_cast<uint32_t>(TK_SMALL)) {                     // many near-equal scores at the threshold
            slow_path_full<THREADS>(sm, src, n, k, out_row, slot);
            continue;
        }
        const uint32_t need1 = need - above_f;                          // scores to take from fine bin fb1, 1..m1
        for (uint32_t i = threadIdx.x; i < C; i += THREADS) {
            const uint32_t fb = cand_fb[i];
            if (fb > fb1) {
                flag_selected(sel_map, cand_idx[i]);
            } else if (fb == fb1) {
                const uint32_t pos = atomicAdd(&rs.small_count, 1u);
                const uint32_t idx = cand_idx[i];
                if (pos < static_cast<uint32_t>(TK_SMALL)) { rs.small_key[pos] = score_key(__ldg(src + idx)); rs.small_idx[pos] = idx; }
            }
        }
        __syncthreads();
        for (uint32_t i = threadIdx.x; i < m1; i += THREADS) {          // larger key first, lower position first among equal keys
            const uint32_t ki = rs.small_key[i], ii = rs.small_idx[i];
            uint32_t beaten_by = 0;
            for (uint32_t j = 0; j < m1; ++j) {
                const uint32_t kj = rs.small_key[j], ij = rs.small_idx[j];
                beaten_by += (kj > ki) | ((kj == ki) & (ij < ii));
            }
            if (beaten_by < need1) flag_selected(sel_map, ii);
        }
        __syncthreads();
        // ---- emission: a lane ranks the selected positions of its run of map words; lanes and warps are offset by
        // prefix sums of their counts
        {
            uint32_t c = 0;
            for (int w = lw0; w < lw1; ++w) c += __popc(sel_map[w] & 0x0F0F0F0Fu);
            uint32_t total;
            uint32_t pos = warp_excl_scan(c, lane, total);
            if (lane == 0) rs.part_a[wid] = total;
            __syncthreads();
#pragma unroll
            for (int w = 0; w < WARPS; ++w) pos += w < wid ? rs.part_a[w] : 0u;
            for (int w = lw0; w < lw1; ++w) {
                uint32_t m = squeeze_nibbles(sel_map[w]);
                const int idx0 = 16 * w;
                while (m) {
                    const int b = __ffs(m) - 1;
                    m &= m - 1;
                    if (pos < k) stage[pos] = idx0 + b;
                    ++pos;
                }
            }
            // the lanes' runs interleave in shared memory; the row leaves in whole 16-byte pieces (a lane's own stores
            // would touch one 32-byte sector per index)
            __syncthreads();
            if ((k_top & 3) == 0 && (reinterpret_cast<uintptr_t>(out_row) & 15) == 0) {
                const int4* s4 = reinterpret_cast<const int4*>(stage);
                int4* o4 = reinterpret_cast<int4*>(out_row);
                for (int j = threadIdx.x; j < (k_top >> 2); j += THREADS) o4[j] = s4[j];
            } else {
                for (int j = threadIdx.x; j < k_top; j += THREADS) out_row[j] = stage[j];
            }
        }
    }
}

template <int THREADS, int MIN_BLOCKS, int CAP>
cudaError_t launch_instance(const float* scores, int64_t ld, int64_t n_rows, int64_t first_len, int64_t len_step,
                            const int32_t* lens, int k_top, int32_t* out, int map_bytes, cudaStream_t stream,
                            const uint8_t* row_mask) {
    auto kern = topk_rows_kernel<THREADS, MIN_BLOCKS, CAP>;
    if (cudaError_t e = ensure_max_dynamic_smem(reinterpret_cast<const void*>(kern), TK_MAP_MAX_BYTES + 8 * CAP); e != cudaSuccess) return e;
    const int64_t max_grid = 1 << 20;
    const unsigned grid = static_cast<unsigned>(n_rows < max_grid ? n_rows : max_grid);
    kern<<<grid, THREADS, map_bytes + 8 * CAP, stream>>>(scores, ld, n_rows, first_len, len_step, lens, k_top, out, map_bytes * 4, row_mask);
    return cudaGetLastError();
}

constexpr int kCapMany = 1536, kCapFew = 8192;    // candidate slots of the two instances

}  // namespace


cudaError_t preload_topk_rows() {
    cudaFuncAttributes fa;
    const void* many = reinterpret_cast<const void*>(topk_rows_kernel<128, 8, kCapMany>);
    const void* few = reinterpret_cast<const void*>(topk_rows_kernel<1024, 1, kCapFew>);
    const void* mid = reinterpret_cast<const void*>(topk_rows_kernel<256, 4, 3072>);
    const void* half = reinterpret_cast<const void*>(topk_rows_kernel<512, 2, 4096>);
    if (cudaError_t e = cudaFuncGetAttributes(&fa, mid); e != cudaSuccess) return e;
    if (cudaError_t e = cudaFuncGetAttributes(&fa, half); e != cudaSuccess) return e;
    if (cudaError_t e = ensure_max_dynamic_smem(mid, TK_MAP_MAX_BYTES + 8 * 3072); e != cudaSuccess) return e;
    if (cudaError_t e = ensure_max_dynamic_smem(half, TK_MAP_MAX_BYTES + 8 * 4096); e != cudaSuccess) return e;
    if (cudaError_t e = cudaFuncGetAttributes(&fa, many); e != cudaSuccess) return e;
    if (cudaError_t e = cudaFuncGetAttributes(&fa, few); e != cudaSuccess) return e;
    if (cudaError_t e = ensure_max_dynamic_smem(many, TK_MAP_MAX_BYTES + 8 * kCapMany); e != cudaSuccess) return e;
    return ensure_max_dynamic_smem(few, TK_MAP_MAX_BYTES + 8 * kCapFew);
}

namespace {

constexpr int kCapMid = 3072, kCapHalf = 4096;
// Row lengths at which the next larger instance reads faster (8192 rows of one length, B200): 128 threads x 8 CTAs per SM
// reads 2.3-2.6 TB/s up to 16K scores per row and falls off beyond (too few loads in flight per row: 1.8 TB/s at 64K,
// 1.4 TB/s at 128K); 256 threads x 4 reads 2.6-3.9 TB/s from 20K to 56K; 512 threads x 2 reads 3.3-3.5 TB/s from 64K on;
// 1024 threads x 1 is for launches of so few rows that the SMs would not fill otherwise.
constexpr int64_t kLenMid = 20480, kLenHalf = 61440;

cudaError_t launch_by_length(const float* scores, int64_t ld, int64_t n_rows, int64_t first_len, int64_t len_step,
                             const int32_t* lens, int k_top, int32_t* out, int64_t longest, int64_t typical_len, cudaStream_t stream,
                             const uint8_t* row_mask) {
    int64_t map_bytes = (longest + 127) / 128 * 32;
    if (map_bytes > TK_MAP_MAX_BYTES) map_bytes = TK_MAP_MAX_BYTES;
    const int mb = static_cast<int>(map_bytes);
    if (n_rows < 296)
        return launch_instance<1024, 1, kCapFew>(scores, ld, n_rows, first_len, len_step, lens, k_top, out, mb, stream, row_mask);
    if (typical_len < kLenMid)
        return launch_instance<128, 8, kCapMany>(scores, ld, n_rows, first_len, len_step, lens, k_top, out, mb, stream, row_mask);
    if (typical_len < kLenHalf)
        return launch_instance<256, 4, kCapMid>(scores, ld, n_rows, first_len, len_step, lens, k_top, out, mb, stream, row_mask);
    return launch_instance<512, 2, kCapHalf>(scores, ld, n_rows, first_len, len_step, lens, k_top, out, mb, stream, row_mask);
}

}  // namespace

cudaError_t launch_topk_rows(const float* scores, int64_t ld, int64_t n_rows, int64_t first_len, int64_t len_step,
                             const int32_t* lens, int k_top, int32_t* out, cudaStream_t stream, const uint8_t* row_mask,
                             int* launches) {
    if (launches) *launches = 0;
    if (n_rows <= 0) return cudaSuccess;
    // the selection map covers the longest row of this launch, rounded up to a whole 128-score block
    int64_t longest = lens ? ld : first_len + (n_rows - 1) * len_step;
    if (longest > ld) longest = ld;
    if (longest < 0) longest = 0;
    if (topk_cluster_applicable(n_rows, longest)) {
        if (launches) *launches = 1;
        return launch_topk_rows_cluster(scores, ld, n_rows, first_len, len_step, lens, k_top, out, longest, stream, row_mask);
    }
    if (lens != nullptr || len_step <= 0 || n_rows < 2048) {
        // lengths on the device, one length for all rows, or few rows: one launch, sized for the longest (mean) row
        if (launches) *launches = 1;
        int64_t typical = lens ? longest : first_len + (n_rows - 1) * len_step / 2;
        if (typical > ld) typical = ld;
        return launch_by_length(scores, ld, n_rows, first_len, len_step, lens, k_top, out, longest, typical, stream, row_mask);
    }
    // Lengths that grow with the row number (a prefill): the rows are cut where the length crosses kLenMid and kLenHalf,
    // and every stretch (of at least 1024 rows) goes to the instance that suits its lengths, as a launch of its own
    // (the rows are independent).
    int64_t cuts[4] = {0, (kLenMid - first_len + len_step - 1) / len_step, (kLenHalf - first_len + len_step - 1) / len_step, n_rows};
    for (int i = 1; i <= 2; ++i) {
        if (cuts[i] < cuts[i - 1]) cuts[i] = cuts[i - 1];
        if (cuts[i] > n_rows) cuts[i] = n_rows;
    }
    // stretches shorter than 1024 rows join their neighbour
    if (cuts[1] - cuts[0] < 1024) cuts[1] = cuts[0];
    if (cuts[3] - cuts[2] < 1024) cuts[2] = cuts[3];
    if (cuts[2] - cuts[1] < 1024) { if (cuts[1] > cuts[0]) cuts[1] = cuts[2]; else cuts[2] = cuts[1]; }
    for (int i = 0; i < 3; ++i) {
        const int64_t r0 = cuts[i], nr = cuts[i + 1] - cuts[i];
        if (nr <= 0) continue;
        const int64_t fl = first_len + r0 * len_step;
        int64_t hi = fl + (nr - 1) * len_step;
        if (hi > ld) hi = ld;
        int64_t typical = fl + (nr - 1) * len_step / 2;
        if (typical > ld) typical = ld;
        if (cudaError_t e = launch_by_length(scores + r0 * ld, ld, nr, fl, len_step, nullptr, k_top, out + r0 * static_cast<int64_t>(k_top), hi,
                                             typical, stream, row_mask ? row_mask + r0 : nullptr);
            e != cudaSuccess)
            return e;
        if (launches) *launches += 1;
    }
    return cudaSuccess;
}

}  // namespace idxc
