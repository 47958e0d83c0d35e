// Top-k select for a FEW LONG rows (decode: one row of up to 128K scores per sequence), Sec. 3
// "Notation" T_t = Top-k(I_t) as in topk.cu, but with one thread-block CLUSTER of 8 CTAs per row so
// that a batch of 8-32 rows fills the GPU. Same one-sweep algorithm as the row kernel; each CTA owns one
// eighth of the row and the CTAs exchange their counts through distributed shared memory:
//   1. every CTA samples the WHOLE row and derives the same two pivot scores (identical arithmetic on identical
//      data: no exchange needed), then sweeps its own part once: scores at or above the upper pivot are flagged
//      in a local map, scores between the pivots are candidates; it publishes its two counts   (cluster sync)
//   2. with A scores above and C candidates over the cluster the bracket held iff A < k <= A + C. Every CTA sorts
//      its candidates into 1024 finer bins across the band                                    (cluster sync)
//   3. every CTA adds the eight histograms up, finds the bin of the wanted rank, flags its candidates in higher
//      bins and appends those inside that bin (a handful) to a list in the leader              (cluster sync)
//   4. every CTA ranks that list by direct comparison of the 32-bit keys (larger key first, lower position first
//      among equal keys), flags its own winners, counts its selected positions and publishes   (cluster sync)
//   5. every CTA emits its positions at rank (selected in lower parts) + local prefix.
// Same result as the one-CTA kernel: ascending positions, ties to the lowest position. Rows the fast path cannot
// separate (bracket missed, crowded threshold bin, a list overflow, constant or non-finite sample, parts longer
// than the map) are selected by the leader alone on keys (slow_path_full of topk_common.cuh).
#include <cooperative_groups.h>

#include "kernels.h"
#include "topk_common.cuh"

namespace cg = cooperative_groups;

namespace idxc {
using namespace topk;
namespace {

constexpr int CL_SIZE = 8;            // CTAs per row
constexpr int CL_THREADS = 512;
constexpr int CL_WARPS = CL_THREADS / 32;
constexpr int CL_BINS = 1024;         // bins of the sample histogram and of the finer candidate histogram
constexpr int CL_CAP = 1024;          // candidates one CTA can list
constexpr int CL_SMALL = 128;         // scores ranked by direct comparison at most
constexpr int CL_MAX_PART = 65536;    // scores per CTA the local map can flag (rows up to 524288)
constexpr int U = TK_UNROLL;

// The per-rank counts are written by the other CTAs of the cluster. They exist twice and successive rows alternate
// between the copies: a CTA that has run ahead into the next row then never writes into counts a slower CTA is still
// reading (it cannot get two rows ahead: every row has a cluster barrier).
struct ClusterExchange {
    uint32_t part_a[2][CL_SIZE];      // scores above the band, per rank (every CTA holds all eight)
    uint32_t part_c[2][CL_SIZE];      // candidates, per rank
    uint32_t sel_cnt[2][CL_SIZE];     // selected positions, per rank
    uint32_t small_count;             // leader: entries of the list below
    uint32_t small_key[CL_SMALL];     // leader: keys and positions of the candidates inside the threshold bin
    uint32_t small_idx[CL_SMALL];
};

struct ClusterRowSmem : SampleSmem {
    uint32_t warp_cnt[2][CL_WARPS];
    uint32_t cand_count;
};

__global__ void __launch_bounds__(CL_THREADS, 2)
topk_rows_cluster_kernel(const float* __restrict__ scores, int64_t ld, int64_t n_rows, int64_t first_len, int64_t len_step,
                         const int32_t* __restrict__ lens, int k_top, int32_t* __restrict__ out, int map_bytes,
                         const uint8_t* __restrict__ row_mask) {
    cg::cluster_group cluster = cg::this_cluster();
    __shared__ __align__(16) TopkSmem<CL_WARPS, 2048> sm;      // [0, 1024): sample histogram, then the summed fine histogram;
                                                               // [1024, 2048): this CTA's fine histogram; all 2048: keys-only path
    __shared__ ClusterRowSmem rs;
    __shared__ ClusterExchange ex;
    extern __shared__ uint32_t dyn[];
    uint32_t* sel_map = dyn;                                   // map_bytes: one byte per 4 scores of my part
    uint8_t* sel_bytes = reinterpret_cast<uint8_t*>(sel_map);
    uint32_t* cand_fb = dyn + map_bytes / 4;                   // my candidates: fine bin ...
    uint32_t* cand_idx = cand_fb + CL_CAP;                     // ... and position in the row
    const unsigned rank = cluster.block_rank();
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int tid = threadIdx.x;
    const uint32_t k = static_cast<uint32_t>(k_top);
    const int64_t n_clusters = gridDim.x / CL_SIZE;
    int slot = 0;

    int par = 1;
    for (int64_t row = blockIdx.x / CL_SIZE; row < n_rows; row += n_clusters) {
        if (row_mask != nullptr && row_mask[row] == 0) continue;      // the same for every CTA of the cluster
        par ^= 1;                                              // which copy of the exchanged counts this row uses
        int64_t len = lens ? static_cast<int64_t>(lens[row]) : first_len + row * len_step;
        len = len < 0 ? 0 : (len > ld ? ld : len);
        const int n = static_cast<int>(len);
        int32_t* out_row = out + row * static_cast<int64_t>(k_top);
        if (n <= k_top) {                                      // the same for every CTA of the cluster
            if (rank == 0)
                for (int j = tid; j < k_top; j += CL_THREADS) out_row[j] = j < n ? j : -1;
            continue;
        }
        const float* src = scores + row * ld;
        // my part of the row and my warp's segment of it, both multiples of 128 scores
        const int part = (((n + CL_SIZE - 1) / CL_SIZE) + 127) & ~127;
        const int pb = static_cast<int>(rank) * part < n ? static_cast<int>(rank) * part : n;
        const int pe = pb + part < n ? pb + part : n;
        const int pn = pe - pb;
        const int seg = (((pn + CL_WARPS - 1) / CL_WARPS) + 127) & ~127;
        const int seg_begin = pb + (wid * seg < pn ? wid * seg : pn);
        const int seg_end = seg_begin + seg < pe ? seg_begin + seg : pe;
        if (part > map_bytes * 4) {                            // cluster-uniform: parts longer than the map
            if (rank == 0) slow_path_full<CL_THREADS>(sm, src, n, k, out_row, slot);
            continue;
        }
        // ---- 1. pivots from a sample of the whole row (the same in every CTA), then one sweep over my part
        __syncthreads();                                       // earlier readers of sm, rs and the map are done
        if (tid == 0) { rs.cand_count = 0u; if (rank == 0) ex.small_count = 0u; }
        const Pivots pv = sample_pivots<CL_THREADS, CL_BINS>(sm, rs, src, n, k_top, slot);
        if (!pv.usable) {                                      // cluster-uniform
            if (rank == 0) slow_path_full<CL_THREADS>(sm, src, n, k, out_row, slot);
            continue;
        }
        {
            const float lo_x = pv.lo_x, hi_x = pv.hi_x;
            const int full_end = seg_begin + (seg_end - seg_begin) / (128 * U) * (128 * U);
            const float* p = src + seg_begin + 4 * lane;
            uint8_t* mb = sel_bytes + ((seg_begin - pb) >> 2) + lane;
            int cb = seg_begin;
            for (; cb < full_end; cb += 128 * U, p += 128 * U, mb += 32 * U) {
                float4 x4[U];
#pragma unroll
                for (int u = 0; u < U; ++u) x4[u] = __ldg(reinterpret_cast<const float4*>(p + 128 * u));
#pragma unroll
                for (int u = 0; u < U; ++u) mb[32 * u] = static_cast<uint8_t>(flag4(x4[u], lo_x, hi_x));
            }
            for (; cb < seg_end; cb += 128) {                  // the ragged rest, one block at a time
                const int base = cb + 4 * lane;
                uint32_t flags = 0;
                if (base < n) {
                    flags = flag4(__ldg(reinterpret_cast<const float4*>(src + base)), lo_x, hi_x);
                    const int left = n - base;                 // scores of this 128-bit load inside the row
                    if (left < 4) flags &= (0x11u << left) - 0x11u;
                }
                sel_bytes[(base - pb) >> 2] = static_cast<uint8_t>(flags);
            }
        }
        __syncwarp();
        // my warp's map words, and every lane's run of them
        const int w_begin = (seg_begin - pb) >> 4, w_end = seg_begin < seg_end ? (seg_end - pb + 15) >> 4 : w_begin;
        const int wpl = (w_end - w_begin + 31) >> 5;
        const int lw0 = w_begin + lane * wpl < w_end ? w_begin + lane * wpl : w_end;
        const int lw1 = lw0 + wpl < w_end ? lw0 + wpl : w_end;
        uint32_t my_cand = 0;                                  // candidates in this lane's run
        {
            uint32_t n_sel = 0;
            for (int w = lw0; w < lw1; ++w) {
                const uint32_t m = sel_map[w];
                n_sel += __popc(m & 0x0F0F0F0Fu);
                my_cand += __popc(m & 0xF0F0F0F0u);
            }
            n_sel = __reduce_add_sync(0xFFFFFFFFu, n_sel);
            const uint32_t n_cand = __reduce_add_sync(0xFFFFFFFFu, my_cand);
            if (lane == 0) { rs.warp_cnt[0][wid] = n_sel; rs.warp_cnt[1][wid] = n_cand; }
        }
        __syncthreads();
        if (tid < CL_SIZE) {                                   // publish my two counts in every CTA of the cluster
            uint32_t a = 0, c = 0;
#pragma unroll
            for (int w = 0; w < CL_WARPS; ++w) { a += rs.warp_cnt[0][w]; c += rs.warp_cnt[1][w]; }
            cluster.map_shared_rank(ex.part_a[par], tid)[rank] = a;
            cluster.map_shared_rank(ex.part_c[par], tid)[rank] = c;
        }
        cluster.sync();                                                                        // (1)
        uint32_t A = 0, C = 0, c_max = 0;
#pragma unroll
        for (int r = 0; r < CL_SIZE; ++r) {
            A += ex.part_a[par][r];
            C += ex.part_c[par][r];
            c_max = ex.part_c[par][r] > c_max ? ex.part_c[par][r] : c_max;
        }
        if (!(A < k && k - A <= C && c_max <= static_cast<uint32_t>(CL_CAP))) {                // cluster-uniform
            if (rank == 0) slow_path_full<CL_THREADS>(sm, src, n, k, out_row, slot);
            continue;
        }
        const uint32_t need = k - A;                           // candidates to take, 1..C
        // ---- 2. list my candidates, sort them into the finer bins
        for (int i = tid; i < CL_BINS; i += CL_THREADS) sm.hist[CL_BINS + i] = 0u;
        const uint32_t my_c = ex.part_c[par][rank];
        {
            uint32_t total;
            uint32_t pos = warp_excl_scan(my_cand, lane, total);
            uint32_t basepos = 0;
            if (lane == 0 && total != 0u) basepos = atomicAdd(&rs.cand_count, total);
            pos += __shfl_sync(0xFFFFFFFFu, basepos, 0);
            for (int w = lw0; w < lw1; ++w) {
                uint32_t m = squeeze_nibbles(sel_map[w] >> 4);
                const uint32_t idx0 = static_cast<uint32_t>(pb) + 16u * static_cast<uint32_t>(w);
                while (m) {
                    const uint32_t b = __ffs(m) - 1;
                    m &= m - 1;
                    if (pos < static_cast<uint32_t>(CL_CAP)) cand_idx[pos] = idx0 + b;
                    ++pos;
                }
            }
        }
        __syncthreads();
        for (uint32_t i = tid; i < my_c; i += CL_THREADS) {    // independent loads (L2), all in flight together
            const uint32_t fb = pv.fine_bin<CL_BINS>(__ldg(src + cand_idx[i]));
            cand_fb[i] = fb;
            atomicAdd(&sm.hist[CL_BINS + fb], 1u);
        }
        cluster.sync();                                                                        // (2)
        // ---- 3. the summed histogram, the bin of the wanted rank
        for (int i = tid; i < CL_BINS; i += CL_THREADS) {
            uint32_t v = 0;
#pragma unroll
            for (int r = 0; r < CL_SIZE; ++r) v += cluster.map_shared_rank(sm.hist, r)[CL_BINS + i];
            sm.hist[i] = v;
        }
        __syncthreads();
        uint32_t fb1, above_f;
        select_bucket<CL_BINS, CL_THREADS>(sm, need, slot, fb1, above_f);
        const uint32_t m1 = sm.hist[fb1];
        const uint32_t need1 = need - above_f;                 // scores to take from fine bin fb1, 1..m1
        if (m1 <= static_cast<uint32_t>(CL_SMALL)) {
            uint32_t* l_count = cluster.map_shared_rank(&ex.small_count, 0);
            uint32_t* l_key = cluster.map_shared_rank(ex.small_key, 0);
            uint32_t* l_idx = cluster.map_shared_rank(ex.small_idx, 0);
            for (uint32_t i = tid; i < my_c; i += CL_THREADS) {
                const uint32_t fb = cand_fb[i];
                const uint32_t idx = cand_idx[i];
                if (fb > fb1) {
                    flag_selected(sel_map, idx - static_cast<uint32_t>(pb));
                } else if (fb == fb1) {
                    const uint32_t pos = atomicAdd(l_count, 1u);
                    if (pos < static_cast<uint32_t>(CL_SMALL)) { l_key[pos] = score_key(__ldg(src + idx)); l_idx[pos] = idx; }
                }
            }
        }
        cluster.sync();                                                                        // (3)
        if (m1 > static_cast<uint32_t>(CL_SMALL)) {            // cluster-uniform: many near-equal scores at the threshold
            if (rank == 0) slow_path_full<CL_THREADS>(sm, src, n, k, out_row, slot);
            continue;
        }
        // ---- 4. rank the listed scores; flag my winners; count my selected positions
        {
            const uint32_t* l_key = cluster.map_shared_rank(ex.small_key, 0);
            const uint32_t* l_idx = cluster.map_shared_rank(ex.small_idx, 0);
            for (uint32_t i = tid; i < m1; i += CL_THREADS) {
                const uint32_t ki = l_key[i], ii = l_idx[i];
                if (ii < static_cast<uint32_t>(pb) || ii >= static_cast<uint32_t>(pe)) continue;      // not mine
                uint32_t beaten_by = 0;
                for (uint32_t j = 0; j < m1; ++j) {
                    const uint32_t kj = l_key[j], ij = l_idx[j];
                    beaten_by += (kj > ki) | ((kj == ki) & (ij < ii));
                }
                if (beaten_by < need1) flag_selected(sel_map, ii - static_cast<uint32_t>(pb));
            }
        }
        __syncthreads();
        uint32_t c_sel = 0;
        for (int w = lw0; w < lw1; ++w) c_sel += __popc(sel_map[w] & 0x0F0F0F0Fu);
        uint32_t w_total;
        uint32_t pos = warp_excl_scan(c_sel, lane, w_total);
        if (lane == 0) rs.warp_cnt[0][wid] = w_total;
        __syncthreads();
        if (tid < CL_SIZE) {
            uint32_t s = 0;
#pragma unroll
            for (int w = 0; w < CL_WARPS; ++w) s += rs.warp_cnt[0][w];
            cluster.map_shared_rank(ex.sel_cnt[par], tid)[rank] = s;
        }
        cluster.sync();                                                                        // (4)
        // ---- 5. emission
        for (unsigned r = 0; r < rank; ++r) pos += ex.sel_cnt[par][r];
#pragma unroll
        for (int w = 0; w < CL_WARPS; ++w) pos += w < wid ? rs.warp_cnt[0][w] : 0u;
        for (int w = lw0; w < lw1; ++w) {
            uint32_t m = squeeze_nibbles(sel_map[w]);
            const int idx0 = pb + 16 * w;
            while (m) {
                const int b = __ffs(m) - 1;
                m &= m - 1;
                if (pos < k) out_row[pos] = idx0 + b;
                ++pos;
            }
        }
    }
    cluster.sync();        // no CTA leaves while another may still address its shared memory
}

}  // namespace

cudaError_t preload_topk_rows_cluster() {
    cudaFuncAttributes fa;
    if (cudaError_t e = cudaFuncGetAttributes(&fa, reinterpret_cast<const void*>(topk_rows_cluster_kernel)); e != cudaSuccess) return e;
    return ensure_max_dynamic_smem(reinterpret_cast<const void*>(topk_rows_cluster_kernel), CL_MAX_PART / 4 + 2 * CL_CAP * 4);
}

bool topk_cluster_applicable(int64_t n_rows, int64_t longest) {
    return n_rows >= 1 && n_rows <= 128 && longest >= 16384 && longest <= static_cast<int64_t>(CL_MAX_PART) * CL_SIZE;
}

cudaError_t launch_topk_rows_cluster(const float* scores, int64_t ld, int64_t n_rows, int64_t first_len, int64_t len_step,
                                     const int32_t* lens, int k_top, int32_t* out, int64_t longest, cudaStream_t stream,
                                     const uint8_t* row_mask) {
    const int64_t part = (((longest + CL_SIZE - 1) / CL_SIZE) + 127) & ~int64_t(127);
    const int map_bytes = static_cast<int>(part / 4);
    const int dyn_bytes = map_bytes + 2 * CL_CAP * 4;
    if (cudaError_t e = ensure_max_dynamic_smem(reinterpret_cast<const void*>(topk_rows_cluster_kernel), CL_MAX_PART / 4 + 2 * CL_CAP * 4); e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(n_rows * CL_SIZE));
    cfg.blockDim = dim3(CL_THREADS);
    cfg.dynamicSmemBytes = dyn_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CL_SIZE;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, topk_rows_cluster_kernel, scores, ld, n_rows, first_len, len_step, lens, k_top, out, map_bytes, row_mask);
}

}  // namespace idxc
