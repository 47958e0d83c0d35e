// Top-k select for a FEW LONG rows (decode: one row of up to 128K scores per sequence), Sec. 3
// "Notation" T_t = Top-k(I_t) as in topk.cu, but with one thread-block CLUSTER of 8 CTAs per row so
// that a batch of 8-32 rows fills the GPU. Each CTA owns one eighth of the row; the CTAs exchange
// their results through distributed shared memory:
//   1. every CTA histograms the top 12 key bits of its part                           (cluster sync)
//   2. CTA r sums bins [512r, 512r+512) over the 8 histograms and publishes the total (cluster sync)
//   3. the CTA whose bins hold the k-th largest score finds the threshold bucket b1 and
//      broadcasts it                                                                   (cluster sync)
//   4. every CTA flags its scores above b1 (selected) and inside it (candidates) in a local map
//      and copies its candidates (low key bits, position) into the leader's buffer     (cluster sync)
//   5. the leader finds the exact threshold among the candidates (digits 2 and 3) and the
//      position limit for ties, and broadcasts them                                    (cluster sync)
//   6. every CTA flags its selected candidates, counts its selected positions and
//      publishes the count                                                             (cluster sync)
//   7. every CTA emits its positions at rank (selected in lower parts) + local prefix.
// Same result as the one-CTA kernel: ascending positions, ties to the lowest position.
// Rows whose threshold bucket holds more candidates than the leader's buffer are finished by the
// leader alone with the slow path of topk_common.cuh.
#include <cooperative_groups.h>

#include "kernels.h"
#include "topk_common.cuh"

namespace cg = cooperative_groups;

namespace idxc {
using namespace topk;
namespace {

constexpr int CL_D1 = 12;             // first digit: top 12 key bits
constexpr int TK_BINS1 = 1 << CL_D1;
constexpr int CL_SIZE = 8;            // CTAs per row
constexpr int CL_THREADS = 512;
constexpr int CL_WARPS = CL_THREADS / 32;
constexpr int CL_BINS_PER_RANK = TK_BINS1 / CL_SIZE;      // 512: one bin per thread in the reduction
constexpr int CL_CAP = 4096;          // candidates the leader can hold
constexpr int CL_MAX_PART = 65536;    // scores per CTA the local map can flag (rows up to 524288)
static_assert(CL_BINS_PER_RANK == CL_THREADS, "the bin reduction assigns one bin per thread");

struct ClusterExchange {
    uint32_t red[CL_BINS_PER_RANK];   // my 512 bins summed over the cluster
    uint32_t part_tot[CL_SIZE];       // total of each rank's 512 bins
    uint32_t bcast[4];                // b1, scores above b1, scores inside b1
    uint32_t cand_total;              // leader: candidate slots handed out
    uint32_t cand_base;               // first slot of this CTA's candidates
    uint32_t tsel[2];                 // low 20 key bits of the threshold, position limit for ties
    uint32_t sel_cnt[CL_SIZE];        // selected positions per part
};

__global__ void __launch_bounds__(CL_THREADS, 2)
topk_rows_cluster_kernel(const float* __restrict__ scores, int64_t ld, int64_t n_rows, int64_t first_len, int64_t len_step,
                         const int32_t* __restrict__ lens, int k_top, int32_t* __restrict__ out, int map_bytes) {
    cg::cluster_group cluster = cg::this_cluster();
    __shared__ __align__(16) TopkSmem<CL_WARPS, TK_BINS1> sm;
    __shared__ ClusterExchange ex;
    extern __shared__ uint32_t dyn[];
    uint32_t* sel_map = dyn;                                   // map_bytes: one byte per 4 scores of my part
    uint8_t* sel_bytes = reinterpret_cast<uint8_t*>(sel_map);
    uint32_t* cand_key = dyn + map_bytes / 4;                  // leader only: CL_CAP keys, CL_CAP positions
    uint32_t* cand_idx = cand_key + CL_CAP;
    const unsigned rank = cluster.block_rank();
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int tid = threadIdx.x;
    const uint32_t k = static_cast<uint32_t>(k_top);
    const int64_t n_clusters = gridDim.x / CL_SIZE;
    int slot = 0;

    for (int64_t row = blockIdx.x / CL_SIZE; row < n_rows; row += n_clusters) {
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

        // ---- 1. local histogram of the top 12 key bits
        __syncthreads();
        zero_hist<CL_THREADS>(sm, TK_BINS1);
        if (tid == 0) ex.cand_total = 0u;
        __syncthreads();
        sweep_segment<TK_UNROLL>(src, n, seg_begin, seg_end, lane, [&](const float4& x, int base) {
            const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (base + e < n) atomicAdd(&sm.hist[score_digit1<CL_D1>(xs[e])], 1u);
        });
        cluster.sync();                                                                        // (1)
        // ---- 2. sum my 512 bins over the cluster
        uint32_t v = 0;
#pragma unroll
        for (int r = 0; r < CL_SIZE; ++r) v += cluster.map_shared_rank(sm.hist, r)[rank * CL_BINS_PER_RANK + tid];
        ex.red[tid] = v;
        uint32_t my_total;
        (void)block_excl_scan<CL_WARPS>(v, sm, slot, my_total);
        if (tid < CL_SIZE) cluster.map_shared_rank(ex.part_tot, tid)[rank] = my_total;
        cluster.sync();                                                                        // (2)
        // ---- 3. the CTA whose bins hold the k-th largest score selects the bucket
        uint32_t above_mine = 0;
        for (unsigned r = rank + 1; r < CL_SIZE; ++r) above_mine += ex.part_tot[r];            // higher ranks hold higher bins
        if (above_mine < k && k <= above_mine + my_total) {                                    // block-uniform
            sm.hist[tid] = ex.red[tid];                                                        // remote readers of hist are done
            __syncthreads();
            uint32_t bl, al;
            select_bucket<CL_BINS_PER_RANK, CL_THREADS>(sm, k - above_mine, slot, bl, al);
            if (tid < CL_SIZE) {
                uint32_t* dst = cluster.map_shared_rank(ex.bcast, tid);
                dst[0] = rank * CL_BINS_PER_RANK + bl;
                dst[1] = above_mine + al;
                dst[2] = ex.red[bl];
            }
        }
        cluster.sync();                                                                        // (3)
        const uint32_t b1 = ex.bcast[0];
        const uint32_t c1 = ex.bcast[2];
        const uint32_t need = k - ex.bcast[1];                 // rank inside bucket b1, 1-based
        if (c1 > static_cast<uint32_t>(CL_CAP) || part > map_bytes * 4 || !bucket_is_finite<CL_D1>(b1)) {   // cluster-uniform
            if (rank == 0) slow_path<CL_THREADS, CL_D1>(sm, src, n, b1, need, k, out_row, slot);
            continue;
        }
        // ---- 4. flag my scores above bucket b1 (selected) and inside it (candidates)
        const float lo = key_to_score(b1 << 20);
        const bool has_above = b1 < TK_BINS1 - 1;
        const float hi = key_to_score(has_above ? ((b1 + 1) << 20) : 0xFFFFFFFFu);
        sweep_segment<TK_UNROLL>(src, n, seg_begin, seg_end, lane, [&](const float4& x4, int base) {
            const float x[4] = {x4.x, x4.y, x4.z, x4.w};
            uint32_t flags = 0;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if (base + e >= n || !(x[e] >= lo)) continue;
                flags |= (has_above && x[e] >= hi) ? (1u << e) : (16u << e);
            }
            sel_bytes[(base - pb) >> 2] = static_cast<uint8_t>(flags);
        });
        __syncthreads();
        const int words = (pn + 15) >> 4;
        const int wpt = (words + CL_THREADS - 1) / CL_THREADS;
        const int w0 = tid * wpt < words ? tid * wpt : words;
        const int w1 = w0 + wpt < words ? w0 + wpt : words;
        {
            uint32_t cnt = 0;
            for (int w = w0; w < w1; ++w) cnt += __popc(sel_map[w] & 0xF0F0F0F0u);
            uint32_t mine;
            uint32_t pos = block_excl_scan<CL_WARPS>(cnt, sm, slot, mine);
            if (tid == 0) ex.cand_base = atomicAdd(cluster.map_shared_rank(&ex.cand_total, 0), mine);
            __syncthreads();
            pos += ex.cand_base;
            uint32_t* lk = cluster.map_shared_rank(cand_key, 0);
            uint32_t* li = cluster.map_shared_rank(cand_idx, 0);
            for (int w = w0; w < w1; ++w) {
                uint32_t m = sel_map[w] & 0xF0F0F0F0u;
                while (m) {
                    const int b = __ffs(m) - 1;
                    m &= m - 1;
                    const int idx = pb + 16 * w + 4 * (b >> 3) + (b & 7) - 4;
                    if (pos < static_cast<uint32_t>(CL_CAP)) {
                        lk[pos] = score_key(__ldg(src + idx)) & 0xFFFFFu;
                        li[pos] = static_cast<uint32_t>(idx);
                    }
                    ++pos;
                }
            }
        }
        cluster.sync();                                                                        // (4)
        // ---- 5. the leader finds the exact threshold among the candidates
        if (rank == 0) {
            uint32_t t_low, need_eq, m_eq;
            candidate_select<CL_THREADS, 32 - CL_D1>(sm, cand_key, c1, need, slot, t_low, need_eq, m_eq);
            if (tid == 0) ex.cand_base = 0xFFFFFFFFu;          // reused: position limit for ties (none: take all)
            __syncthreads();
            if (m_eq != need_eq) {                             // ties compete: the need_eq lowest positions win
                for (uint32_t i = tid; i < c1; i += CL_THREADS) {
                    if (cand_key[i] != t_low) continue;
                    uint32_t before = 0;
                    for (uint32_t i2 = 0; i2 < c1; ++i2) before += (cand_key[i2] == t_low) & (cand_idx[i2] < cand_idx[i]);
                    if (before == need_eq - 1) ex.cand_base = cand_idx[i];
                }
            }
            __syncthreads();
            if (tid < CL_SIZE) {
                uint32_t* dst = cluster.map_shared_rank(ex.tsel, tid);
                dst[0] = t_low;
                dst[1] = ex.cand_base;
            }
        }
        cluster.sync();                                                                        // (5)
        const uint32_t t_low = ex.tsel[0], idx_limit = ex.tsel[1];
        // ---- 6. flag my selected candidates; count my selected positions
        uint32_t cnt = 0;
        for (int w = w0; w < w1; ++w) {
            uint32_t word = sel_map[w];
            uint32_t m = word & 0xF0F0F0F0u;
            while (m) {
                const int b = __ffs(m) - 1;
                m &= m - 1;
                const uint32_t idx = static_cast<uint32_t>(pb + 16 * w + 4 * (b >> 3) + (b & 7) - 4);
                const uint32_t low = score_key(__ldg(src + idx)) & 0xFFFFFu;
                if (low > t_low || (low == t_low && idx <= idx_limit)) word |= 1u << (b - 4);
            }
            word &= 0x0F0F0F0Fu;
            sel_map[w] = word;                                 // only this thread touches its words
            cnt += __popc(word);
        }
        uint32_t mine;
        uint32_t rnk = block_excl_scan<CL_WARPS>(cnt, sm, slot, mine);
        if (tid < CL_SIZE) cluster.map_shared_rank(ex.sel_cnt, tid)[rank] = mine;
        cluster.sync();                                                                        // (6)
        // ---- 7. emission
        for (unsigned r = 0; r < rank; ++r) rnk += ex.sel_cnt[r];
        for (int w = w0; w < w1; ++w) {
            uint32_t m = sel_map[w];
            while (m) {
                const int b = __ffs(m) - 1;
                m &= m - 1;
                if (rnk < k) out_row[rnk] = pb + 16 * w + 4 * (b >> 3) + (b & 7);
                ++rnk;
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
                                     const int32_t* lens, int k_top, int32_t* out, int64_t longest, cudaStream_t stream) {
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
    return cudaLaunchKernelEx(&cfg, topk_rows_cluster_kernel, scores, ld, n_rows, first_len, len_step, lens, k_top, out, map_bytes);
}

}  // namespace idxc
