// Pattern tooling on index tensors (the paper's Appendix A, Appendix C and Algorithm 1).
//   * overlap kernel: per query row |T_a n T_b| / (valid entries of T_a), for one pair of index tensors or
//     for every pair of N layers in one launch. One row's entries set bits of a shared-memory bitmap, the other row's
//     entries test them (indices below 131072); rows that reach further are ascending runs merged in shared memory.
//     2 * 4 * k bytes per row pair (the pairs of a row run together: repeats hit the L2).
//   * similarity DP (host): the exact pattern with M Full layers that maximises the summed similarity of
//     the Shared layers to their source layers.
//   * greedy layer selection (host): Algorithm 1 with the caller's loss function.
#include <string>
#include <vector>

#include "../../include/idxc.h"
#include "kernels.h"

namespace idxc {
namespace {

constexpr int OV_THREADS = 256;
constexpr int OV_PER_THREAD = IDXC_MAX_K_TOP / OV_THREADS;      // entries of a row per thread: 8
constexpr int OV_BITMAP_WORDS = 4096;                           // one bit per position below 131072
static_assert(OV_PER_THREAD * OV_THREADS == IDXC_MAX_K_TOP && OV_PER_THREAD % 4 == 0, "a thread holds a row's share in registers");

// grid.x: pair index (fastest, so that the pairs of one row run together and the row's index lists are read from HBM
// once and from the L2 afterwards), grid.y: row blocks (grid-stride). pairs[2p], pairs[2p+1]: layer indices of pair p.
// means[p] accumulates the row ratios (double, atomicAdd); a second, tiny kernel divides by the number of rows: the
// average of Appendix A. row_out (optional, single pair) gets each ratio.
// A thread holds eight consecutive entries of both rows in registers. While T_b's largest entry is below 131072 the
// intersection is counted through a bitmap in shared memory: T_b's entries set their bits, T_a's entries test theirs
// (independent accesses, no search), and every thread clears the words it set, so the bitmap is zero again for the next
// row. Rows that reach further are merged: both rows go to shared memory (over the bitmap, which is cleared afterwards),
// rows being ascending, a thread takes a run of consecutive entries of T_a, finds where the run starts in T_b with one
// binary search and walks both lists together.
__global__ void __launch_bounds__(OV_THREADS)
overlap_kernel(const int32_t* const* __restrict__ layers, const int* __restrict__ pairs, int64_t rows, int k_top,
               double* __restrict__ means, float* __restrict__ row_out) {
    extern __shared__ __align__(16) int32_t sh[];   // the bitmap (OV_BITMAP_WORDS), or row of T_b then row of T_a (k_top each)
    uint32_t* bitmap = reinterpret_cast<uint32_t*>(sh);
    __shared__ int warp_cnt[3][OV_THREADS / 32];    // per warp: hits, valid entries of T_a, largest entry of T_b
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int p = blockIdx.x;
    const int32_t* Ta = layers[pairs[2 * p]];
    const int32_t* Tb = layers[pairs[2 * p + 1]];
    // rows whose bytes start on a 16-byte boundary are read with 128-bit loads
    const bool wide = (k_top & 3) == 0 && ((reinterpret_cast<uintptr_t>(Ta) | reinterpret_cast<uintptr_t>(Tb)) & 15) == 0;
    const int i0 = threadIdx.x * OV_PER_THREAD;     // my entries: [i0, i0 + 8) of both rows
    for (int i = threadIdx.x; i < OV_BITMAP_WORDS; i += OV_THREADS) bitmap[i] = 0u;
    double local_sum = 0.0;
    for (int64_t r = blockIdx.y; r < rows; r += gridDim.y) {
        const int32_t* a = Ta + r * k_top;
        const int32_t* b = Tb + r * k_top;
        int32_t va[OV_PER_THREAD], vb[OV_PER_THREAD];
        if (wide) {
#pragma unroll
            for (int v = 0; v < OV_PER_THREAD / 4; ++v) {
                const int i = i0 + 4 * v;
                const int4 none = make_int4(-1, -1, -1, -1);
                const int4 xa = i < k_top ? __ldg(reinterpret_cast<const int4*>(a + i)) : none;
                const int4 xb = i < k_top ? __ldg(reinterpret_cast<const int4*>(b + i)) : none;
                va[4 * v] = xa.x; va[4 * v + 1] = xa.y; va[4 * v + 2] = xa.z; va[4 * v + 3] = xa.w;
                vb[4 * v] = xb.x; vb[4 * v + 1] = xb.y; vb[4 * v + 2] = xb.z; vb[4 * v + 3] = xb.w;
            }
        } else {
#pragma unroll
            for (int e = 0; e < OV_PER_THREAD; ++e) {
                va[e] = i0 + e < k_top ? __ldg(a + i0 + e) : -1;
                vb[e] = i0 + e < k_top ? __ldg(b + i0 + e) : -1;
            }
        }
        int na = 0, top_b = -1;
#pragma unroll
        for (int e = 0; e < OV_PER_THREAD; ++e) {
            na += va[e] >= 0;
            top_b = vb[e] > top_b ? vb[e] : top_b;
        }
        na = __reduce_add_sync(0xFFFFFFFFu, na);
        top_b = __reduce_max_sync(0xFFFFFFFFu, top_b);
        if (lane == 0) { warp_cnt[1][wid] = na; warp_cnt[2][wid] = top_b; }
        __syncthreads();                              // (1) also: the previous row's bitmap words are cleared
        na = 0; top_b = -1;
#pragma unroll
        for (int w = 0; w < OV_THREADS / 32; ++w) {
            na += warp_cnt[1][w];
            top_b = warp_cnt[2][w] > top_b ? warp_cnt[2][w] : top_b;
        }
        int hits = 0;
        if (top_b < OV_BITMAP_WORDS * 32) {           // block-uniform
#pragma unroll
            for (int e = 0; e < OV_PER_THREAD; ++e)
                if (vb[e] >= 0) atomicOr(&bitmap[vb[e] >> 5], 1u << (vb[e] & 31));
            __syncthreads();                          // (2)
#pragma unroll
            for (int e = 0; e < OV_PER_THREAD; ++e)
                if (va[e] >= 0 && va[e] <= top_b) hits += (bitmap[va[e] >> 5] >> (va[e] & 31)) & 1u;
        } else {
            int32_t* sb = sh;
            int32_t* sa = sh + k_top;
            int nb = 0;
#pragma unroll
            for (int e = 0; e < OV_PER_THREAD; ++e) {
                if (i0 + e < k_top) { sb[i0 + e] = vb[e]; sa[i0 + e] = va[e]; }
                nb += vb[e] >= 0;
            }
            nb = __reduce_add_sync(0xFFFFFFFFu, nb);
            if (lane == 0) warp_cnt[0][wid] = nb;
            __syncthreads();
            nb = 0;
#pragma unroll
            for (int w = 0; w < OV_THREADS / 32; ++w) nb += warp_cnt[0][w];
            const int i1 = i0 + OV_PER_THREAD < na ? i0 + OV_PER_THREAD : na;   // valid entries come first (padding is at the end)
            if (i0 < i1) {
                const int32_t first = sa[i0];
                int lo = 0, hi = nb;                  // first position with sb[pos] >= first
                while (lo < hi) {
                    const int mid = (lo + hi) >> 1;
                    if (sb[mid] < first) lo = mid + 1; else hi = mid;
                }
                int j = lo;
                for (int i = i0; i < i1 && j < nb; ++i) {
                    const int32_t v = sa[i];
                    while (j < nb && sb[j] < v) ++j;
                    hits += (j < nb && sb[j] == v);
                }
            }
            __syncthreads();                          // every walk is done before the rows are wiped
        }
        hits = __reduce_add_sync(0xFFFFFFFFu, hits);
        __syncthreads();                              // (3) warp_cnt[0] of the merge path has been read; the bit tests are done
        if (lane == 0) warp_cnt[0][wid] = hits;
        if (top_b < OV_BITMAP_WORDS * 32) {           // the words I set are zero again before the next row sets its bits
#pragma unroll
            for (int e = 0; e < OV_PER_THREAD; ++e)
                if (vb[e] >= 0) bitmap[vb[e] >> 5] = 0u;
        } else {
            for (int i = threadIdx.x; i < OV_BITMAP_WORDS; i += OV_THREADS) bitmap[i] = 0u;
        }
        __syncthreads();                              // (4)
        if (threadIdx.x == 0) {
            int h = 0;
            for (int w = 0; w < OV_THREADS / 32; ++w) h += warp_cnt[0][w];
            const double ratio = na ? static_cast<double>(h) / na : 0.0;
            local_sum += ratio;
            if (row_out) row_out[r] = static_cast<float>(ratio);
        }
    }
    if (threadIdx.x == 0) atomicAdd(&means[p], local_sum);
}

__global__ void overlap_mean_kernel(double* __restrict__ means, int n_pairs, double rows) {
    const int p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p < n_pairs) means[p] /= rows;
}

}  // namespace

cudaError_t launch_overlap(const int32_t* const* layers_dev, const int* pairs_dev, int n_pairs, int64_t rows, int k_top,
                           double* sums_dev, float* row_out, cudaStream_t stream) {
    if (n_pairs <= 0 || rows <= 0) return cudaSuccess;
    const unsigned gy = static_cast<unsigned>(rows < 4096 ? rows : 4096);
    dim3 grid(static_cast<unsigned>(n_pairs), gy);
    const size_t rows_bytes = 2 * static_cast<size_t>(k_top) * sizeof(int32_t), map_bytes = OV_BITMAP_WORDS * sizeof(uint32_t);
    overlap_kernel<<<grid, OV_THREADS, rows_bytes > map_bytes ? rows_bytes : map_bytes, stream>>>(layers_dev, pairs_dev, rows, k_top, sums_dev, row_out);
    if (cudaError_t e = cudaGetLastError(); e != cudaSuccess) return e;
    overlap_mean_kernel<<<(n_pairs + 255) / 256, 256, 0, stream>>>(sums_dev, n_pairs, static_cast<double>(rows));
    return cudaGetLastError();
}

}  // namespace idxc

using namespace idxc;

extern "C" {

idxc_status idxc_topk_overlap(const int32_t* const* layers, const int32_t* pairs, int n_pairs, int64_t rows, int k_top,
                              double* sums_out, float* row_out, void* cuda_stream) {
    if (n_pairs < 0 || rows < 0 || k_top < 1 || k_top > IDXC_MAX_K_TOP) return IDXC_ERR_INVALID_ARG;
    if (n_pairs == 0 || rows == 0) return IDXC_OK;
    if (!layers || !pairs || !sums_out) return IDXC_ERR_INVALID_ARG;
    if (row_out && n_pairs != 1) return IDXC_ERR_INVALID_ARG;
    if (n_pairs > 65535) return IDXC_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemsetAsync(sums_out, 0, sizeof(double) * n_pairs, stream) != cudaSuccess) return IDXC_ERR_CUDA;
    return launch_overlap(layers, pairs, n_pairs, rows, k_top, sums_out, row_out, stream) == cudaSuccess ? IDXC_OK
                                                                                                          : IDXC_ERR_CUDA;
}

// Appendix C: dp[i][m] = best total similarity of layers 0..i with m Full layers, layer i Full.
idxc_status idxc_pattern_search_dp(const double* S, int N, int M, char* pattern_out, double* value_out) {
    if (!S || !pattern_out || N < 1 || M < 1 || M > N) return IDXC_ERR_INVALID_ARG;
    const double NEG = -1e300;
    // seg[j][i] = sum_{t=j+1}^{i-1} S[t][j]: the Shared layers between Full layers j and i (i == N: to the end)
    std::vector<std::vector<double>> seg(N, std::vector<double>(N + 1, 0.0));
    for (int j = 0; j < N; ++j) {
        double run = 0.0;
        for (int i = j + 1; i <= N; ++i) {
            seg[j][i] = run;
            if (i < N) run += S[static_cast<size_t>(i) * N + j];
        }
    }
    std::vector<std::vector<double>> dp(N, std::vector<double>(M + 1, NEG));
    std::vector<std::vector<int>> prev(N, std::vector<int>(M + 1, -1));
    dp[0][1] = 0.0;                                  // the first layer is always Full
    for (int i = 1; i < N; ++i)
        for (int m = 2; m <= M && m <= i + 1; ++m)
            for (int j = m - 2; j < i; ++j) {
                if (dp[j][m - 1] <= NEG) continue;
                const double v = dp[j][m - 1] + seg[j][i];
                if (v > dp[i][m]) { dp[i][m] = v; prev[i][m] = j; }
            }
    double best = NEG;
    int last = -1;
    for (int i = M - 1; i < N; ++i) {
        if (dp[i][M] <= NEG) continue;
        const double v = dp[i][M] + seg[i][N];
        if (v > best) { best = v; last = i; }
    }
    if (last < 0) return IDXC_ERR_INVALID_ARG;
    for (int l = 0; l < N; ++l) pattern_out[l] = 'S';
    for (int i = last, m = M; i >= 0 && m >= 1; i = prev[i][m], --m) {
        pattern_out[i] = 'F';
        if (prev[i][m] < 0) break;
    }
    if (value_out) *value_out = best;
    return IDXC_OK;
}

// Greedy layer selection (Algorithm 1): from the all-Full pattern, K times turn into a Shared layer the still-Full
// layer (never layer 0) whose conversion leaves the lowest loss. State is one pattern buffer in which a trial is a
// single character flipped and restored; the lowest trial of a step wins, the lowest layer among equal losses.
idxc_status idxc_pattern_search_greedy(int N, int K, idxc_eval_loss_fn eval_loss, void* user, char* pattern_out,
                                       int* order_out, double* step_loss_out, int64_t* evaluations_out) {
    if (N < 1 || K < 0 || K > N - 1 || !eval_loss || !pattern_out) return IDXC_ERR_INVALID_ARG;
    std::string pattern(static_cast<size_t>(N), 'F');            // NUL-terminated through c_str()
    int64_t evals = 0;
    for (int step = 0; step < K; ++step) {
        int winner = -1;
        double winner_loss = 0.0;
        for (int l = 1; l < N; ++l) {
            if (pattern[l] != 'F') continue;                     // already Shared
            pattern[l] = 'S';
            const double loss = eval_loss(pattern.c_str(), N, user);
            pattern[l] = 'F';
            ++evals;
            if (winner < 0 || loss < winner_loss) { winner = l; winner_loss = loss; }
        }
        pattern[winner] = 'S';                                   // K <= N - 1: a Full layer other than 0 is always left
        if (order_out) order_out[step] = winner;
        if (step_loss_out) step_loss_out[step] = winner_loss;
    }
    pattern.copy(pattern_out, static_cast<size_t>(N));
    if (evaluations_out) *evaluations_out = evals;
    return IDXC_OK;
}

}  // extern "C"
