// Internal launch interface between the C-ABI layer (api.cu) and the kernel files.
// Every launcher enqueues on `stream` and returns the CUDA error of the launch.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace idxc {

// Raises a kernel's dynamic shared-memory limit to `bytes` once per (kernel, device); thread-safe (api.cu).
cudaError_t ensure_max_dynamic_smem(const void* kernel, int bytes);

// Row-wise top-k select (topk.cu). Row r has length lens[r] (device) if lens != nullptr,
// else first_len + r * len_step, clamped to [0, ld]. row_mask: nullptr, or one byte per row: rows whose byte is 0 are
// left alone (neither read nor written). launches: if given, receives the number of kernels launched (rows whose lengths
// grow with the row number go out in up to three launches, one per range of lengths).
cudaError_t launch_topk_rows(const float* scores, int64_t ld, int64_t n_rows, int64_t first_len,
                             int64_t len_step, const int32_t* lens, int k_top, int32_t* out,
                             cudaStream_t stream, const uint8_t* row_mask = nullptr, int* launches = nullptr);

// Cluster variant for a few long rows (topk_cluster.cu): 8 CTAs per row exchanging through
// distributed shared memory. `longest` = longest row of the launch.
bool topk_cluster_applicable(int64_t n_rows, int64_t longest);
cudaError_t launch_topk_rows_cluster(const float* scores, int64_t ld, int64_t n_rows, int64_t first_len,
                                     int64_t len_step, const int32_t* lens, int k_top, int32_t* out,
                                     int64_t longest, cudaStream_t stream, const uint8_t* row_mask = nullptr);

// Streaming top-k of the prefill scorer (the score write replaced by a filtered candidate list per query row):
// the scorer visits a strided sample of a work item's key tiles first, takes from each row's sample a threshold that
// with high probability lies below the row's k_top-th largest score, and from then on appends only the (score, key
// index) pairs at or above the threshold. finish_topk_stream (topk_stream.cu) takes the exact top-k of each list,
// or flags the row (threshold too high after all, or a list overflow) for the ordinary score + select path.
// A row's list is kStreamRowSlots pairs (x = score bits, y = key index): first the sample's own scores at or above the
// threshold (up to kStreamSampleCap), then 128 lists of kStreamLaneCap slots, one per scorer thread that sees keys of the
// row (TMEM lane quarter * 32 + lane): a thread appends at a position it keeps in a register, with no vote or atomic.
constexpr int kStreamSampleCap = 1024;
constexpr int kStreamLaneCap = 64;
constexpr int kStreamLanes = 128;
constexpr int kStreamRowSlots = kStreamSampleCap + kStreamLanes * kStreamLaneCap;   // 9216 pairs = 72 KB per row
constexpr int kStreamMaxKeys = 262144;      // longest row the second half's position bitmap covers
struct StreamTopk {
    uint2* cand;            // [n_rows, kStreamRowSlots]; nullptr: ordinary score write
    uint32_t* sample_count; // [n_rows] pairs in the sample part
    uint8_t* lane_count;    // [n_rows, kStreamLanes] pairs appended by each thread, saturating at 255 (> kStreamLaneCap: overflow)
    float* tau;             // [n_rows] the row's threshold (-inf: none)
    int k_top;
};

// topk_stream.cu: exact top-k of every row's candidate list into out [n_rows, k_top] (ascending key indices, -1
// padding), or row_fail[row] = 1 where the list cannot give it; item_fail[b] = 1 where block b of rows_per_item rows
// holds a flagged row (both arrays are written in full).
cudaError_t launch_finish_topk_stream(const StreamTopk& st, int64_t n_rows, int64_t q_begin, int rows_per_item, int32_t* out,
                                      uint8_t* row_fail, uint8_t* item_fail, cudaStream_t stream);

// Arguments shared by the scorers. A "row" is one query vector set [H, d].
struct ScoreArgs {
    const void* q;          // [n_rows, H, d]
    const void* k;          // [k_rows, d]
    const float* w;         // [n_rows, H]
    const float* q_scale;   // [n_rows] or nullptr
    const float* k_scale;   // [k_rows] or nullptr
    const int64_t* k_offsets;  // decode: [n_rows] first key row of each sequence; prefill: nullptr
    const int32_t* lens;       // decode: [n_rows] keys per sequence; prefill: nullptr
    int64_t q_begin;        // prefill: position of row 0 (row r sees keys 0 .. q_begin + r)
    int64_t n_rows;
    int64_t k_rows;         // rows of k that may be addressed
    int64_t max_len;        // decode: host bound on lens
    int H, d;
    int fp8;                // 0: bf16, 1: e4m3 codes with scales
    float* scores;          // [n_rows, ld]
    int64_t ld;
    StreamTopk stream;      // prefill only; cand == nullptr: scores are written
    const uint8_t* item_mask;   // prefill only: nullptr, or one byte per block of rows_per_item rows: 0 = skip the block
};

// Plain CUDA-core scorer (scorer_simt.cu): debugging aid and cross-check.
cudaError_t launch_score_simt(const ScoreArgs& a, cudaStream_t stream);
// -inf into columns q_begin + r + 1 .. n_cols - 1 of every row r (the causal mask, IDXC_FLAG_FILL_MASKED).
cudaError_t launch_fill_masked(float* scores, int64_t ld, int64_t q_begin, int64_t n_rows, int64_t n_cols, cudaStream_t stream);

// tcgen05 scorers (scorer_tc.cu). `status` is the device status word. The tensor maps are
// encoded by the caller: q as [n_rows*H, d] and k as [k_rows, d], 128-byte swizzle, inner
// box 128 bytes, box rows 256 (q) and 128 (k) for prefill; box rows H (q) for decode.
cudaError_t launch_score_prefill_tc(const ScoreArgs& a, const CUtensorMap& q_map, const CUtensorMap& k_map,
                                    unsigned int* status, int sm_count, cudaStream_t stream);
cudaError_t launch_score_decode_tc(const ScoreArgs& a, const CUtensorMap& q_map, const CUtensorMap& k_map,
                                   unsigned int* status, int sm_count, cudaStream_t stream);
bool score_tc_supported(int H, int d, int fp8);
// Streaming top-k is built for the shapes whose work item leaves room for the sample (scorer_tc.cu).
bool score_prefill_stream_supported(int H, int d, int fp8);
// Query rows per work item of the prefill scorer (the granularity of item_mask).
int score_prefill_rows_per_item(int H);
// Load every kernel a decode step can launch on the current device and set its attributes (scorer_tc.cu, topk.cu,
// topk_cluster.cu, scorer_simt.cu), so that later launches find them resident.
cudaError_t preload_score_decode_tc();
cudaError_t preload_topk_rows();
cudaError_t preload_topk_rows_cluster();
cudaError_t preload_score_simt();

// quantize.cu: per-token e4m3 quantiser (row_elems a multiple of 8, at most 8192), optional row scatter.
cudaError_t launch_quantize_e4m3(const void* x, int64_t n_tokens, int row_elems, void* codes, float* scale,
                                 const int64_t* dst_rows, cudaStream_t stream);

// sparse_attn.cu: attention over the selected rows. q_map: q as [n_q * H, 576] bf16, 128-byte swizzle, box
// 64 columns x H rows; kv_map: kv as [n_kv, 576] bf16, 128-byte swizzle, box 64 columns x 1 row (gather form). n_eff: [n_q][2] int32 scratch; scratch: sparse_attn_scratch_bytes(n_q, k_top) bytes, 16-byte
// aligned (the probabilities of a query between its two passes, per CTA). At most kSparseAttnMaxGrid CTAs run.
constexpr int kSparseAttnMaxGrid = 160;
bool sparse_attn_supported(int H, int d_qk, int d_v);
size_t sparse_attn_scratch_bytes(int64_t n_q, int k_top);
// With few queries (a decode step) a query's rows are split over several CTAs, whose fp32 partial results (sized for
// 128 heads) are merged by a second kernel; 0 bytes when every query has its own CTA.
size_t sparse_attn_partial_bytes(int64_t n_q);
cudaError_t launch_sparse_attn(const void* kv, const int32_t* topk, const int64_t* kv_base, int64_t n_q, int64_t n_kv, int H,
                               int k_top, float scale, void* out, float* lse, int32_t* n_eff, void* scratch, void* partial,
                               const CUtensorMap& q_map, unsigned int* status, int sm_count,
                               cudaStream_t stream);

// selftest.cu: one tiny kernel whose only wait can never be satisfied; it must record a time-out in
// `status` after `budget_cycles` and return.
cudaError_t launch_selftest_bounded_wait(unsigned int* status, long long budget_cycles, cudaStream_t stream);
// selftest.cu: every SM reads `iters` 128 x 256 fp32 accumulators per reading warp out of tensor memory with the
// prefill epilogue's load pattern (8 warps per SM); `sink` is a device word that is never written in practice.
cudaError_t launch_selftest_tmem_readout(uint32_t iters, uint32_t* sink, int sm_count, cudaStream_t stream);
// Issue rates of seven instruction kinds (selftest.cu); cycles: DEVICE [7], zeroed by the caller.
cudaError_t launch_selftest_issue_rates(uint32_t iters, unsigned long long* cycles, float* sink, int sm_count, cudaStream_t stream);
// The same read-out with a warp filling the accumulators by MMAs beside it; counters: DEVICE [2], see selftest.cu.
cudaError_t launch_selftest_tmem_readout_mma(uint32_t iters, bool fp8, uint32_t* sink, unsigned long long* counters,
                                             unsigned int* status, int sm_count, cudaStream_t stream);

}  // namespace idxc
