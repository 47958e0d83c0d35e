/*
 * idxc -- lightning-indexer scoring, causal top-k selection and the IndexCache
 * Full/Shared layer schedule for one NVIDIA B200 (sm_100a).
 *
 * Plain C ABI. Every pointer is a DEVICE pointer unless its comment says HOST.
 * The caller owns every buffer; the library allocates no device memory. All
 * work is enqueued on the CUDA stream passed in (a cudaStream_t cast to
 * void*, NULL = the legacy default stream) and the calls return without
 * synchronising. Every call returns an idxc_status; nothing throws or aborts.
 * Inputs are assumed finite (NaN / Inf scores give an unspecified selection).
 *
 * Notation follows the paper: L sequence length, H_I indexer heads, d_I indexer
 * head dimension, k_top selected tokens per query (k = 2048 in the paper),
 * N layers, pattern string c over {F, S}. Positions and layers are 0-based.
 */
#ifndef IDXC_H_
#define IDXC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    IDXC_OK = 0,
    IDXC_ERR_INVALID_ARG = 1,    /* null / misaligned pointer, size out of range, inconsistent sizes      */
    IDXC_ERR_UNSUPPORTED = 2,    /* a valid request this build has no kernel for (H_I, d_I, dtype combo)  */
    IDXC_ERR_WORKSPACE = 3,      /* workspace missing or smaller than the matching *_workspace_bytes()    */
    IDXC_ERR_PATTERN = 4,        /* pattern string invalid, or layers visited out of order                */
    IDXC_ERR_CUDA = 5,           /* a CUDA runtime/driver call failed (launch, tensor-map encode, ...)    */
    IDXC_ERR_DEVICE_TIMEOUT = 6  /* a bounded device-side wait gave up; results of that launch are void   */
} idxc_status;

/* Storage type of q and k. w and the scales are always fp32.
 * IDXC_FP8_E4M3 is the finite-only e4m3 ("FN": max 448, no infinities) with one
 * fp32 scale per token: value = code * scale. */
typedef enum { IDXC_BF16 = 0, IDXC_FP8_E4M3 = 1 } idxc_dtype;

/* flags (bitwise or) */
#define IDXC_FLAG_COPY_SHARED 0x1u  /* schedule: S layers copy the cached indices into topk_buf instead of aliasing */
#define IDXC_FLAG_SIMT_SCORER 0x2u  /* debugging aid: score with the plain CUDA-core kernel instead of tcgen05     */
#define IDXC_FLAG_FILL_MASKED 0x4u  /* prefill with scores_out: entries s > t of every row, up to column L_k - 1, are set
                                       to -infinity (the causal mask as a soft-max expects it) instead of left untouched */

#define IDXC_FLAG_STREAM_TOPK 0x8u  /* prefill with topk_out only: the scorer keeps, per query row, only the scores that can
                                       still be among the k_top largest (see idxc_indexer_prefill) instead of writing all */

/* Limits checked before any launch. */
#define IDXC_MAX_K_TOP 2048
#define IDXC_MAX_HEADS 64

const char* idxc_status_string(idxc_status s);

/* ---------------------------------------------------------------------------
 * Prefill: indexer scores and causal top-k for a block of query positions.
 *
 * Operation (Sec. 2.1 "DeepSeek Sparse Attention": the lightning indexer scores
 * all preceding tokens with a multi-head ReLU-gated dot product; Sec. 3
 * "Notation": T_t = Top-k(I_t)):
 *     I[t, s] = sum_h w[t, h] * max(q[t, h, :] . k[s, :], 0)      for s <= t
 *     T[t]    = the min(k_top, t + 1) positions s <= t with the largest I[t, s]
 * Ties go to the lowest position. T[t] is written in ascending position order
 * and padded with -1 up to k_top entries. With IDXC_FP8_E4M3 the dot product
 * uses the codes and the result is multiplied by q_scale[t] * k_scale[s].
 *
 *   q        [q_len, H_I, d_I] row-major; row r is position t = q_begin + r
 *   k        [L_k, d_I] row-major, L_k >= q_begin + q_len
 *   w        [q_len, H_I] fp32
 *   q_scale  [q_len] fp32, k_scale [L_k] fp32: IDXC_FP8_E4M3 only, else NULL
 *   scores_out  NULL, or [q_len, ld_scores] fp32 (ld_scores >= L_k, a multiple of 4;
 *               base 16-byte aligned). Only entries s <= t are written (IDXC_FLAG_FILL_MASKED: the other entries of the
 *               row up to column L_k - 1 are set to -infinity).
 *   topk_out    NULL, or [q_len, k_top] int32
 *   workspace   at least idxc_prefill_workspace_bytes(...) bytes, 256-byte aligned;
 *               contents are scratch. With scores_out == NULL the scores go through it
 *               in query chunks, so its size does not grow with q_len beyond a cap.
 * IDXC_FLAG_STREAM_TOPK (north star: "the score write or streaming top-k in the epilogue"; needs topk_out, scores_out
 * == NULL, L_k <= 262144 and a workspace sized with the same flag): the scorer visits a strided sample of a row's
 * keys first, takes from it a threshold that almost surely lies below the row's k_top-th largest score, and from then
 * on writes only (score, position) pairs at or above it to a per-row list; a second kernel selects exactly from the
 * list after checking, with its own count, that at least k_top listed scores reach the threshold. Rows that fail the
 * check (or whose list overflowed: many equal scores) are computed again by the ordinary score + select kernels,
 * which run after it and skip every other row. T is the same as without the flag, entry for entry.
 * A full prefill is q_begin = 0, q_len = L_k = L; chunked prefill calls this once
 * per chunk with the full K and gives the same rows.
 * Supported: d_I in {64, 128}; H_I in {16, 32, 64}; 1 <= k_top <= 2048; q_len * H_I < 2^31;
 * q, k, w 16-byte aligned. Other sizes return IDXC_ERR_UNSUPPORTED / INVALID_ARG
 * before anything is launched.
 * ------------------------------------------------------------------------- */
size_t idxc_prefill_workspace_bytes(int64_t q_len, int64_t L_k, int H_I, int d_I, int k_top,
                                    idxc_dtype dt, uint32_t flags);

idxc_status idxc_indexer_prefill(const void* q, const void* k, const float* w,
                                 const float* q_scale, const float* k_scale,
                                 int64_t q_begin, int64_t q_len, int64_t L_k,
                                 int H_I, int d_I, int k_top, idxc_dtype dt,
                                 float* scores_out, int64_t ld_scores, int32_t* topk_out,
                                 void* workspace, size_t workspace_bytes, uint32_t flags,
                                 void* cuda_stream);

/* ---------------------------------------------------------------------------
 * Decode: one new query per sequence against that sequence's cached indexer keys
 * (Sec. 4.2 "Decode": a per-token indexer pass over the full context).
 *     I[b, s] = sum_h w[b, h] * max(q_step[b, h, :] . K_b[s, :], 0)   for s < lens[b]
 *     T[b]    = Top-k over s in [0, lens[b]), same order / tie / padding rules
 *
 *   q_step    [B, H_I, d_I]
 *   k_cache   base of a [rows, d_I] row-major array; sequence b owns rows
 *             k_offsets[b] .. k_offsets[b] + lens[b] - 1 (the new token's key included)
 *   cache_rows  number of rows of k_cache that may be addressed (bounds the tensor map)
 *   w         [B, H_I] fp32
 *   q_scale   [B], k_scale [cache_rows] (same row indexing as k_cache): FP8 only
 *   k_offsets [B] int64, lens [B] int32 (device memory, read by the kernels)
 *   max_len   HOST upper bound on lens[b]; sizes the grid and the workspace
 *   scores_out NULL or [B, ld_scores] fp32, ld_scores >= max_len, multiple of 4
 *   topk_out  NULL or [B, k_top] int32
 * ------------------------------------------------------------------------- */
size_t idxc_decode_workspace_bytes(int B, int64_t max_len, int H_I, int d_I, int k_top,
                                   idxc_dtype dt, uint32_t flags);

idxc_status idxc_indexer_decode(const void* q_step, const void* k_cache, int64_t cache_rows,
                                const float* w, const float* q_scale, const float* k_scale,
                                const int64_t* k_offsets, const int32_t* lens,
                                int B, int64_t max_len, int H_I, int d_I, int k_top, idxc_dtype dt,
                                float* scores_out, int64_t ld_scores, int32_t* topk_out,
                                void* workspace, size_t workspace_bytes, uint32_t flags,
                                void* cuda_stream);

/* ---------------------------------------------------------------------------
 * Decode without caller-provided scratch. (The paper has no counterpart: this entry point
 * exists for hosts that cannot allocate device memory where they decode, e.g. a serving
 * process whose KV-cache pool already owns all free HBM, or a decode loop that cannot
 * afford the device-wide stall of cudaMalloc / cudaFree.)
 * Same operation, arguments and rules as idxc_indexer_decode with scores_out == NULL, but the
 * fp32 score scratch lives in an array built into the library (IDXC_NOALLOC_SCRATCH_BYTES on
 * every GPU this entry point is used on, until the process exits) instead of a workspace.
 * Limits and behaviour:
 *   - FIRST CALL ON A DEVICE: CUDA creates a library's device data lazily, so the array comes into
 *     being when the first call on a device looks its address up. That call makes the driver set
 *     aside the IDXC_NOALLOC_SCRATCH_BYTES (it fails with IDXC_ERR_CUDA if the device has no room
 *     left) and sets up per-kernel attributes. Make it once per device at start-up -- a warm-up
 *     step on small inputs is enough -- BEFORE the host gives the remaining HBM to its cache pool
 *     and before any stream capture, with that device current. Every later call on the device,
 *     whatever its shape or dtype, allocates nothing on the device or on the host.
 *   - B * round_up(max_len, 32) * 4 bytes must not exceed IDXC_NOALLOC_SCRATCH_BYTES (e.g.
 *     B = 32 sequences of up to 131072 keys); larger requests return IDXC_ERR_WORKSPACE and
 *     launch nothing. topk_out is required.
 *   - Every call shares the one array. Calls whose kernels can overlap on the GPU (different
 *     streams without an ordering between them) race and return unspecified indices; calls on
 *     one stream, or ordered by events, are safe. The array keeps the previous call's scores
 *     and needs no clearing: each call writes every score it later reads.
 * ------------------------------------------------------------------------- */
#define IDXC_NOALLOC_SCRATCH_BYTES (16u << 20)

idxc_status idxc_indexer_decode_noalloc(const void* q_step, const void* k_cache, int64_t cache_rows,
                                        const float* w, const float* q_scale, const float* k_scale,
                                        const int64_t* k_offsets, const int32_t* lens,
                                        int B, int64_t max_len, int H_I, int d_I, int k_top, idxc_dtype dt,
                                        int32_t* topk_out, uint32_t flags, void* cuda_stream);

/* ---------------------------------------------------------------------------
 * Top-k alone (Sec. 3 "Notation"), for rows of fp32 scores already in memory.
 * Row r has length lens[r] if lens != NULL (device int32), else
 * first_len + r * len_step (len_step = 1: causal rows; 0: equal rows), clamped to
 * [0, ld]. scores: [n_rows, ld] fp32, 16-byte aligned, ld a multiple of 4.
 * Same order / tie / padding rules as above. Needs no workspace.
 * ------------------------------------------------------------------------- */
idxc_status idxc_topk_rows(const float* scores, int64_t ld, int64_t n_rows,
                           int64_t first_len, int64_t len_step, const int32_t* lens,
                           int k_top, int32_t* topk_out, void* cuda_stream);

/* ---------------------------------------------------------------------------
 * Per-token FP8 quantiser with optional K-cache append: the step in front of the indexer
 * (Sec. 2.1: the lightning indexer uses FP8 arithmetic). For token r:
 *     scale[r]  = max(max_i |x[r, i]|, 1e-12) / 448                    (fp32)
 *     code[r,i] = e4m3(x[r, i] / scale[r])      round to nearest even, saturating at +-448
 * exactly the format idxc_indexer_prefill / idxc_indexer_decode read with IDXC_FP8_E4M3.
 *   x          [n_tokens, row_elems] bf16, 16-byte aligned; row_elems = d_I for keys, H_I * d_I for
 *              queries: a multiple of 8, at most 8192
 *   codes_out  [rows, row_elems] uint8 (8-byte aligned), scale_out [rows] fp32
 *   dst_rows   NULL: token r is written at row r. Otherwise a device array [n_tokens] int64: token r is
 *              written at row dst_rows[r] of codes_out / scale_out (appending new keys to an indexer K
 *              cache). The caller guarantees the rows are in range and distinct.
 * ------------------------------------------------------------------------- */
idxc_status idxc_quantize_e4m3(const void* x, int64_t n_tokens, int row_elems, void* codes_out, float* scale_out,
                               const int64_t* dst_rows, void* cuda_stream);

/* ---------------------------------------------------------------------------
 * IndexCache layer schedule (Sec. 3 "Overview", Figure 2(b)).
 * pattern c_0 .. c_{N-1} over {'F','S'}: an F (Full) layer runs its indexer and its
 * result becomes the cached index tensor; an S (Shared) layer returns the cached
 * tensor of f(l) = max{ j < l : c_j = F } without running anything. c_0 must be 'F'.
 * The schedule object is HOST state only (the pattern, f(l), the cached pointer and
 * counters); it is not thread-safe. Layers of one forward pass are visited in
 * increasing order; idxc_schedule_begin_pass() forgets the cached tensor.
 * ------------------------------------------------------------------------- */
typedef struct idxc_schedule idxc_schedule;

idxc_status idxc_schedule_create(const char* pattern /* HOST, N chars */, int N, idxc_schedule** out /* HOST */);
void        idxc_schedule_destroy(idxc_schedule* s);
idxc_status idxc_schedule_begin_pass(idxc_schedule* s);
/* f(layer); equals layer on F layers. src_layer is a HOST pointer. */
idxc_status idxc_schedule_source(const idxc_schedule* s, int layer, int* src_layer);
/* HOST outputs: number of F and S layers in the pattern, indexer launches made so far. */
idxc_status idxc_schedule_stats(const idxc_schedule* s, int* n_full, int* n_shared, int64_t* indexer_calls);

/* One layer of a prefill pass. On an F layer: runs idxc_indexer_prefill with the given
 * arguments into topk_buf ([q_len, k_top] int32, required) and caches it. On an S layer:
 * q, k, w, scales, scores_out and workspace are ignored (may be NULL) and nothing is
 * launched; *topk_result (HOST out) is the cached pointer, i.e. it aliases the F layer's
 * buffer, which the caller must therefore keep intact until the next F layer. With
 * IDXC_FLAG_COPY_SHARED an S layer instead copies the cached tensor into topk_buf
 * (one device-to-device copy) and returns topk_buf. Visiting an S layer whose source
 * layer was not the last F layer run in this pass returns IDXC_ERR_PATTERN. */
idxc_status idxc_schedule_prefill_layer(idxc_schedule* s, int layer,
                                        const void* q, const void* k, const float* w,
                                        const float* q_scale, const float* k_scale,
                                        int64_t q_begin, int64_t q_len, int64_t L_k,
                                        int H_I, int d_I, int k_top, idxc_dtype dt,
                                        float* scores_out, int64_t ld_scores, int32_t* topk_buf,
                                        void* workspace, size_t workspace_bytes, uint32_t flags,
                                        void* cuda_stream, const int32_t** topk_result);

/* One layer of a decode step; same rules, wrapping idxc_indexer_decode ([B, k_top]). */
idxc_status idxc_schedule_decode_layer(idxc_schedule* s, int layer,
                                       const void* q_step, const void* k_cache, int64_t cache_rows,
                                       const float* w, const float* q_scale, const float* k_scale,
                                       const int64_t* k_offsets, const int32_t* lens,
                                       int B, int64_t max_len, int H_I, int d_I, int k_top, idxc_dtype dt,
                                       float* scores_out, int64_t ld_scores, int32_t* topk_buf,
                                       void* workspace, size_t workspace_bytes, uint32_t flags,
                                       void* cuda_stream, const int32_t** topk_result);

/* ---------------------------------------------------------------------------
 * Pattern tooling on index tensors.
 *
 * idxc_topk_overlap -- the cross-layer top-k index overlap of Appendix A: for a pair of index tensors
 * T_a, T_b ([rows, k_top] int32, ascending, -1 padded, as produced above) the per-row ratio
 * |T_a[r] n T_b[r]| / (valid entries of T_a[r]) and its mean over the rows (the figure Appendix A plots).
 *   layers   DEVICE array of device pointers to the index tensors
 *   pairs    DEVICE int32 [2 * n_pairs]: pair p compares layers[pairs[2p]] with layers[pairs[2p+1]]
 *   means_out DEVICE double [n_pairs]: mean over the rows of the ratio; zeroed by the call
 *   row_out  NULL, or DEVICE float [rows] (only with n_pairs == 1): the per-row ratios
 * One launch covers all pairs (n_pairs <= 65535).
 *
 * idxc_pattern_search_dp -- the similarity-based search of Appendix C (HOST only, no GPU work): S is a HOST
 * row-major [N, N] matrix, S[l*N + j] (j < l) = how well layer j's indices serve layer l. Writes to
 * pattern_out (HOST, N chars, not terminated) a pattern with exactly M Full layers, the first layer Full, that
 * maximises the sum over Shared layers l of S[l, f(l)], and that maximum to value_out (HOST, may be NULL).
 *
 * idxc_pattern_search_greedy -- Algorithm 1 (HOST driver): starting from all-Full, K times flip to Shared the
 * remaining layer (never layer 0) whose flip gives the lowest eval_loss(pattern, N, user); ties go to the
 * lowest layer. eval_loss receives a NUL-terminated pattern. order_out (HOST, K ints, may be NULL) gets the
 * flipped layers in order, step_loss_out (HOST, K doubles, may be NULL) the loss of the pattern after each step,
 * evaluations_out (HOST, may be NULL) the number of loss evaluations (N(N-1)/2 for K = N-1).
 * ------------------------------------------------------------------------- */
typedef double (*idxc_eval_loss_fn)(const char* pattern, int N, void* user);

idxc_status idxc_topk_overlap(const int32_t* const* layers, const int32_t* pairs, int n_pairs, int64_t rows, int k_top,
                              double* means_out, float* row_out, void* cuda_stream);
idxc_status idxc_pattern_search_dp(const double* S, int N, int M, char* pattern_out, double* value_out);
idxc_status idxc_pattern_search_greedy(int N, int K, idxc_eval_loss_fn eval_loss, void* user, char* pattern_out,
                                       int* order_out, double* step_loss_out, int64_t* evaluations_out);

/* ---------------------------------------------------------------------------
 * Multi-layer distillation loss of training-aware IndexCache, forward value (Eq. 1):
 *     L_multi = sum_{j=0..m} 1/(m+1) sum_t KL( p_t^(l+j) || Softmax(I_t) )
 * I = indexer scores of the Full layer l, p^(l+j) = target distributions of the layers it serves.
 *   scores   [rows, ld] fp32 (without topk: 16-byte aligned, ld a multiple of 4, targets too); row r covers
 *            positions [0, first_len + r * len_step) (causal: 1, 1)
 *   targets  HOST array of n_targets (= m + 1, at most 16) DEVICE pointers to [rows, ld] fp32 distributions
 *   topk     NULL, or [rows, k_top] int32 (ascending, -1 padded): the sparse-training form, the KL is taken
 *            over these positions only, with the target renormalised over them
 *   loss_out DEVICE double[1] (zeroed by the call); row_loss_out NULL or DEVICE float [rows]
 * Entries with p = 0 contribute 0.
 * ------------------------------------------------------------------------- */
idxc_status idxc_distill_kl(const float* scores, int64_t ld, int64_t rows, int64_t first_len, int64_t len_step,
                            const float* const* targets, int n_targets, const int32_t* topk, int k_top,
                            double* loss_out, float* row_loss_out, void* cuda_stream);

/* ---------------------------------------------------------------------------
 * Sparse core attention over the selected positions (Sec. 2.1 "DeepSeek Sparse Attention": "the main attention
 * is computed only over this sparse subset"; Fig. 2: X <- SparseAttn_l(X, T^(l))). The paper runs it under
 * Multi-head Latent Attention and prints no shapes; this entry point takes the multi-query form latent
 * attention is served in: all heads of a query attend the same row per token, whose leading d_v columns are
 * also the value:
 *     s[t,h,j]   = scale * < q[t,h,:], kv[kv_base[t] + topk[t,j], 0:d_qk] >      for usable entries
 *     out[t,h,:] = sum_j Softmax_j(s[t,h,:])[j] * kv[kv_base[t] + topk[t,j], 0:d_v]
 *     lse[t,h]   = log sum_j exp(s[t,h,j])                                        (natural logarithm)
 * An entry is usable when topk[t,j] >= 0 and the row it names lies inside [0, n_kv); other entries are
 * skipped (they may sit anywhere in the row, order is free, duplicates count twice). A query without usable
 * entries gets out = 0 and lse = -inf.
 *   q        DEVICE bf16 [n_q, H, d_qk], 16-byte aligned      kv  DEVICE bf16 [n_kv, d_qk], 16-byte aligned
 *   topk     DEVICE int32 [n_q, k_top] (k_top >= 1)            kv_base  NULL or DEVICE int64 [n_q] (decode: the
 *            first cache row of the query's sequence; prefill: NULL)
 *   out      DEVICE bf16 [n_q, H, d_v], 16-byte aligned        lse  NULL or DEVICE fp32 [n_q, H]
 *   workspace DEVICE, idxc_sparse_attention_workspace_bytes(n_q, k_top) bytes, 16-byte aligned; caller-owned.
 *            It holds per-query entry counts and, per resident CTA, a query's probabilities between its two
 *            passes over the selected rows (about 0.5 MB per CTA at k_top = 2048) and, with fewer than 64
 *            queries, the fp32 partial results of the thread blocks that share a query
 * Supported shape: 1 <= H <= 128, d_qk = 576, d_v = 512 (tcgen05 path); anything else IDXC_ERR_UNSUPPORTED.
 * Arithmetic: bf16 products with fp32 accumulation, fp32 softmax with the probabilities rounded to bf16 for
 * the second product, bf16 output. Rows that are not selected are never read (they may hold anything).
 * Enqueues 2 kernels (3 with fewer than 64 queries, whose rows are split over several thread blocks and merged
 * by the third); nothing is allocated. Errors: IDXC_ERR_INVALID_ARG (null or misaligned pointer, sizes out of range),
 * IDXC_ERR_WORKSPACE, IDXC_ERR_UNSUPPORTED, IDXC_ERR_CUDA.
 * ------------------------------------------------------------------------- */
size_t idxc_sparse_attention_workspace_bytes(int64_t n_q, int k_top);
idxc_status idxc_sparse_attention(const void* q, const void* kv, const int32_t* topk, const int64_t* kv_base,
                                  int64_t n_q, int64_t n_kv, int H, int d_qk, int d_v, int k_top, float scale,
                                  void* out, float* lse, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Synchronises the stream, then returns IDXC_OK, IDXC_ERR_CUDA, or
 * IDXC_ERR_DEVICE_TIMEOUT if any kernel of this library recorded a bounded wait that
 * ran out since the last poll (the record is cleared). */
idxc_status idxc_poll_device_status(void* cuda_stream);

/* Self-test of the bounded device waits (no counterpart in the paper). Every spin-wait in this library's
 * kernels gives up after a cycle budget, records a code in a device status word and lets the kernel return,
 * so that a lost signal shows up as IDXC_ERR_DEVICE_TIMEOUT instead of a hung GPU. This call enqueues a
 * one-warp kernel whose only wait can never be satisfied, with a budget of wait_cycles SM cycles (clamped to
 * 1e8, about 50 ms); the next idxc_poll_device_status on the stream then returns IDXC_ERR_DEVICE_TIMEOUT
 * once, and IDXC_OK afterwards. Nothing traps or faults. */
idxc_status idxc_selftest_bounded_wait(uint32_t wait_cycles, void* cuda_stream);

/* Measurement aid (no counterpart in the paper): the rate at which the prefill scorer's epilogue can read fp32
 * accumulators out of tensor memory, which bounds the FP8 scorer (its tensor work per accumulator is half the bf16
 * scorer's, its read-out the same). Enqueues one kernel with the scorer's CTA shape (one CTA per SM, 8 reading warps)
 * in which every reading warp reads its share (32 lanes x 128 columns) of accumulators_per_warp accumulators with the
 * epilogue's own loads and nothing else runs. *bytes_read_out (HOST, may be NULL) = accumulator bytes the launch reads
 * over all SMs; time the launch with events around the call to get bytes per second. 1 <= accumulators_per_warp <= 2^24. */
idxc_status idxc_selftest_tmem_readout(uint32_t accumulators_per_warp, int64_t* bytes_read_out, void* cuda_stream);

/* Measurement aid (no counterpart in the paper): the same read-out while one more warp per SM keeps the tensor pipe busy
 * filling the two 128 x 256 accumulators with MMAs of the scorer's shape (fp8 != 0: e4m3, four K = 32 steps per fill;
 * else bf16, eight K = 16 steps; operands are zero tiles in shared memory) until the reading warps are done. It tells
 * whether tensor-memory reads and MMAs slow each other down. counters (DEVICE, uint64 [2], zeroed by the call):
 * [0] = accumulator fills completed over all SMs while the readers ran (each 2 * 128 * 256 * 128 flops),
 * [1] = cycles of the slowest reading warp. *bytes_read_out (HOST, may be NULL) as above; time the launch with events. */
idxc_status idxc_selftest_tmem_readout_under_mma(uint32_t accumulators_per_warp, int fp8, int64_t* bytes_read_out,
                                                 uint64_t* counters, void* cuda_stream);

/* Measurement aid (no counterpart in the paper): how fast one scheduler of an SM takes instructions of seven kinds,
 * which is what bounds the scorer's epilogue and the select (both are limited by instruction issue, not by bytes).
 * Enqueues seven kernels (one CTA of 256 threads per SM: two warps per scheduler); in each, every thread runs `rounds`
 * rounds of 16 independent instructions of one kind (8 for the packed kind). cycles (DEVICE, uint64
 * [IDXC_ISSUE_RATE_KINDS], zeroed by the call) receives the slowest warp's cycles per kind, in this order: 0 float min/max,
 * 1 add with |x|, 2 fma, 3 packed fma.rn.f32x2 (8 per round), 4 compare + select (a pair per slot), 5 three-input logic,
 * 6 warp shuffle. cycles[i] / (rounds * 16 * 2) (8 for kind 3) = scheduler cycles per
 * warp instruction. 1 <= rounds <= 2^20. */
#define IDXC_ISSUE_RATE_KINDS 7
idxc_status idxc_selftest_issue_rates(uint32_t rounds, uint64_t* cycles, void* cuda_stream);

/* Number of kernel launches this library has made in this process (all streams). */
int64_t idxc_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* IDXC_H_ */
