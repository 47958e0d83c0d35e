// C-ABI layer: argument validation, TMA tensor-map encoding, launch sequencing and the
// host-side IndexCache schedule object. No device memory is allocated here.
#include <atomic>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <utility>
#include <vector>

#include "../../include/idxc.h"
#include "kernels.h"

namespace idxc {

__device__ unsigned int g_device_status = 0;   // first bounded-wait failure since the last poll

namespace {

std::atomic<int64_t> g_launches{0};

struct DeviceInfo {
    bool ready = false;
    bool ok = false;
    int sm_count = 0;
    unsigned int* status_ptr = nullptr;
    decltype(&cuTensorMapEncodeTiled) encode = nullptr;
};

constexpr int kMaxDevices = 64;
std::mutex g_info_mutex;

// Per-device facts (SM count, address of this device's status word), looked up once per device
// under a mutex: a process may drive several devices and call from several threads.
DeviceInfo& device_info() {
    static DeviceInfo infos[kMaxDevices];
    static DeviceInfo bad;            // ok == false: no current device, or an index beyond the table
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return bad;
    std::lock_guard<std::mutex> lock(g_info_mutex);
    DeviceInfo& info = infos[dev];
    if (!info.ready) {
        info.ready = true;
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaDeviceGetAttribute(&info.sm_count, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess &&
            cudaGetSymbolAddress(reinterpret_cast<void**>(&info.status_ptr), g_device_status) == cudaSuccess &&
            cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess && fn != nullptr) {
            info.encode = reinterpret_cast<decltype(&cuTensorMapEncodeTiled)>(fn);
            info.ok = true;
        }
    }
    return info;
}

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }
inline int64_t round_up(int64_t x, int64_t m) { return (x + m - 1) / m * m; }

constexpr int64_t kMinChunkRows = 32;
constexpr int64_t kPreferredScratchBytes = int64_t(8) << 30;

// Row-major [rows, d] operand, 128-byte swizzle, box = 128 bytes x box_rows rows.
bool encode_operand_map(CUtensorMap* map, const void* base, int64_t rows, int d, bool fp8, int box_rows) {
    DeviceInfo& di = device_info();
    const cuuint64_t gdim[2] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(rows)};
    const cuuint64_t gstride[1] = {static_cast<cuuint64_t>(d) * (fp8 ? 1u : 2u)};
    const cuuint32_t box[2] = {fp8 ? 128u : 64u, static_cast<cuuint32_t>(box_rows)};
    const cuuint32_t estr[2] = {1u, 1u};
    CUresult r = di.encode(map, fp8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                           const_cast<void*>(base), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

idxc_status check_common(int H, int d, int k_top, idxc_dtype dt, uint32_t flags) {
    if (dt != IDXC_BF16 && dt != IDXC_FP8_E4M3) return IDXC_ERR_INVALID_ARG;
    if (k_top < 1 || k_top > IDXC_MAX_K_TOP) return IDXC_ERR_INVALID_ARG;
    if (H < 1 || H > IDXC_MAX_HEADS || d < 1) return IDXC_ERR_INVALID_ARG;
    if (flags & ~(IDXC_FLAG_COPY_SHARED | IDXC_FLAG_SIMT_SCORER | IDXC_FLAG_FILL_MASKED | IDXC_FLAG_STREAM_TOPK)) return IDXC_ERR_INVALID_ARG;
    if ((flags & IDXC_FLAG_STREAM_TOPK) && (flags & IDXC_FLAG_SIMT_SCORER)) return IDXC_ERR_INVALID_ARG;
    if (!(flags & IDXC_FLAG_SIMT_SCORER) && !score_tc_supported(H, d, dt == IDXC_FP8_E4M3)) return IDXC_ERR_UNSUPPORTED;
    return IDXC_OK;
}

// Streaming top-k: bytes of workspace per query row of a chunk (full scores for the rows that are computed again, the
// candidate lists, their lengths, the threshold, two flag bytes) and the slack for aligning the seven regions.
int64_t stream_bytes_per_row(int64_t ld) { return ld * 4 + static_cast<int64_t>(kStreamRowSlots) * 8 + kStreamLanes + 4 + 4 + 2; }
constexpr int64_t kStreamSlack = 7 * 256;

idxc_status launch_scorer(const ScoreArgs& a, bool decode, uint32_t flags, cudaStream_t stream) {
    if (flags & IDXC_FLAG_SIMT_SCORER) {
        g_launches += 1;
        return launch_score_simt(a, stream) == cudaSuccess ? IDXC_OK : IDXC_ERR_CUDA;
    }
    DeviceInfo& di = device_info();
    CUtensorMap q_map, k_map;
    const int q_box_rows = decode ? a.H : 256;
    if (!encode_operand_map(&q_map, a.q, a.n_rows * a.H, a.d, a.fp8 != 0, q_box_rows)) return IDXC_ERR_CUDA;
    if (!encode_operand_map(&k_map, a.k, a.k_rows, a.d, a.fp8 != 0, 128)) return IDXC_ERR_CUDA;
    cudaError_t e = decode ? launch_score_decode_tc(a, q_map, k_map, di.status_ptr, di.sm_count, stream)
                           : launch_score_prefill_tc(a, q_map, k_map, di.status_ptr, di.sm_count, stream);
    g_launches += 1;
    return e == cudaSuccess ? IDXC_OK : IDXC_ERR_CUDA;
}

}  // namespace

// Function attributes are per device: remember which (kernel, device) pairs have been raised. The table is a
// fixed array in static storage (this function never allocates); once it is full the attribute is simply set again
// on every call, which is harmless.
cudaError_t ensure_max_dynamic_smem(const void* kernel, int bytes) {
    constexpr int kSlots = 1024;
    static std::mutex mu;
    static const void* done_kernel[kSlots];
    static int done_dev[kSlots];
    static int n_done = 0;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(mu);
    for (int i = 0; i < n_done; ++i)
        if (done_kernel[i] == kernel && done_dev[i] == dev) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess && n_done < kSlots) {
        done_kernel[n_done] = kernel;
        done_dev[n_done] = dev;
        ++n_done;
    }
    return e;
}

}  // namespace idxc

using namespace idxc;

struct idxc_schedule {
    std::string pattern;
    std::vector<int> src;
    int n_full = 0;
    int n_shared = 0;
    int64_t indexer_calls = 0;
    int cache_layer = -1;              // F layer whose indices are cached, -1: none yet in this pass
    const int32_t* cache_ptr = nullptr;
    int64_t cache_rows = 0;
    int cache_k_top = 0;
};

extern "C" {

const char* idxc_status_string(idxc_status s) {
    switch (s) {
        case IDXC_OK: return "ok";
        case IDXC_ERR_INVALID_ARG: return "invalid argument";
        case IDXC_ERR_UNSUPPORTED: return "unsupported shape or dtype";
        case IDXC_ERR_WORKSPACE: return "workspace missing or too small";
        case IDXC_ERR_PATTERN: return "invalid pattern or layer order";
        case IDXC_ERR_CUDA: return "CUDA call failed";
        case IDXC_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

int64_t idxc_launch_count(void) { return g_launches.load(); }

size_t idxc_prefill_workspace_bytes(int64_t q_len, int64_t L_k, int H_I, int d_I, int k_top, idxc_dtype dt,
                                    uint32_t flags) {
    (void)L_k; (void)H_I; (void)d_I; (void)k_top; (void)dt;
    if (q_len <= 0) return 0;
    // scratch rows of round_up(L_k, 32) floats; L_k bounds q_begin + q_len
    const int64_t ld = round_up(L_k > q_len ? L_k : q_len, 32);
    const int64_t per_row = (flags & IDXC_FLAG_STREAM_TOPK) ? stream_bytes_per_row(ld) : ld * 4;
    int64_t rows = round_up(q_len, kMinChunkRows);
    const int64_t cap = (kPreferredScratchBytes / per_row) / kMinChunkRows * kMinChunkRows;
    if (rows > cap) rows = cap < kMinChunkRows ? kMinChunkRows : cap;
    return static_cast<size_t>(rows * per_row + ((flags & IDXC_FLAG_STREAM_TOPK) ? kStreamSlack : 0));
}

idxc_status idxc_indexer_prefill(const void* q, const void* k, const float* w, const float* q_scale,
                                 const float* k_scale, int64_t q_begin, int64_t q_len, int64_t L_k, int H_I,
                                 int d_I, int k_top, idxc_dtype dt, float* scores_out, int64_t ld_scores,
                                 int32_t* topk_out, void* workspace, size_t workspace_bytes, uint32_t flags,
                                 void* cuda_stream) {
    idxc_status st = check_common(H_I, d_I, k_top, dt, flags);
    if (st != IDXC_OK) return st;
    if (q_begin < 0 || q_len < 0 || L_k < q_begin + q_len || L_k > (int64_t(1) << 30)) return IDXC_ERR_INVALID_ARG;
    // the kernels address q through a tensor map whose row coordinate (query * H_I + head) is a 32-bit int
    if (q_len * H_I >= (int64_t(1) << 31)) return IDXC_ERR_INVALID_ARG;
    if (q_len == 0) return IDXC_OK;
    if (!scores_out && !topk_out) return IDXC_ERR_INVALID_ARG;
    if (!q || !k || !w || !aligned(q, 16) || !aligned(k, 16) || !aligned(w, 16)) return IDXC_ERR_INVALID_ARG;
    const bool fp8 = dt == IDXC_FP8_E4M3;
    if (fp8 && (!q_scale || !k_scale)) return IDXC_ERR_INVALID_ARG;
    if (scores_out && (ld_scores < L_k || (ld_scores & 3) || !aligned(scores_out, 16))) return IDXC_ERR_INVALID_ARG;
    if (topk_out && !aligned(topk_out, 4)) return IDXC_ERR_INVALID_ARG;
    const bool streaming = (flags & IDXC_FLAG_STREAM_TOPK) != 0;
    if (streaming) {
        if (scores_out || !topk_out) return IDXC_ERR_INVALID_ARG;
        if (L_k > kStreamMaxKeys || !score_prefill_stream_supported(H_I, d_I, fp8 ? 1 : 0)) return IDXC_ERR_UNSUPPORTED;
    }
    if (!device_info().ok) return IDXC_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int64_t elem = fp8 ? 1 : 2;

    ScoreArgs a{};
    a.k = k; a.k_scale = fp8 ? k_scale : nullptr; a.k_offsets = nullptr; a.lens = nullptr;
    a.k_rows = L_k; a.max_len = 0; a.H = H_I; a.d = d_I; a.fp8 = fp8 ? 1 : 0;

    auto run_rows = [&](int64_t r0, int64_t nr, float* sc, int64_t ld) -> idxc_status {
        a.q = static_cast<const char*>(q) + r0 * H_I * d_I * elem;
        a.w = w + r0 * H_I;
        a.q_scale = fp8 ? q_scale + r0 : nullptr;
        a.q_begin = q_begin + r0;
        a.n_rows = nr;
        a.scores = sc;
        a.ld = ld;
        idxc_status s2 = launch_scorer(a, false, flags, stream);
        if (s2 != IDXC_OK) return s2;
        if (topk_out) {
            int n_l = 0;
            const cudaError_t e = launch_topk_rows(sc, ld, nr, q_begin + r0 + 1, 1, nullptr, k_top, topk_out + r0 * k_top, stream, nullptr, &n_l);
            g_launches += n_l;
            if (e != cudaSuccess) return IDXC_ERR_CUDA;
        }
        return IDXC_OK;
    };

    if (scores_out) {
        if (flags & IDXC_FLAG_FILL_MASKED) {                   // disjoint from what the scorer writes: any order
            g_launches += 1;
            if (launch_fill_masked(scores_out, ld_scores, q_begin, q_len, L_k, stream) != cudaSuccess) return IDXC_ERR_CUDA;
        }
        return run_rows(0, q_len, scores_out, ld_scores);
    }

    // scores go through the workspace in query chunks
    const int64_t ld = round_up(q_begin + q_len, 32);
    if (!workspace || !aligned(workspace, 256)) return IDXC_ERR_WORKSPACE;
    if (streaming) {
        if (workspace_bytes < static_cast<size_t>(kStreamSlack)) return IDXC_ERR_WORKSPACE;
        const int64_t per_row = stream_bytes_per_row(ld);
        const int64_t chunk = static_cast<int64_t>((workspace_bytes - kStreamSlack) / static_cast<size_t>(per_row)) / kMinChunkRows * kMinChunkRows;
        if (chunk < kMinChunkRows) return IDXC_ERR_WORKSPACE;
        // regions of the workspace, each 256-byte aligned (chunk is a multiple of 32 rows)
        char* base = static_cast<char*>(workspace);
        auto take = [&](int64_t bytes) { char* r = base; base += round_up(bytes, 256); return r; };
        float* sc = reinterpret_cast<float*>(take(chunk * ld * 4));
        StreamTopk stt{};
        stt.cand = reinterpret_cast<uint2*>(take(chunk * kStreamRowSlots * 8));
        stt.sample_count = reinterpret_cast<uint32_t*>(take(chunk * 4));
        stt.lane_count = reinterpret_cast<uint8_t*>(take(chunk * kStreamLanes));
        stt.tau = reinterpret_cast<float*>(take(chunk * 4));
        stt.k_top = k_top;
        uint8_t* row_fail = reinterpret_cast<uint8_t*>(take(chunk));
        uint8_t* item_fail = reinterpret_cast<uint8_t*>(take(chunk));
        const int rows_per_item = score_prefill_rows_per_item(H_I);
        for (int64_t r0 = 0; r0 < q_len; r0 += chunk) {
            const int64_t nr = q_len - r0 < chunk ? q_len - r0 : chunk;
            a.q = static_cast<const char*>(q) + r0 * H_I * d_I * elem;
            a.w = w + r0 * H_I;
            a.q_scale = fp8 ? q_scale + r0 : nullptr;
            a.q_begin = q_begin + r0;
            a.n_rows = nr;
            // 1. scorer with the filtered lists instead of the score write; 2. exact selection from the lists
            a.scores = nullptr; a.ld = 0; a.stream = stt; a.item_mask = nullptr;
            st = launch_scorer(a, false, flags, stream);
            if (st != IDXC_OK) return st;
            g_launches += 1;
            if (launch_finish_topk_stream(stt, nr, q_begin + r0, rows_per_item, topk_out + r0 * k_top, row_fail, item_fail, stream) != cudaSuccess)
                return IDXC_ERR_CUDA;
            // 3. the blocks of rows with a flagged row, scored in full; 4. the flagged rows, selected the ordinary way
            a.scores = sc; a.ld = ld; a.stream = StreamTopk{}; a.item_mask = item_fail;
            st = launch_scorer(a, false, flags, stream);
            if (st != IDXC_OK) return st;
            int n_l = 0;
            const cudaError_t e = launch_topk_rows(sc, ld, nr, q_begin + r0 + 1, 1, nullptr, k_top, topk_out + r0 * k_top, stream, row_fail, &n_l);
            g_launches += n_l;
            if (e != cudaSuccess) return IDXC_ERR_CUDA;
        }
        return IDXC_OK;
    }
    int64_t chunk = static_cast<int64_t>(workspace_bytes / static_cast<size_t>(ld * 4)) / kMinChunkRows * kMinChunkRows;
    if (chunk < kMinChunkRows) return IDXC_ERR_WORKSPACE;
    for (int64_t r0 = 0; r0 < q_len; r0 += chunk) {
        const int64_t nr = q_len - r0 < chunk ? q_len - r0 : chunk;
        st = run_rows(r0, nr, static_cast<float*>(workspace), ld);
        if (st != IDXC_OK) return st;
    }
    return IDXC_OK;
}

size_t idxc_decode_workspace_bytes(int B, int64_t max_len, int H_I, int d_I, int k_top, idxc_dtype dt, uint32_t flags) {
    (void)H_I; (void)d_I; (void)k_top; (void)dt; (void)flags;
    if (B <= 0 || max_len <= 0) return 0;
    return static_cast<size_t>(B) * static_cast<size_t>(round_up(max_len, 32)) * 4;
}

idxc_status idxc_indexer_decode(const void* q_step, const void* k_cache, int64_t cache_rows, const float* w,
                                const float* q_scale, const float* k_scale, const int64_t* k_offsets,
                                const int32_t* lens, int B, int64_t max_len, int H_I, int d_I, int k_top,
                                idxc_dtype dt, float* scores_out, int64_t ld_scores, int32_t* topk_out,
                                void* workspace, size_t workspace_bytes, uint32_t flags, void* cuda_stream) {
    idxc_status st = check_common(H_I, d_I, k_top, dt, flags);
    if (st != IDXC_OK) return st;
    // cache rows and (sequence, head) rows are 32-bit tensor-map coordinates in the kernels
    if (B < 0 || max_len < 0 || max_len > (int64_t(1) << 30) || cache_rows < 0 || cache_rows > (int64_t(1) << 31) - 256 ||
        static_cast<int64_t>(B) * H_I >= (int64_t(1) << 31))
        return IDXC_ERR_INVALID_ARG;
    if (B == 0) return IDXC_OK;
    if (!scores_out && !topk_out) return IDXC_ERR_INVALID_ARG;
    if (!q_step || !k_cache || !w || !k_offsets || !lens) return IDXC_ERR_INVALID_ARG;
    if (!aligned(q_step, 16) || !aligned(k_cache, 16) || !aligned(k_offsets, 8) || !aligned(lens, 4)) return IDXC_ERR_INVALID_ARG;
    const bool fp8 = dt == IDXC_FP8_E4M3;
    if (fp8 && (!q_scale || !k_scale)) return IDXC_ERR_INVALID_ARG;
    if (scores_out && (ld_scores < max_len || (ld_scores & 3) || !aligned(scores_out, 16))) return IDXC_ERR_INVALID_ARG;
    if (!device_info().ok) return IDXC_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    float* sc = scores_out;
    int64_t ld = ld_scores;
    if (!sc) {
        ld = round_up(max_len, 32);
        if (max_len > 0 && (!workspace || !aligned(workspace, 256) ||
                            workspace_bytes < static_cast<size_t>(B) * static_cast<size_t>(ld) * 4))
            return IDXC_ERR_WORKSPACE;
        sc = static_cast<float*>(workspace);
    }
    ScoreArgs a{};
    a.q = q_step; a.k = k_cache; a.w = w;
    a.q_scale = fp8 ? q_scale : nullptr; a.k_scale = fp8 ? k_scale : nullptr;
    a.k_offsets = k_offsets; a.lens = lens; a.q_begin = 0; a.n_rows = B; a.k_rows = cache_rows;
    a.max_len = max_len; a.H = H_I; a.d = d_I; a.fp8 = fp8 ? 1 : 0; a.scores = sc; a.ld = ld;
    if (max_len > 0) {
        st = launch_scorer(a, true, flags, stream);
        if (st != IDXC_OK) return st;
    }
    if (topk_out) {
        g_launches += 1;
        if (launch_topk_rows(sc, ld, B, 0, 0, lens, k_top, topk_out, stream) != cudaSuccess) return IDXC_ERR_CUDA;
    }
    return IDXC_OK;
}

idxc_status idxc_topk_rows(const float* scores, int64_t ld, int64_t n_rows, int64_t first_len, int64_t len_step,
                           const int32_t* lens, int k_top, int32_t* topk_out, void* cuda_stream) {
    if (k_top < 1 || k_top > IDXC_MAX_K_TOP || n_rows < 0 || ld < 0 || (ld & 3) || ld > (int64_t(1) << 30))
        return IDXC_ERR_INVALID_ARG;
    if (n_rows == 0) return IDXC_OK;
    if (!scores || !topk_out || !aligned(scores, 16) || !aligned(topk_out, 4)) return IDXC_ERR_INVALID_ARG;
    if (!lens && (first_len < 0 || len_step < 0)) return IDXC_ERR_INVALID_ARG;
    int n_l = 0;
    const cudaError_t e = launch_topk_rows(scores, ld, n_rows, first_len, len_step, lens, k_top, topk_out,
                                           static_cast<cudaStream_t>(cuda_stream), nullptr, &n_l);
    g_launches += n_l;
    return e == cudaSuccess ? IDXC_OK : IDXC_ERR_CUDA;
}

// ------------------------------------------------------------------ schedule (Figure 2(b))

idxc_status idxc_schedule_create(const char* pattern, int N, idxc_schedule** out) {
    if (!out) return IDXC_ERR_INVALID_ARG;
    *out = nullptr;
    if (!pattern || N < 1) return IDXC_ERR_PATTERN;
    for (int l = 0; l < N; ++l)
        if (pattern[l] != 'F' && pattern[l] != 'S') return IDXC_ERR_PATTERN;
    if (pattern[0] != 'F') return IDXC_ERR_PATTERN;   // the first layer seeds the indices
    idxc_schedule* s = new (std::nothrow) idxc_schedule();
    if (!s) return IDXC_ERR_INVALID_ARG;
    s->pattern.assign(pattern, pattern + N);
    s->src.resize(N);
    int last_full = 0;
    for (int l = 0; l < N; ++l) {
        if (pattern[l] == 'F') { last_full = l; ++s->n_full; } else { ++s->n_shared; }
        s->src[l] = last_full;                          // f(l) = nearest preceding F layer (l itself on F layers)
    }
    *out = s;
    return IDXC_OK;
}

void idxc_schedule_destroy(idxc_schedule* s) { delete s; }

idxc_status idxc_schedule_begin_pass(idxc_schedule* s) {
    if (!s) return IDXC_ERR_INVALID_ARG;
    s->cache_layer = -1;
    s->cache_ptr = nullptr;
    s->cache_rows = 0;
    s->cache_k_top = 0;
    return IDXC_OK;
}

idxc_status idxc_schedule_source(const idxc_schedule* s, int layer, int* src_layer) {
    if (!s || !src_layer || layer < 0 || layer >= static_cast<int>(s->src.size())) return IDXC_ERR_INVALID_ARG;
    *src_layer = s->src[layer];
    return IDXC_OK;
}

idxc_status idxc_schedule_stats(const idxc_schedule* s, int* n_full, int* n_shared, int64_t* indexer_calls) {
    if (!s) return IDXC_ERR_INVALID_ARG;
    if (n_full) *n_full = s->n_full;
    if (n_shared) *n_shared = s->n_shared;
    if (indexer_calls) *indexer_calls = s->indexer_calls;
    return IDXC_OK;
}

}  // extern "C"

namespace {

// Shared tail of the two *_layer calls: S layers hand back the cached tensor.
idxc_status shared_layer(idxc_schedule* s, int layer, int64_t rows, int k_top, int32_t* topk_buf, uint32_t flags,
                         cudaStream_t stream, const int32_t** topk_result) {
    if (s->cache_layer != s->src[layer] || !s->cache_ptr) return IDXC_ERR_PATTERN;
    if (rows != s->cache_rows || k_top != s->cache_k_top) return IDXC_ERR_INVALID_ARG;
    if (flags & IDXC_FLAG_COPY_SHARED) {
        if (!topk_buf) return IDXC_ERR_INVALID_ARG;
        if (topk_buf != s->cache_ptr &&
            cudaMemcpyAsync(topk_buf, s->cache_ptr, static_cast<size_t>(rows) * k_top * sizeof(int32_t),
                            cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
            return IDXC_ERR_CUDA;
        *topk_result = topk_buf;
    } else {
        *topk_result = s->cache_ptr;
    }
    return IDXC_OK;
}

}  // namespace

extern "C" {

idxc_status idxc_schedule_prefill_layer(idxc_schedule* s, int layer, const void* q, const void* k, const float* w,
                                        const float* q_scale, const float* k_scale, int64_t q_begin, int64_t q_len,
                                        int64_t L_k, int H_I, int d_I, int k_top, idxc_dtype dt, float* scores_out,
                                        int64_t ld_scores, int32_t* topk_buf, void* workspace, size_t workspace_bytes,
                                        uint32_t flags, void* cuda_stream, const int32_t** topk_result) {
    if (!s || !topk_result || layer < 0 || layer >= static_cast<int>(s->src.size())) return IDXC_ERR_INVALID_ARG;
    *topk_result = nullptr;
    if (s->pattern[layer] == 'S')
        return shared_layer(s, layer, q_len, k_top, topk_buf, flags, static_cast<cudaStream_t>(cuda_stream), topk_result);
    if (!topk_buf) return IDXC_ERR_INVALID_ARG;
    idxc_status st = idxc_indexer_prefill(q, k, w, q_scale, k_scale, q_begin, q_len, L_k, H_I, d_I, k_top, dt,
                                          scores_out, ld_scores, topk_buf, workspace, workspace_bytes,
                                          flags & ~IDXC_FLAG_COPY_SHARED, cuda_stream);
    if (st != IDXC_OK) return st;
    s->indexer_calls += 1;
    s->cache_layer = layer;
    s->cache_ptr = topk_buf;
    s->cache_rows = q_len;
    s->cache_k_top = k_top;
    *topk_result = topk_buf;
    return IDXC_OK;
}

idxc_status idxc_schedule_decode_layer(idxc_schedule* s, int layer, const void* q_step, const void* k_cache,
                                       int64_t cache_rows, const float* w, const float* q_scale, const float* k_scale,
                                       const int64_t* k_offsets, const int32_t* lens, int B, int64_t max_len, int H_I,
                                       int d_I, int k_top, idxc_dtype dt, float* scores_out, int64_t ld_scores,
                                       int32_t* topk_buf, void* workspace, size_t workspace_bytes, uint32_t flags,
                                       void* cuda_stream, const int32_t** topk_result) {
    if (!s || !topk_result || layer < 0 || layer >= static_cast<int>(s->src.size())) return IDXC_ERR_INVALID_ARG;
    *topk_result = nullptr;
    if (s->pattern[layer] == 'S')
        return shared_layer(s, layer, B, k_top, topk_buf, flags, static_cast<cudaStream_t>(cuda_stream), topk_result);
    if (!topk_buf) return IDXC_ERR_INVALID_ARG;
    idxc_status st = idxc_indexer_decode(q_step, k_cache, cache_rows, w, q_scale, k_scale, k_offsets, lens, B, max_len,
                                         H_I, d_I, k_top, dt, scores_out, ld_scores, topk_buf, workspace,
                                         workspace_bytes, flags & ~IDXC_FLAG_COPY_SHARED, cuda_stream);
    if (st != IDXC_OK) return st;
    s->indexer_calls += 1;
    s->cache_layer = layer;
    s->cache_ptr = topk_buf;
    s->cache_rows = B;
    s->cache_k_top = k_top;
    *topk_result = topk_buf;
    return IDXC_OK;
}

idxc_status idxc_quantize_e4m3(const void* x, int64_t n_tokens, int row_elems, void* codes_out, float* scale_out,
                               const int64_t* dst_rows, void* cuda_stream) {
    if (n_tokens < 0 || row_elems < 8 || (row_elems & 7) || row_elems > 8192) return IDXC_ERR_INVALID_ARG;
    if (n_tokens == 0) return IDXC_OK;
    if (!x || !codes_out || !scale_out || !aligned(x, 16) || !aligned(codes_out, 8) || !aligned(scale_out, 4))
        return IDXC_ERR_INVALID_ARG;
    if (dst_rows && !aligned(dst_rows, 8)) return IDXC_ERR_INVALID_ARG;
    g_launches += 1;
    return launch_quantize_e4m3(x, n_tokens, row_elems, codes_out, scale_out, dst_rows,
                                static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? IDXC_OK : IDXC_ERR_CUDA;
}

size_t idxc_sparse_attention_workspace_bytes(int64_t n_q, int k_top) {
    if (n_q <= 0 || k_top < 1) return 0;
    return static_cast<size_t>(round_up(n_q * 8, 256)) + static_cast<size_t>(round_up(sparse_attn_scratch_bytes(n_q, k_top), 256)) +
           sparse_attn_partial_bytes(n_q);
}

idxc_status idxc_sparse_attention(const void* q, const void* kv, const int32_t* topk, const int64_t* kv_base, int64_t n_q,
                                  int64_t n_kv, int H, int d_qk, int d_v, int k_top, float scale, void* out, float* lse,
                                  void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (n_q < 0 || n_kv < 0 || H < 1 || d_qk < 1 || d_v < 1 || d_v > d_qk || k_top < 1) return IDXC_ERR_INVALID_ARG;
    if (!sparse_attn_supported(H, d_qk, d_v)) return IDXC_ERR_UNSUPPORTED;
    if (n_q == 0) return IDXC_OK;
    if (n_q * H >= (int64_t(1) << 31)) return IDXC_ERR_INVALID_ARG;
    if (!q || !topk || !out || (n_kv > 0 && !kv)) return IDXC_ERR_INVALID_ARG;
    if (!aligned(q, 16) || !aligned(kv, 16) || !aligned(out, 16) || !aligned(topk, 4) || (kv_base && !aligned(kv_base, 8)) ||
        (lse && !aligned(lse, 4)))
        return IDXC_ERR_INVALID_ARG;
    if (!workspace || !aligned(workspace, 16) || workspace_bytes < idxc_sparse_attention_workspace_bytes(n_q, k_top)) return IDXC_ERR_WORKSPACE;
    DeviceInfo& di = device_info();
    if (!di.ok) return IDXC_ERR_CUDA;
    CUtensorMap q_map;
    if (!encode_operand_map(&q_map, q, n_q * H, d_qk, false, H)) return IDXC_ERR_CUDA;
    if (n_kv >= (int64_t(1) << 31)) return IDXC_ERR_INVALID_ARG;
    g_launches += 2;
    uint8_t* scratch = static_cast<uint8_t*>(workspace) + round_up(n_q * 8, 256);
    void* partial = sparse_attn_partial_bytes(n_q) ? scratch + round_up(sparse_attn_scratch_bytes(n_q, k_top), 256) : nullptr;
    g_launches += partial ? 1 : 0;
    return launch_sparse_attn(kv, topk, kv_base, n_q, n_kv, H, k_top, scale, out, lse, static_cast<int32_t*>(workspace), scratch,
                              partial, q_map, di.status_ptr, di.sm_count, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
               ? IDXC_OK : IDXC_ERR_CUDA;
}

idxc_status idxc_selftest_bounded_wait(uint32_t wait_cycles, void* cuda_stream) {
    if (!device_info().ok) return IDXC_ERR_CUDA;
    const long long budget = wait_cycles > 100000000u ? 100000000LL : static_cast<long long>(wait_cycles);
    g_launches += 1;
    return launch_selftest_bounded_wait(device_info().status_ptr, budget, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
               ? IDXC_OK : IDXC_ERR_CUDA;
}

idxc_status idxc_selftest_tmem_readout(uint32_t accumulators_per_warp, int64_t* bytes_read_out, void* cuda_stream) {
    DeviceInfo& di = device_info();
    if (!di.ok) return IDXC_ERR_CUDA;
    if (accumulators_per_warp == 0 || accumulators_per_warp > (1u << 24)) return IDXC_ERR_INVALID_ARG;
    // each of the 8 reading warps of an SM reads its 32 lanes x 128 columns share of `accumulators_per_warp` accumulators
    if (bytes_read_out) *bytes_read_out = static_cast<int64_t>(di.sm_count) * 8 * accumulators_per_warp * (32 * 128 * 4);
    g_launches += 1;
    // the status word doubles as the sink: the kernel never writes it in practice (see selftest.cu)
    return launch_selftest_tmem_readout(accumulators_per_warp, di.status_ptr, di.sm_count, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
               ? IDXC_OK : IDXC_ERR_CUDA;
}

idxc_status idxc_selftest_tmem_readout_under_mma(uint32_t accumulators_per_warp, int fp8, int64_t* bytes_read_out,
                                                 uint64_t* counters, void* cuda_stream) {
    DeviceInfo& di = device_info();
    if (!di.ok) return IDXC_ERR_CUDA;
    if (accumulators_per_warp == 0 || accumulators_per_warp > (1u << 24) || !counters) return IDXC_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (bytes_read_out) *bytes_read_out = static_cast<int64_t>(di.sm_count) * 8 * accumulators_per_warp * (32 * 128 * 4);
    if (cudaMemsetAsync(counters, 0, 2 * sizeof(uint64_t), stream) != cudaSuccess) return IDXC_ERR_CUDA;
    g_launches += 1;
    return launch_selftest_tmem_readout_mma(accumulators_per_warp, fp8 != 0, di.status_ptr, reinterpret_cast<unsigned long long*>(counters),
                                            di.status_ptr, di.sm_count, stream) == cudaSuccess ? IDXC_OK : IDXC_ERR_CUDA;
}

idxc_status idxc_selftest_issue_rates(uint32_t rounds, uint64_t* cycles, void* cuda_stream) {
    DeviceInfo& di = device_info();
    if (!di.ok) return IDXC_ERR_CUDA;
    if (rounds == 0 || rounds > (1u << 20) || !cycles) return IDXC_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemsetAsync(cycles, 0, IDXC_ISSUE_RATE_KINDS * sizeof(uint64_t), stream) != cudaSuccess) return IDXC_ERR_CUDA;
    g_launches += IDXC_ISSUE_RATE_KINDS;
    // the status word doubles as the sink: the kernels never write it in practice (see selftest.cu)
    return launch_selftest_issue_rates(rounds, reinterpret_cast<unsigned long long*>(cycles), reinterpret_cast<float*>(di.status_ptr),
                                       di.sm_count, stream) == cudaSuccess ? IDXC_OK : IDXC_ERR_CUDA;
}

idxc_status idxc_poll_device_status(void* cuda_stream) {
    if (!device_info().ok) return IDXC_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaStreamSynchronize(stream) != cudaSuccess) return IDXC_ERR_CUDA;
    unsigned int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_device_status, sizeof(v)) != cudaSuccess) return IDXC_ERR_CUDA;
    if (v != 0) {
        const unsigned int zero = 0;
        if (cudaMemcpyToSymbol(g_device_status, &zero, sizeof(zero)) != cudaSuccess) return IDXC_ERR_CUDA;
        return IDXC_ERR_DEVICE_TIMEOUT;
    }
    return IDXC_OK;
}

}  // extern "C"
