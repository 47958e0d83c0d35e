// idxc_indexer_decode_noalloc: the decode step for callers that cannot provide scratch memory.
//
// Some hosts of this library may not allocate device memory at the point where they decode:
// a serving engine that has already handed every free byte of HBM to its KV-cache pool (a
// cudaMalloc there fails), or a latency-critical decode loop in which cudaMalloc / cudaFree
// would stall the whole device. idxc_indexer_decode needs a scratch buffer for the fp32 scores
// between its scoring kernel and its top-k kernel; this variant keeps that scratch in a
// fixed-size array that is part of the library image, so the caller passes inputs and the
// output only.
//
// The array costs IDXC_NOALLOC_SCRATCH_BYTES on every GPU this entry point is used on, for the
// life of the process. CUDA loads a library's device code and data lazily, so the array comes into
// being when the FIRST call on a device looks its address up: that one call makes the driver set
// aside the 16 MiB and must therefore be made while the device still has them free, i.e. before
// the host hands the rest of HBM to its cache pool (a warm-up step at start-up does it). Every
// later call on that device allocates nothing, on the device or on the host. All calls share it: two calls whose kernels may overlap on the GPU (different
// streams, no dependency between them) race on it and give unspecified indices. It keeps the
// previous call's scores; nothing in it has to start at zero, because the scoring kernel writes
// every score the top-k kernel reads before that kernel runs.
#include <cuda_runtime.h>

#include <mutex>

#include "../../include/idxc.h"
#include "kernels.h"

namespace {

// In host code this name is only a handle for the symbol, not an address a kernel could use;
// the device address is looked up once per device below.
static __device__ __align__(256) unsigned char g_noalloc_scratch[IDXC_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_addr[kMaxDevices] = {};   // device address of the array, per device ordinal

// First call on a device: resolve the array's device address with that device current. With lazy module
// loading this lookup is also what makes the driver create the array on that device.
idxc_status scratch_for_current_device(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return IDXC_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return IDXC_ERR_CUDA;
        // The driver also loads a kernel's code when it is first used on a device. Load every kernel a decode step can
        // launch now, so that a later call with another head count, dtype or batch shape finds it resident.
        if (idxc::preload_score_decode_tc() != cudaSuccess || idxc::preload_topk_rows() != cudaSuccess ||
            idxc::preload_topk_rows_cluster() != cudaSuccess || idxc::preload_score_simt() != cudaSuccess)
            return IDXC_ERR_CUDA;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return IDXC_OK;
}

}  // namespace

extern "C" idxc_status idxc_indexer_decode_noalloc(const void* q_step, const void* k_cache, int64_t cache_rows,
                                                   const float* w, const float* q_scale, const float* k_scale,
                                                   const int64_t* k_offsets, const int32_t* lens, int B,
                                                   int64_t max_len, int H_I, int d_I, int k_top, idxc_dtype dt,
                                                   int32_t* topk_out, uint32_t flags, void* cuda_stream) {
    if (B < 0 || max_len < 0 || !topk_out) return IDXC_ERR_INVALID_ARG;
    // the scores of one step must fit the built-in array: B rows of round_up(max_len, 32) floats
    const size_t need = idxc_decode_workspace_bytes(B, max_len, H_I, d_I, k_top, dt, flags);
    if (need > static_cast<size_t>(IDXC_NOALLOC_SCRATCH_BYTES)) return IDXC_ERR_WORKSPACE;
    void* scratch = nullptr;
    idxc_status st = scratch_for_current_device(&scratch);
    if (st != IDXC_OK) return st;
    return idxc_indexer_decode(q_step, k_cache, cache_rows, w, q_scale, k_scale, k_offsets, lens, B, max_len, H_I,
                               d_I, k_top, dt, /*scores_out=*/nullptr, 0, topk_out, scratch,
                               static_cast<size_t>(IDXC_NOALLOC_SCRATCH_BYTES), flags, cuda_stream);
}
