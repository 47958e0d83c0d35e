// Sparse core attention over the indexer's selection (Sec. 2.1: "the main attention is computed only over
// this sparse subset"; Fig. 2: SparseAttn_l(X, T^(l))), multi-query form over a shared latent row per token:
//   out[t,h,:] = sum_j softmax_j(scale * <q[t,h,:], kv[T_t[j], 0:d_qk]>) * kv[T_t[j], 0:d_v]
// for the 128-head, d_qk = 576, d_v = 512 shape of latent attention.
//
// One persistent CTA per SM walks queries. The 128 heads of a query are the M dimension of every UMMA, so a
// thread of the softmax warps owns one head row (no cross-lane reductions). The output accumulator of a
// query, 128 x 512 fp32, is all of tensor memory, so a query is processed in two passes over its selected
// rows, one per 256-column half of d_v; each pass recomputes the scores.
//   tensor memory (512 columns): O half [0,256) | S [256,320) | P as bf16 pairs [320,352) | 5 of the 9
//     64-column blocks of Q as bf16 pairs [352,512) (the A operand of the score MMAs; the other 4 blocks of Q
//     stay in shared memory: there is no room for both a resident Q and two tiles of gathered rows)
//   shared memory: 2 stages x (64 gathered rows x 576 bf16, as 9 blocks of [64 rows x 128 B], 128-byte
//     swizzle) | 4 blocks of Q [128 rows x 128 B]. A block of gathered rows is at once the K-major B operand
//     of S = Q K^T (rows = keys) and the MN-major B operand of O += P V (64 contiguous value columns).
//   warps: 0 MMA issuer, 1 Q loader (TMA), 2-5 row gather (16-byte cp.async into the swizzled layout),
//     6-9 softmax: S from tensor memory, running reference maximum with a lazy rescale of O (only when the
//     maximum grows by more than 2^8), P written back to tensor memory as the A operand of the PV MMAs.
// Entries < 0 or pointing outside the cache are skipped; a query's tiles end at its last usable entry
// (counted by a small kernel first).
#include <cuda_bf16.h>

#include "kernels.h"
#include "ptx_sm100.cuh"

namespace idxc {
namespace {

constexpr int kSaThreads = 320;
constexpr int kSaBK = 64;                 // gathered rows per tile
constexpr int kSaNB = 9;                  // 64-column blocks of d_qk = 576
constexpr int kSaNVH = 4;                 // value blocks per pass (256 columns)
constexpr int kSaQT = 5;                  // Q blocks held in tensor memory
constexpr int kSaQS = kSaNB - kSaQT;      // Q blocks held in shared memory
constexpr uint32_t kSaQBlockBytes = 128 * 128;
constexpr uint32_t kSaKBlockBytes = kSaBK * 128;
constexpr uint32_t kSaStageBytes = kSaNB * kSaKBlockBytes;            // 73728
constexpr uint32_t kSaQSmemBytes = kSaQS * kSaQBlockBytes;            // 65536
constexpr uint32_t kSaSmemBytes = 2 * kSaStageBytes + kSaQSmemBytes + 256 + 1024;
static_assert(kSaQT * kSaQBlockBytes <= 2 * kSaStageBytes, "the Q staging area lives in the tile stages");
constexpr uint32_t kColO = 0, kColS = 256, kColP = 320, kColQ = 352;
constexpr float kRescaleThreshold = 8.f;  // log2 units: P stays below 2^8

struct SaParams {
    const uint8_t* kv;          // [n_kv, 576] bf16
    const int32_t* topk;        // [n_q, k_top]
    const int64_t* kv_base;     // [n_q] or nullptr
    const int32_t* n_eff;       // [n_q] entries to visit per query
    int64_t n_q, n_kv;
    int H, k_top;
    float scale_log2;           // scale * log2(e)
    __nv_bfloat16* out;         // [n_q, H, 512]
    float* lse;                 // [n_q, H] or nullptr
    unsigned int* status;
};

__device__ __forceinline__ void sa_give_up(volatile uint32_t* abort_flag, unsigned int* status, unsigned int code) {
    *abort_flag = 1u;
    atomicCAS(status, 0u, code);
}
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

// n_eff[t] = 1 + position of the last entry of row t that is >= 0 and inside the cache (0 if none).
__global__ void sparse_attn_count_kernel(const int32_t* __restrict__ topk, const int64_t* __restrict__ kv_base, int64_t n_q,
                                         int64_t n_kv, int k_top, int32_t* __restrict__ n_eff) {
    const int64_t t = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (t >= n_q) return;
    const int64_t base = kv_base ? kv_base[t] : 0;
    int last = 0;
    for (int j = lane; j < k_top; j += 32) {
        const int64_t idx = topk[t * k_top + j];
        if (idx >= 0 && base + idx >= 0 && base + idx < n_kv) last = j + 1;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) last = max(last, __shfl_xor_sync(0xFFFFFFFFu, last, o));
    if (lane == 0) n_eff[t] = last;
}

__global__ void __launch_bounds__(kSaThreads, 1)
sparse_attn_kernel(const __grid_constant__ CUtensorMap q_map, const SaParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t* stage_smem = smem;                               // [2][9][64 x 128 B]; Q blocks 0..4 are staged here first
    uint8_t* q_smem = smem + 2 * kSaStageBytes;               // [4][128 x 128 B]: Q blocks 5..8
    uint64_t* bars = reinterpret_cast<uint64_t*>(q_smem + kSaQSmemBytes);
    const uint32_t bar_q_full = smem_u32(bars + 0);
    const uint32_t bar_q_ready = smem_u32(bars + 1);          // Q blocks 0..4 copied to tensor memory, staging free
    const uint32_t bar_q_empty = smem_u32(bars + 2);
    const uint32_t bar_kv_full = smem_u32(bars + 3);          // [2]
    const uint32_t bar_kv_empty = smem_u32(bars + 5);         // [2]
    const uint32_t bar_s_full = smem_u32(bars + 7);
    const uint32_t bar_p_ready = smem_u32(bars + 8);
    const uint32_t bar_o_full = smem_u32(bars + 9);
    const uint32_t bar_o_free = smem_u32(bars + 10);
    uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(bars + 11);
    volatile uint32_t* abort_flag = tmem_base_slot + 1;
    volatile uint16_t* tile_mask = reinterpret_cast<volatile uint16_t*>(bars + 12);   // [2 stages][4 gather warps]

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        mbar_init(bar_q_full, 1);
        mbar_init(bar_q_ready, 4);
        mbar_init(bar_q_empty, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar_kv_full + 8 * i, 4);
            mbar_init(bar_kv_empty + 8 * i, 1);
        }
        mbar_init(bar_s_full, 1);
        mbar_init(bar_p_ready, 4);
        mbar_init(bar_o_full, 1);
        mbar_init(bar_o_free, 4);
        *abort_flag = 0u;
        fence_mbar_init();
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(tmem_base_slot), 512);
        tmem_relinquish_alloc_permit();
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    tcgen05_fence_after_sync();
    const uint32_t tmem_base = *tmem_base_slot;

    auto tiles_of = [&](int64_t t) -> int { return (__ldg(p.n_eff + t) + kSaBK - 1) / kSaBK; };

    if (warp == 0) {
        if (lane == 0) {
            // ------------------------------------------------------------ MMA issuer
            constexpr uint32_t kIdescS = umma_idesc(1, 1, 128, kSaBK);
            constexpr uint32_t kIdescPV = umma_idesc(1, 1, 128, 64 * kSaNVH) | kUmmaBMajorMN;
            uint32_t ph_q_full = 0, ph_q_ready = 0, ph_p_ready = 0, ph_o_free = 0;
            uint32_t ph_kv_full[2] = {0u, 0u};
            int stage = 0;
            bool ok = true;
            for (int64_t t = blockIdx.x; t < p.n_q && ok; t += gridDim.x) {
                const int nt = tiles_of(t);
                if (nt == 0) continue;
                ok = mbar_wait(bar_q_full, ph_q_full, abort_flag) && mbar_wait(bar_q_ready, ph_q_ready, abort_flag);
                if (!ok) break;
                ph_q_full ^= 1u;
                ph_q_ready ^= 1u;
                for (int half = 0; half < 2 && ok; ++half) {
                    ok = mbar_wait(bar_o_free, ph_o_free ^ 1u, abort_flag);    // the previous pass's O has been read out
                    if (!ok) break;
                    ph_o_free ^= 1u;
                    for (int i = 0; i < nt; ++i) {
                        ok = mbar_wait(bar_kv_full + 8 * stage, ph_kv_full[stage], abort_flag);
                        if (!ok) break;
                        ph_kv_full[stage] ^= 1u;
                        tcgen05_fence_after_sync();
                        const uint32_t tile = smem_u32(stage_smem + stage * kSaStageBytes);
                        // S = Q K^T over the 9 column blocks
#pragma unroll
                        for (int b = 0; b < kSaNB; ++b) {
#pragma unroll
                            for (int ks = 0; ks < 4; ++ks) {
                                const uint64_t b_desc = umma_smem_desc_sw128(tile + b * kSaKBlockBytes + ks * 32);
                                if (b < kSaQT)
                                    umma_f16_ts(tmem_base + kColS, tmem_base + kColQ + b * 32 + ks * 8, b_desc, kIdescS, (b | ks) != 0);
                                else
                                    umma_f16(tmem_base + kColS,
                                             umma_smem_desc_sw128(smem_u32(q_smem + (b - kSaQT) * kSaQBlockBytes) + ks * 32), b_desc,
                                             kIdescS, 1u);
                            }
                        }
                        umma_commit(bar_s_full);
                        ok = mbar_wait(bar_p_ready, ph_p_ready, abort_flag);
                        if (!ok) break;
                        ph_p_ready ^= 1u;
                        tcgen05_fence_after_sync();
                        // O[:, 256 half .. +256] += P V: 16 gathered rows per MMA
#pragma unroll
                        for (int ks = 0; ks < kSaBK / 16; ++ks) {
                            const uint64_t v_desc = umma_smem_desc_sw128_mn(
                                tile + (half * kSaNVH) * kSaKBlockBytes + ks * 16 * 128, kSaKBlockBytes);
                            umma_f16_ts(tmem_base + kColO, tmem_base + kColP + ks * 8, v_desc, kIdescPV, (i | ks) != 0);
                        }
                        umma_commit(bar_kv_empty + 8 * stage);
                        if (i == nt - 1) umma_commit(bar_o_full);
                        stage ^= 1;
                    }
                }
                if (ok) umma_commit(bar_q_empty);
            }
            if (!ok) sa_give_up(abort_flag, p.status, DEV_TIMEOUT_MMA);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ------------------------------------------------------------ Q loader
            tma_prefetch_desc(&q_map);
            uint32_t ph_q_empty = 0;
            bool ok = true;
            for (int64_t t = blockIdx.x; t < p.n_q; t += gridDim.x) {
                if (tiles_of(t) == 0) continue;
                ok = mbar_wait(bar_q_empty, ph_q_empty ^ 1u, abort_flag);   // every MMA of the previous query is done
                if (!ok) break;
                ph_q_empty ^= 1u;
                mbar_arrive_expect_tx(bar_q_full, static_cast<uint32_t>(kSaNB * p.H * 128));
                const int row0 = static_cast<int>(t * p.H);
                for (int b = 0; b < kSaNB; ++b) {
                    uint8_t* dst = b < kSaQT ? stage_smem + b * kSaQBlockBytes : q_smem + (b - kSaQT) * kSaQBlockBytes;
                    tma_load_2d(smem_u32(dst), &q_map, bar_q_full, b * 64, row0);
                }
            }
            if (!ok) sa_give_up(abort_flag, p.status, DEV_TIMEOUT_PRODUCER);
        }
    } else if (warp < 6) {
        // ---------------------------------------------------------------- row gather
        const int gw = warp - 2;                      // rows 16 gw .. 16 gw + 15 of every tile
        uint32_t ph_q_ready = 0;
        uint32_t ph_kv_empty[2] = {0u, 0u};
        int stage = 0;
        bool ok = true;
        for (int64_t t = blockIdx.x; t < p.n_q && ok; t += gridDim.x) {
            const int nt = tiles_of(t);
            if (nt == 0) continue;
            ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar_q_ready, ph_q_ready, abort_flag));   // the staging area is free again
            if (!ok) break;
            ph_q_ready ^= 1u;
            const int64_t base = p.kv_base ? __ldg(p.kv_base + t) : 0;
            const int32_t* row_idx = p.topk + t * p.k_top;
            for (int half = 0; half < 2 && ok; ++half) {
                for (int i = 0; i < nt; ++i) {
                    ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar_kv_empty + 8 * stage, ph_kv_empty[stage] ^ 1u, abort_flag));
                    if (!ok) break;
                    ph_kv_empty[stage] ^= 1u;
                    // lanes 0..15 look up this warp's rows
                    const int j = i * kSaBK + gw * 16 + (lane & 15);
                    int64_t src_row = -1;
                    if (j < p.k_top) {
                        const int64_t idx = __ldg(row_idx + j);
                        if (idx >= 0 && base + idx >= 0 && base + idx < p.n_kv) src_row = base + idx;
                    }
                    const uint32_t valid = __ballot_sync(0xFFFFFFFFu, src_row >= 0) & 0xFFFFu;
                    if (src_row < 0) src_row = 0;             // skipped entries load row 0 and are masked later
                    uint8_t* tile = stage_smem + stage * kSaStageBytes;
#pragma unroll 4
                    for (int rr = 0; rr < 16; ++rr) {
                        const int64_t r_src = __shfl_sync(0xFFFFFFFFu, src_row, rr);
                        const uint8_t* src = p.kv + r_src * (kSaNB * 128);
                        const int r = gw * 16 + rr;
#pragma unroll
                        for (int c = lane; c < kSaNB * 8; c += 32) {      // 72 chunks of 16 bytes per row
                            const int b = c >> 3, ch = c & 7;
                            cp_async_16(smem_u32(tile + b * kSaKBlockBytes + r * 128 + ((ch ^ (r & 7)) << 4)), src + c * 16);
                        }
                    }
                    if (lane == 0) tile_mask[stage * 4 + gw] = static_cast<uint16_t>(valid);
                    cp_async_wait_all();
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_kv_full + 8 * stage);
                    stage ^= 1;
                }
            }
        }
        cp_async_wait_all();
        if (!ok && lane == 0) sa_give_up(abort_flag, p.status, DEV_TIMEOUT_GATHER);
    } else {
        // ---------------------------------------------------------------- softmax and output
        const int quarter = warp & 3;                  // TMEM lane quarter this warp may access
        const int row = quarter * 32 + lane;           // head
        const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        uint32_t ph_q_full = 0, ph_s_full = 0, ph_o_full = 0;
        int stage = 0;
        bool ok = true;
        for (int64_t t = blockIdx.x; t < p.n_q && ok; t += gridDim.x) {
            const int nt = tiles_of(t);
            __nv_bfloat16* out_row = p.out + (t * p.H + row) * 512;
            if (nt == 0) {                              // nothing selected: zeros
                if (row < p.H) {
                    for (int c = 0; c < 512 / 8; ++c) reinterpret_cast<uint4*>(out_row)[c] = make_uint4(0u, 0u, 0u, 0u);
                    if (p.lse) p.lse[t * p.H + row] = -INFINITY;
                }
                continue;
            }
            // ---- Q blocks 0..4: staging (swizzled rows) -> tensor memory, two bf16 per column
            ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar_q_full, ph_q_full, abort_flag));
            if (!ok) break;
            ph_q_full ^= 1u;
#pragma unroll 1
            for (int b = 0; b < kSaQT; ++b) {
                uint32_t r[32];
                const uint8_t* src = stage_smem + b * kSaQBlockBytes + row * 128;
#pragma unroll
                for (int ch = 0; ch < 8; ++ch) {
                    const uint4 v = *reinterpret_cast<const uint4*>(src + ((ch ^ (row & 7)) << 4));
                    r[4 * ch + 0] = v.x; r[4 * ch + 1] = v.y; r[4 * ch + 2] = v.z; r[4 * ch + 3] = v.w;
                }
                tmem_st_32x32b_x32(lane_base + kColQ + b * 32, r);
            }
            tmem_st_wait();
            tcgen05_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_q_ready);

            float lse_val = 0.f;
            for (int half = 0; half < 2 && ok; ++half) {
                float m_ref = -INFINITY, l = 0.f;
                for (int i = 0; i < nt; ++i) {
                    ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar_s_full, ph_s_full, abort_flag));
                    if (!ok) break;
                    ph_s_full ^= 1u;
                    tcgen05_fence_after_sync();
                    uint32_t sa[32], sb[32];
                    tmem_ld_32x32b_x32(lane_base + kColS, sa);
                    tmem_ld_32x32b_x32(lane_base + kColS + 32, sb);
                    tmem_ld_wait(sa);
                    tmem_ld_wait(sb);
                    const uint32_t mlo = static_cast<uint32_t>(tile_mask[stage * 4 + 0]) | (static_cast<uint32_t>(tile_mask[stage * 4 + 1]) << 16);
                    const uint32_t mhi = static_cast<uint32_t>(tile_mask[stage * 4 + 2]) | (static_cast<uint32_t>(tile_mask[stage * 4 + 3]) << 16);
                    float mt = -INFINITY;
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const float xa = (mlo >> j) & 1u ? __uint_as_float(sa[j]) * p.scale_log2 : -INFINITY;
                        const float xb = (mhi >> j) & 1u ? __uint_as_float(sb[j]) * p.scale_log2 : -INFINITY;
                        sa[j] = __float_as_uint(xa);
                        sb[j] = __float_as_uint(xb);
                        mt = fmaxf(mt, fmaxf(xa, xb));
                    }
                    // lazy reference maximum: move it only when the row maximum outgrew it by 2^8
                    const bool move = mt > m_ref + kRescaleThreshold;      // also true for the first usable score (m_ref = -inf)
                    if (__any_sync(0xFFFFFFFFu, move)) {
                        float alpha = 1.f;
                        if (move) {
                            alpha = m_ref == -INFINITY ? 0.f : fast_exp2(m_ref - mt);
                            m_ref = mt;
                            l *= alpha;
                        }
                        if (i > 0) {                                       // every earlier PV MMA is complete (S was committed after them)
#pragma unroll 1
                            for (int c = 0; c < 8; ++c) {
                                uint32_t o[32];
                                tmem_ld_32x32b_x32(lane_base + kColO + c * 32, o);
                                tmem_ld_wait(o);
#pragma unroll
                                for (int j = 0; j < 32; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * alpha);
                                tmem_st_32x32b_x32(lane_base + kColO + c * 32, o);
                            }
                        }
                    }
                    const float m_sub = m_ref == -INFINITY ? 0.f : m_ref;   // no usable score yet: every P is exp2(-inf) = 0
                    uint32_t pr[32];
                    float sum = 0.f;
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const float p0 = fast_exp2(__uint_as_float(sa[2 * j]) - m_sub), p1 = fast_exp2(__uint_as_float(sa[2 * j + 1]) - m_sub);
                        const float p2 = fast_exp2(__uint_as_float(sb[2 * j]) - m_sub), p3 = fast_exp2(__uint_as_float(sb[2 * j + 1]) - m_sub);
                        sum += (p0 + p1) + (p2 + p3);
                        pr[j] = pack_bf16x2(p0, p1);
                        pr[16 + j] = pack_bf16x2(p2, p3);
                    }
                    l += sum;
                    tmem_st_32x32b_x32(lane_base + kColP, pr);
                    tmem_st_wait();
                    tcgen05_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_p_ready);
                    stage ^= 1;
                }
                if (!ok) break;
                // ---- this pass's 256 output columns
                ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar_o_full, ph_o_full, abort_flag));
                if (!ok) break;
                ph_o_full ^= 1u;
                tcgen05_fence_after_sync();
                const float inv = l > 0.f ? 1.f / l : 0.f;
#pragma unroll 1
                for (int c = 0; c < 8; ++c) {
                    uint32_t o[32];
                    tmem_ld_32x32b_x32(lane_base + kColO + c * 32, o);
                    tmem_ld_wait(o);
                    if (row < p.H) {
                        uint4* dst = reinterpret_cast<uint4*>(out_row + half * 256 + c * 32);
#pragma unroll
                        for (int v = 0; v < 4; ++v) {
                            uint4 w;
                            w.x = pack_bf16x2(__uint_as_float(o[8 * v + 0]) * inv, __uint_as_float(o[8 * v + 1]) * inv);
                            w.y = pack_bf16x2(__uint_as_float(o[8 * v + 2]) * inv, __uint_as_float(o[8 * v + 3]) * inv);
                            w.z = pack_bf16x2(__uint_as_float(o[8 * v + 4]) * inv, __uint_as_float(o[8 * v + 5]) * inv);
                            w.w = pack_bf16x2(__uint_as_float(o[8 * v + 6]) * inv, __uint_as_float(o[8 * v + 7]) * inv);
                            dst[v] = w;
                        }
                    }
                }
                tcgen05_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_o_free);
                if (half == 0) lse_val = l > 0.f ? (m_ref + log2f(l)) * 0.6931471805599453f : -INFINITY;
            }
            if (ok && p.lse && row < p.H) p.lse[t * p.H + row] = lse_val;
        }
        if (!ok && lane == 0) sa_give_up(abort_flag, p.status, DEV_TIMEOUT_EPILOGUE);
    }

    // ------------------------------------------------------------------- teardown
    __syncwarp();
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        tcgen05_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
}

}  // namespace

bool sparse_attn_supported(int H, int d_qk, int d_v) { return H >= 1 && H <= 128 && d_qk == 64 * kSaNB && d_v == 128 * kSaNVH; }

cudaError_t launch_sparse_attn(const void* kv, const int32_t* topk, const int64_t* kv_base, int64_t n_q, int64_t n_kv, int H,
                               int k_top, float scale, void* out, float* lse, int32_t* n_eff, const CUtensorMap& q_map,
                               unsigned int* status, int sm_count, cudaStream_t stream) {
    if (n_q <= 0) return cudaSuccess;
    const int64_t count_blocks = (n_q * 32 + 255) / 256;
    sparse_attn_count_kernel<<<static_cast<unsigned>(count_blocks), 256, 0, stream>>>(topk, kv_base, n_q, n_kv, k_top, n_eff);
    if (cudaError_t e = cudaGetLastError(); e != cudaSuccess) return e;
    if (cudaError_t e = ensure_max_dynamic_smem(reinterpret_cast<const void*>(sparse_attn_kernel), kSaSmemBytes); e != cudaSuccess) return e;
    SaParams p{static_cast<const uint8_t*>(kv), topk, kv_base, n_eff, n_q, n_kv, H, k_top, scale * 1.4426950408889634f,
               static_cast<__nv_bfloat16*>(out), lse, status};
    const int grid = static_cast<int>(n_q < sm_count ? n_q : sm_count);
    sparse_attn_kernel<<<grid, kSaThreads, kSaSmemBytes, stream>>>(q_map, p);
    return cudaGetLastError();
}

}  // namespace idxc
