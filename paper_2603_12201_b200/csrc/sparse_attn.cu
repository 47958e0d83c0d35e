// Sparse core attention over the indexer's selection (Sec. 2.1: "the main attention is computed only over
// this sparse subset"; Fig. 2: SparseAttn_l(X, T^(l))), multi-query form over a shared latent row per token:
//   out[t,h,:] = sum_j softmax_j(scale * <q[t,h,:], kv[T_t[j], 0:d_qk]>) * kv[T_t[j], 0:d_v]
// for the 128-head, d_qk = 576, d_v = 512 shape of latent attention.
//
// One persistent CTA per SM walks queries. The 128 heads of a query are the M dimension of every UMMA, so a
// thread of the softmax warps owns one head row (no cross-lane reductions). The output accumulator of a
// query, 128 x 512 fp32, is all of tensor memory, so a query takes two passes over its selected rows, one per
// 256-column half of d_v:
//   pass 1  gathers whole rows (576 columns), S = Q K^T, softmax, O[:, 0:256] += P V; the bf16 probabilities P
//           and the rescale factors of the running maximum also go to a per-CTA scratch area in global memory
//   pass 2  gathers only columns 256..511 of the same rows and does O[:, 256:512] += P V with the saved P and the
//           same sequence of rescales: no second score product, half the gather bytes. A saved tile of P is stored
//           as [16-byte chunk][row][16 B], which is at once what a warp of softmax threads writes contiguously and
//           the unswizzled K-major operand layout, so one bulk copy per tile brings it back (four tiles ahead, into
//           the shared memory that held Q) and the PV MMAs read it there: no thread touches P in pass 2. The softmax
//           warps note in pass 1 which tiles moved a reference maximum; only those tiles wait for them in pass 2.
// Tensor memory (512 columns): O half of pass 1 [0,256) | S double-buffered [256,320), [320,384); in pass 1 P overwrites
//   the first 32 columns of its S buffer as bf16 pairs and is the A operand of the PV MMAs | Q blocks 0..3 (of 9 blocks
//   of 64 columns) as bf16 pairs [384,512), the A operand of their score MMAs; Q blocks 4..8 stay in shared memory.
//   Pass 2 accumulates its half of O in [256,512): S and Q are not needed then, and pass 1's half can still be read out.
// Shared memory: 2 stages x 9 blocks of [64 gathered rows x 128 B] (128-byte swizzle) | 5 blocks of Q
//   [128 rows x 128 B]. A block of gathered rows is at once the K-major B operand of S (rows = keys) and the
//   MN-major B operand of P V (64 contiguous value columns). A stage is two slots with their own barriers:
//   "V" = blocks 0..3 (needed until the PV product) and "E" = blocks 4..8 (free again once the scores are
//   done), so the next tile's E part is gathered while this tile is still in its softmax. Pass 2 uses the four
//   slots as a ring of four value tiles.
// Warps (16; three idle): 0 MMA issuer (warp-uniform, one elected lane issues; order S(i+1) blocks 4..8 | P(i) V(i) |
//   S(i+1) blocks 0..3), 4 Q loader (TMA) and, in pass 2, loader of the saved P, eight row-gather warps (16-byte
//   cp.async into the swizzled layout; two warps per slot, each slot its own acquire/copy/publish stream), 12-15
//   softmax (running reference maximum with a lazy rescale of O, only when the maximum grows by more than 2^8).
// The hot loops are rolled on purpose: with everything unrolled the kernel was 150 KB of code and every role
// stalled on instruction fetch.
// Entries < 0 or pointing outside the cache are skipped; a query's tiles end at its last usable entry
// (counted by a small kernel first).
#include <cuda_bf16.h>

#include "kernels.h"
#include "ptx_sm100.cuh"

namespace idxc {
namespace {

constexpr int kSaGatherWarps = 8;          // warps 1 2 3 5 6 7 9 10
constexpr int kSaThreads = 32 * 16;
static_assert(kSaGatherWarps == 8, "two gather warps per slot, four slots");
constexpr int kSaBK = 64;                 // gathered rows per tile
constexpr int kSaNB = 9;                  // 64-column blocks of d_qk = 576
constexpr int kSaNVH = 4;                 // value blocks per pass (256 columns)
constexpr int kSaQT = 4;                  // Q blocks held in tensor memory (blocks 0..3)
constexpr int kSaQS = kSaNB - kSaQT;      // Q blocks held in shared memory (blocks 4..8)
constexpr uint32_t kSaQBlockBytes = 128 * 128;
constexpr uint32_t kSaKBlockBytes = kSaBK * 128;
constexpr uint32_t kSaStageBytes = kSaNB * kSaKBlockBytes;            // 73728
constexpr uint32_t kSaQSmemBytes = kSaQS * kSaQBlockBytes;            // 81920
constexpr uint32_t kSaBarBytes = 512;     // mbarriers and a few words of per-query state
constexpr uint32_t kSaSmemBytes = 2 * kSaStageBytes + kSaQSmemBytes + kSaBarBytes + 1024;
constexpr int kSaFlagTiles = 256;         // tiles of a query whose "rescaled" flag is kept; later tiles count as flagged
static_assert(kSaQT * kSaQBlockBytes <= 2 * kSaStageBytes, "the Q staging area lives in the tile stages");
static_assert(kSaSmemBytes <= 232448, "shared memory budget of one CTA");
constexpr int kSaPRing = 4;               // pass 2: saved P tiles in flight
constexpr uint32_t kColO = 0, kColS = 256, kColQ = 384;   // S buffer b at kColS + 64 b; P in its first 32 columns
constexpr uint32_t kColO2 = 256;          // pass 2 accumulates over the S and Q columns (unused then), so it need not wait for pass 1's read-out
constexpr float kRescaleThreshold = 8.f;  // log2 units: P stays below 2^8
constexpr uint32_t kSaPTileBytes = 128 * kSaBK * 2;
constexpr uint32_t kSaScratchTileBytes = kSaPTileBytes + 128 * 4;     // P as [8 chunks][128 rows][16 B] + rescale factors [128] fp32
static_assert(kSaPRing * kSaPTileBytes <= kSaQSmemBytes && kSaScratchTileBytes % 16 == 0, "the P ring lives where Q blocks 4..8 were");

struct SaParams {
    const uint8_t* kv;          // [n_kv, 576] bf16
    const int32_t* topk;        // [n_q, k_top]
    const int64_t* kv_base;     // [n_q] or nullptr
    const int32_t* n_eff;       // [n_q][2] entries to visit per query, cache row of its first usable entry
    uint8_t* scratch;           // [grid][tiles per query][kSaScratchTileBytes]
    int64_t n_q, n_kv;
    int H, k_top;
    float scale_log2;           // scale * log2(e)
    __nv_bfloat16* out;         // [n_q, H, 512]
    float* lse;                 // [n_q, H] or nullptr
    int splits;                 // CTAs that share a query's selected rows (few queries: decode); 1 = the CTA writes out itself
    float* part_out;            // splits > 1: [n_q, splits, H, 512] fp32, each split's own normalised result
    float* part_lse;            // splits > 1: [n_q, splits, H] natural-log sum of the split (-inf: nothing usable)
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

// n_eff[2t] = 1 + position of the last entry of row t that is >= 0 and inside the cache (0 if none);
// n_eff[2t+1] = the cache row of its first usable entry (stands in for skipped entries, with weight 0: rows that
// are not selected are never read).
constexpr int kSaCountThreads = 128;
__global__ void __launch_bounds__(kSaCountThreads)
sparse_attn_count_kernel(const int32_t* __restrict__ topk, const int64_t* __restrict__ kv_base, int64_t n_q, int64_t n_kv, int k_top,
                         int32_t* __restrict__ n_eff) {
    // one CTA per query: a decode step has few queries, and a single warp walking a row is one long chain of dependent loads
    const int64_t t = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t base = kv_base ? kv_base[t] : 0;
    const int32_t* row = topk + t * k_top;
    int last = 0;
    unsigned long long first = ~0ull;          // (position << 32) | cache row of the first usable entry
#pragma unroll 4
    for (int j = threadIdx.x; j < k_top; j += kSaCountThreads) {
        const int64_t idx = __ldg(row + j);
        if (idx >= 0 && base + idx >= 0 && base + idx < n_kv) {
            last = j + 1;
            if (first == ~0ull) first = (static_cast<unsigned long long>(j) << 32) | static_cast<unsigned long long>(base + idx);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        last = max(last, __shfl_xor_sync(0xFFFFFFFFu, last, o));
        const unsigned long long other = __shfl_xor_sync(0xFFFFFFFFu, first, o);
        first = other < first ? other : first;
    }
    __shared__ int s_last[kSaCountThreads / 32];
    __shared__ unsigned long long s_first[kSaCountThreads / 32];
    if (lane == 0) { s_last[warp] = last; s_first[warp] = first; }
    __syncthreads();
    if (threadIdx.x == 0) {
#pragma unroll
        for (int w = 1; w < kSaCountThreads / 32; ++w) {
            last = max(last, s_last[w]);
            first = s_first[w] < first ? s_first[w] : first;
        }
        n_eff[2 * t] = last;
        n_eff[2 * t + 1] = last ? static_cast<int32_t>(first & 0xFFFFFFFFull) : 0;
    }
}

__global__ void __launch_bounds__(kSaThreads, 1)
sparse_attn_kernel(const __grid_constant__ CUtensorMap q_map, const SaParams p) {
    extern __shared__ uint8_t smem_raw[];
    // aligned by an offset into the array (not by an integer round trip), so that the compiler still knows that these
    // pointers are shared memory and emits shared-space loads and stores for them
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint8_t* stage_smem = smem;                               // [2][9][64 x 128 B]; Q blocks 0..3 are staged here first
    uint8_t* q_smem = smem + 2 * kSaStageBytes;               // [5][128 x 128 B]: Q blocks 4..8
    uint64_t* bars = reinterpret_cast<uint64_t*>(q_smem + kSaQSmemBytes);
    const uint32_t bar_q_full = smem_u32(bars + 0);
    const uint32_t bar_q_ready = smem_u32(bars + 1);          // Q blocks 0..3 copied to tensor memory, staging free
    const uint32_t bar_q_empty = smem_u32(bars + 2);
    // slot = 2 * stage + group, group 0 = "V" (blocks 0..3), group 1 = "E" (blocks 4..8)
    const uint32_t bar_slot_full = smem_u32(bars + 3);        // [4]
    const uint32_t bar_slot_empty = smem_u32(bars + 7);       // [4]
    const uint32_t bar_s_full = smem_u32(bars + 11);          // [2] S buffers
    const uint32_t bar_p_ready = smem_u32(bars + 13);         // [4] pass 1 uses two (P in its S buffer); pass 2: rescales of tile i replayed, ring of four
    const uint32_t bar_p_free = smem_u32(bars + 17);          // [4] pass 2: the PV product has read P ring buffer b
    const uint32_t bar_o_full = smem_u32(bars + 21);          // pass 1's half of O is complete
    const uint32_t bar_o_free = smem_u32(bars + 22);
    const uint32_t bar_pv_done = smem_u32(bars + 23);         // one phase per PV tile
    uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(bars + 24);
    volatile uint32_t* abort_flag = tmem_base_slot + 1;
    volatile uint32_t* tile_mask = reinterpret_cast<volatile uint32_t*>(bars + 25);   // [2 stages][2]: usable entries of the tile, rows 0..31 and 32..63
    const uint32_t bar_p_full = smem_u32(bars + 27);          // [4] pass 2: the saved P tile has landed in ring buffer b
    const uint32_t bar_p2_go = smem_u32(bars + 31);           // pass 1 is over: P is in the scratch area and Q's shared memory is free
    // bit i: some row's reference maximum moved at tile i of the current query (O must be rescaled before PV(i))
    volatile uint32_t* resc_mask = reinterpret_cast<volatile uint32_t*>(bars + 32);   // [kSaFlagTiles / 32]
    const uint32_t bar_resc_go = smem_u32(bars + 36);         // pass 2: every PV product before a flagged tile is complete
    // Pass 2's half of O is complete. A barrier of its own: pass 2 does not wait for the softmax warps (unless a tile is
    // flagged), so with few tiles it can end before a warp has even looked at pass 1's completion; on one barrier that
    // warp would find the phase it waits for two completions back, which a parity wait cannot tell from "not yet".
    const uint32_t bar_o2_full = smem_u32(bars + 37);
    static_assert(38 * 8 <= kSaBarBytes && kSaFlagTiles / 8 <= 32, "barrier area");
    auto tile_rescales = [&](int i) -> bool { return i > 0 && (i >= kSaFlagTiles || ((resc_mask[i >> 5] >> (i & 31)) & 1u)); };

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    // Roles by warp. A warp's scheduler is warp % 4: the MMA warp shares its scheduler with the loader (mostly asleep),
    // an idle warp and one softmax warp only, so that its issue slots are not taken by polling or copying warps.
    //   0 MMA | 4 loader | 8, 11 idle | 1 2 3 5 6 7 9 10 gather | 12..15 softmax (TMEM lane quarter = warp % 4)
    const int gather_index = warp < 4 ? warp - 1 : (warp < 8 ? warp - 2 : warp - 3);   // for warps 1 2 3 5 6 7 9 10
    const bool is_gather = warp != 0 && warp != 4 && warp != 8 && warp < 11;
    // L2 residency: the cache rows (read again by later queries) and the saved probabilities (read back within the
    // query) are kept in preference to q and the output, which stream through once
    const uint64_t pol_keep = l2_policy_evict_last();
    const uint64_t pol_stream = l2_policy_evict_first();

    if (threadIdx.x == 0) {
        mbar_init(bar_q_full, 1);
        mbar_init(bar_q_ready, 4);
        mbar_init(bar_q_empty, 1);
        for (int i = 0; i < 4; ++i) {
            mbar_init(bar_slot_full + 8 * i, 2);         // one arrive per gather warp of the slot
            mbar_init(bar_slot_empty + 8 * i, 1);
        }
        for (int i = 0; i < 2; ++i) mbar_init(bar_s_full + 8 * i, 1);
        for (int i = 0; i < 4; ++i) {
            mbar_init(bar_p_ready + 8 * i, 4);
            mbar_init(bar_p_free + 8 * i, 1);
            mbar_init(bar_p_full + 8 * i, 1);
        }
        mbar_init(bar_p2_go, 4);
        mbar_init(bar_resc_go, 1);
        mbar_init(bar_o_full, 1);
        mbar_init(bar_o2_full, 1);
        mbar_init(bar_o_free, 4);
        mbar_init(bar_pv_done, 1);
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

    auto tiles_of = [&](int64_t t) -> int { return (__ldg(p.n_eff + 2 * t) + kSaBK - 1) / kSaBK; };
    // work item = (query t, split s): split s of a query covers its tiles [nt * s / splits, nt * (s + 1) / splits)
    const int64_t n_items = p.n_q * p.splits;
    auto item_of = [&](int64_t item, int64_t& t, int& i0) -> int {
        t = item / p.splits;
        const int s = static_cast<int>(item - t * p.splits);
        const int nt_all = tiles_of(t);
        i0 = nt_all * s / p.splits;
        return nt_all * (s + 1) / p.splits - i0;
    };
    // first block of a slot's data inside the stage area
    auto slot_smem = [&](int slot) -> uint8_t* { return stage_smem + (slot >> 1) * kSaStageBytes + (slot & 1) * (kSaNVH * kSaKBlockBytes); };
    const int tiles_per_query = (p.k_top + kSaBK - 1) / kSaBK;
    uint8_t* scratch = p.scratch + static_cast<size_t>(blockIdx.x) * tiles_per_query * kSaScratchTileBytes;

    if (warp == 0) {
        // ---------------------------------------------------------------- MMA issuer
        // The whole warp runs this role with uniform control flow and one elected lane issues each MMA (see
        // umma_f16_elect); descriptors are a per-tile base plus compile-time offsets in 16-byte units.
        constexpr uint32_t kIdescS = umma_idesc(1, 1, 128, kSaBK);
        constexpr uint32_t kIdescPV = umma_idesc(1, 1, 128, 64 * kSaNVH) | kUmmaBMajorMN;
        uint32_t ph_q_full = 0, ph_q_ready = 0, ph_o_free = 0;
        uint32_t ph_slot_full[4] = {0u, 0u, 0u, 0u}, ph_p_ready[4] = {0u, 0u, 0u, 0u}, ph_p_full[4] = {0u, 0u, 0u, 0u};
        int stage_s = 0, stage_pv = 0;      // pass 1: stage of the next tile to score / to multiply by V
        bool ok = true;
        const uint64_t q_desc0 = umma_smem_desc_sw128(smem_u32(q_smem));
        auto wait_bar = [&](uint32_t bar, uint32_t parity) -> bool {
            return __all_sync(0xFFFFFFFFu, mbar_wait(bar, parity, abort_flag));
        };
        auto wait_slot = [&](int slot) -> bool {
            if (!wait_bar(bar_slot_full + 8 * slot, ph_slot_full[slot])) return false;
            ph_slot_full[slot] ^= 1u;
            tcgen05_fence_after_sync();
            return true;
        };
        // 16 gathered rows per MMA; P (bf16 pairs) starts at tensor-memory column p_col
        auto issue_pv = [&](uint32_t v_blocks, uint32_t p_col, bool first_tile) {
            const uint64_t v_desc0 = umma_smem_desc_sw128_mn(v_blocks, kSaKBlockBytes);
#pragma unroll
            for (int ks = 0; ks < kSaBK / 16; ++ks)
                umma_f16_ts_elect_acc(tmem_base + kColO, tmem_base + p_col + ks * 8, v_desc0 + (ks * 16 * 128) / 16, kIdescPV,
                                      (first_tile && ks == 0) ? 0u : 1u);
        };
        for (int64_t item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
            int64_t t;
            int i0;
            const int nt = item_of(item, t, i0);
            if (nt == 0) continue;
            ok = wait_bar(bar_q_full, ph_q_full) && wait_bar(bar_q_ready, ph_q_ready);
            if (!ok) break;
            ph_q_full ^= 1u;
            ph_q_ready ^= 1u;
            // ---- pass 1: scores and the first half of the output
            ok = wait_bar(bar_o_free, ph_o_free ^ 1u);        // the previous query's second half (and so all of its O) has been read out
            if (!ok) break;
            ph_o_free ^= 1u;
            // Issue order: S(i+1) blocks 4..8 | P(i) V(i) | S(i+1) blocks 0..3. The first part keeps the tensor pipe busy
            // while the softmax warps turn S(i) into P(i); the PV product comes before the second part so that
            // its value slot is free again (and refilled) well before the tile after next needs it.
            auto issue_s_e = [&](int i) -> bool {            // blocks 4..8 against Q in shared memory
                if (!wait_slot(2 * stage_s + 1)) return false;
                const uint32_t s_tmem = tmem_base + kColS + (i & 1) * 64;
                const uint64_t k_desc0 = umma_smem_desc_sw128(smem_u32(stage_smem + stage_s * kSaStageBytes));
                // rolled over the blocks: the instruction footprint of the issuing warp stays small
                uint64_t a_desc = q_desc0, b_desc = k_desc0 + (kSaQT * kSaKBlockBytes) / 16;
#pragma unroll 1
                for (int b = kSaQT; b < kSaNB; ++b) {
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        umma_f16_elect_acc(s_tmem, a_desc + (ks * 32) / 16, b_desc + (ks * 32) / 16, kIdescS, (b != kSaQT || ks != 0) ? 1u : 0u);
                    a_desc += kSaQBlockBytes / 16;
                    b_desc += kSaKBlockBytes / 16;
                }
                umma_commit_elect(bar_slot_empty + 8 * (2 * stage_s + 1));    // blocks 4..8 are not needed again
                return true;
            };
            auto issue_s_v = [&](int i) -> bool {            // blocks 0..3 against Q in tensor memory
                if (!wait_slot(2 * stage_s)) return false;
                const uint32_t s_tmem = tmem_base + kColS + (i & 1) * 64;
                const uint64_t k_desc0 = umma_smem_desc_sw128(smem_u32(stage_smem + stage_s * kSaStageBytes));
                uint64_t b_desc = k_desc0;
                uint32_t a_tmem = tmem_base + kColQ;
#pragma unroll 1
                for (int b = 0; b < kSaQT; ++b) {
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        umma_f16_ts_elect_acc(s_tmem, a_tmem + ks * 8, b_desc + (ks * 32) / 16, kIdescS, 1u);
                    a_tmem += 32;
                    b_desc += kSaKBlockBytes / 16;
                }
                umma_commit_elect(bar_s_full + 8 * (i & 1));
                stage_s ^= 1;
                return true;
            };
            ok = issue_s_e(0) && issue_s_v(0);
            for (int i = 0; i < nt && ok; ++i) {
                if (i + 1 < nt) {
                    ok = issue_s_e(i + 1);
                    if (!ok) break;
                }
                ok = wait_bar(bar_p_ready + 8 * (i & 1), ph_p_ready[i & 1]);
                if (!ok) break;
                ph_p_ready[i & 1] ^= 1u;
                tcgen05_fence_after_sync();
                issue_pv(smem_u32(stage_smem + stage_pv * kSaStageBytes), kColS + (i & 1) * 64, i == 0);
                umma_commit_elect(bar_slot_empty + 8 * (2 * stage_pv));
                umma_commit_elect(bar_pv_done);
                if (i == nt - 1) umma_commit_elect(bar_o_full);
                stage_pv ^= 1;
                if (i + 1 < nt) {
                    ok = issue_s_v(i + 1);
                    if (!ok) break;
                }
            }
            if (!ok) break;
            // ---- pass 2: the second half of the output from the saved P; the four slots are a ring of value tiles
            // (accumulates in columns 256..511: no wait for the read-out of the first half)
            for (int i = 0; i < nt; ++i) {
                const int slot = i & 3;
                ok = wait_slot(slot) && wait_bar(bar_p_full + 8 * slot, ph_p_full[slot]);
                if (!ok) break;
                ph_p_full[slot] ^= 1u;
                if (tile_rescales(i)) {                          // the softmax warps rescale O first (rare after the first tiles)
                    ok = wait_bar(bar_p_ready + 8 * slot, ph_p_ready[slot]);
                    if (!ok) break;
                    ph_p_ready[slot] ^= 1u;
                }
                tcgen05_fence_after_sync();
                // P from the ring: chunks of a row are 2048 bytes apart, 8-row groups 128 bytes; 16 gathered rows per MMA
                const uint64_t p_desc0 = umma_smem_desc_noswizzle(smem_u32(q_smem) + slot * kSaPTileBytes, 128 * 16, 128);
                const uint64_t v_desc0 = umma_smem_desc_sw128_mn(smem_u32(slot_smem(slot)), kSaKBlockBytes);
#pragma unroll
                for (int ks = 0; ks < kSaBK / 16; ++ks)
                    umma_f16_elect_acc(tmem_base + kColO2, p_desc0 + (ks * 2 * 128 * 16) / 16, v_desc0 + (ks * 16 * 128) / 16, kIdescPV,
                                       (i == 0 && ks == 0) ? 0u : 1u);
                umma_commit_elect(bar_slot_empty + 8 * slot);
                umma_commit_elect(bar_p_free + 8 * slot);
                umma_commit_elect(bar_pv_done);
                if (i == nt - 1) umma_commit_elect(bar_o2_full);
                else if (tile_rescales(i + 1)) umma_commit_elect(bar_resc_go);   // tells the softmax warps when O may be rescaled
            }
            if (ok) umma_commit_elect(bar_q_empty);
        }
        if (!ok && lane == 0) sa_give_up(abort_flag, p.status, DEV_TIMEOUT_MMA);
    } else if (warp == 4) {
        if (lane == 0) {
            // ------------------------------------------------------------ Q loader
            tma_prefetch_desc(&q_map);
            uint32_t ph_q_empty = 0, ph_go = 0;
            uint32_t ph_p_free[kSaPRing] = {0u, 0u, 0u, 0u};
            bool ok = true;
            for (int64_t item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
                int64_t t;
                int i0;
                const int nt = item_of(item, t, i0);
                if (nt == 0) continue;
                ok = mbar_wait(bar_q_empty, ph_q_empty ^ 1u, abort_flag, kWaitCycleBudget, 500);   // every MMA of the previous query is done
                if (!ok) break;
                ph_q_empty ^= 1u;
                mbar_arrive_expect_tx(bar_q_full, static_cast<uint32_t>(kSaNB * p.H * 128));
                const int row0 = static_cast<int>(t * p.H);
                for (int b = 0; b < kSaNB; ++b) {
                    uint8_t* dst = b < kSaQT ? stage_smem + b * kSaQBlockBytes : q_smem + (b - kSaQT) * kSaQBlockBytes;
                    tma_load_2d_hint(smem_u32(dst), &q_map, bar_q_full, b * 64, row0, pol_stream);
                }
                // ---- pass 2: the saved P tiles come back, kSaPRing tiles ahead
                ok = mbar_wait(bar_p2_go, ph_go, abort_flag, kWaitCycleBudget, 500);
                if (!ok) break;
                ph_go ^= 1u;
                for (int i = 0; i < nt; ++i) {
                    const int b = i & (kSaPRing - 1);
                    ok = mbar_wait(bar_p_free + 8 * b, ph_p_free[b] ^ 1u, abort_flag, kWaitCycleBudget, 100);   // the PV product that read this buffer is done
                    if (!ok) break;
                    ph_p_free[b] ^= 1u;
                    // the tile that was in this buffer has been multiplied: its saved copy is dead, and L2 need not write it
                    // back (the last kSaPRing tiles of a query are left alone: the next query's pass 1 overwrites them)
                    if (i >= kSaPRing) {
                        const uint8_t* dead = scratch + static_cast<size_t>(i - kSaPRing) * kSaScratchTileBytes;
#pragma unroll 4
                        for (uint32_t o = 0; o < kSaPTileBytes; o += 128) l2_discard_128(dead + o);
                    }
                    mbar_arrive_expect_tx(bar_p_full + 8 * b, kSaPTileBytes);
                    bulk_load_1d_hint(smem_u32(q_smem) + b * kSaPTileBytes, scratch + static_cast<size_t>(i) * kSaScratchTileBytes,
                                      kSaPTileBytes, bar_p_full + 8 * b, pol_keep);
                }
            }
            if (!ok) sa_give_up(abort_flag, p.status, DEV_TIMEOUT_PRODUCER);
        }
    } else if (is_gather) {
        // ---------------------------------------------------------------- row gather
        // Two warps per slot (32 rows each): a pair only ever fills its own slot, so the four slots are four
        // independent acquire -> copy -> publish streams and a tile's landing time overlaps other tiles' copies.
        const int gw = gather_index;
        const int slot = gw >> 1;                     // 2 * stage + group
        const int row0 = (gw & 1) * 32;               // this warp's rows of every tile it handles
        uint32_t ph_q_ready = 0, ph_empty = 0;
        uint32_t tile_seq = 0;                        // pass-1 tiles before the current query: tile i sits in stage (tile_seq + i) & 1
        bool ok = true;
        uint8_t* const slot_base = slot_smem(slot);
        for (int64_t item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
            int64_t t;
            int i0;
            const int nt = item_of(item, t, i0);
            if (nt == 0) continue;
            ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar_q_ready, ph_q_ready, abort_flag, kWaitCycleBudget, 200));   // the staging area is free again
            if (!ok) break;
            ph_q_ready ^= 1u;
            const int64_t base = p.kv_base ? __ldg(p.kv_base + t) : 0;
            const int32_t* row_idx = p.topk + t * p.k_top;
            const int stand_in = __ldg(p.n_eff + 2 * t + 1);     // a selected row: skipped entries load it and get weight 0
            // lane l looks up row row0 + l of tile i; returns the mask of usable entries
            auto lookup = [&](int i, int& src_row) -> uint32_t {
                const int j = (i0 + i) * kSaBK + row0 + lane;
                src_row = -1;
                if (j < p.k_top) {
                    const int64_t idx = __ldg(row_idx + j);
                    if (idx >= 0 && base + idx >= 0 && base + idx < p.n_kv) src_row = static_cast<int>(base + idx);
                }
                const uint32_t valid = __ballot_sync(0xFFFFFFFFu, src_row >= 0);
                if (src_row < 0) src_row = stand_in;
                return valid;
            };
            // Copies column blocks [cb0, cb0 + n_blocks) of this warp's 32 rows into the slot's blocks 0..n_blocks-1 with
            // 16-byte cp.async into the swizzled layout: a warp instruction moves 512 contiguous bytes of one row. Eight
            // rows' addresses are formed before their copies issue. (TMA gather4 was measured too: one instruction per
            // four rows and block, about 22 cycles each at the TMA unit, 2.4x slower than this for the same bytes.)
            auto gather = [&](int src_row, int cb0, int n_blocks) {
                const uint32_t dst0 = smem_u32(slot_base) + (lane >> 3) * kSaKBlockBytes + row0 * 128 + ((lane & 7) << 4);
                const uint32_t dst1 = dst0 + 4 * kSaKBlockBytes;        // chunk lane + 32 lies four blocks further
                const bool second = lane + 32 < n_blocks * 8;
#pragma unroll 1
                for (int bt = 0; bt < 4; ++bt) {
                    const uint8_t* src[8];
#pragma unroll
                    for (int rr = 0; rr < 8; ++rr)
                        src[rr] = p.kv + static_cast<int64_t>(__shfl_sync(0xFFFFFFFFu, src_row, bt * 8 + rr)) * (kSaNB * 128) +
                                  (cb0 * 8 + lane) * 16;
                    // row r = row0 + 8 bt + rr: r & 7 == rr, so the swizzle is an XOR of rr into the chunk index
#pragma unroll
                    for (int rr = 0; rr < 8; ++rr) {
                        const uint32_t off = (bt * 8 + rr) * 128;
                        cp_async_16_hint((dst0 ^ (rr << 4)) + off, src[rr], pol_keep);
                        if (second) cp_async_16_hint((dst1 ^ (rr << 4)) + off, src[rr] + 512, pol_keep);
                    }
                }
                cp_async_wait_all();
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_slot_full + 8 * slot);
            };
            auto acquire = [&]() -> bool {
                const bool got = __all_sync(0xFFFFFFFFu, mbar_wait(bar_slot_empty + 8 * slot, ph_empty ^ 1u, abort_flag, kWaitCycleBudget, 100));
                ph_empty ^= 1u;
                return got;
            };
            // ---- pass 1: the tiles that sit in this slot's stage; group 1 = columns 256..575, group 0 = columns 0..255
            {
                int src_row = 0, src_next = 0;
                uint32_t valid_next = 0;
                const int first = ((slot >> 1) ^ static_cast<int>(tile_seq & 1u)) & 1;
                uint32_t valid = first < nt ? lookup(first, src_row) : 0u;
                for (int i = first; i < nt; i += 2) {
                    if (i + 2 < nt) valid_next = lookup(i + 2, src_next);
                    ok = acquire();
                    if (!ok) break;
                    if (slot & 1) {
                        gather(src_row, kSaNVH, kSaNB - kSaNVH);
                    } else {
                        if (lane == 0) tile_mask[(slot >> 1) * 2 + (gw & 1)] = valid;
                        gather(src_row, 0, kSaNVH);
                    }
                    src_row = src_next;
                    valid = valid_next;
                }
                tile_seq += static_cast<uint32_t>(nt);
            }
            // ---- pass 2: columns 256..511 only; tile i sits in slot i & 3
            if (ok) {
                int src_row = 0, src_next = 0;
                if (slot < nt) lookup(slot, src_row);
                for (int i = slot; i < nt; i += 4) {
                    if (i + 4 < nt) lookup(i + 4, src_next);
                    ok = acquire();
                    if (!ok) break;
                    gather(src_row, kSaNVH, kSaNVH);
                    src_row = src_next;
                }
            }
        }
        if (!ok && lane == 0) sa_give_up(abort_flag, p.status, DEV_TIMEOUT_GATHER);
    } else if (warp >= 12) {
        // ---------------------------------------------------------------- softmax and output
        const int quarter = warp & 3;                  // TMEM lane quarter this warp may access
        const int row = quarter * 32 + lane;           // head
        const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        uint32_t ph_q_full = 0, ph_o_full = 0;
        uint32_t ph_s_full[2] = {0u, 0u}, ph_resc_go = 0;
        uint32_t pv_tiles = 0;                         // PV tiles before the current one, over the whole kernel
        int stage = 0;
        bool ok = true;
        // Saved P of a tile: [8 chunks of 16 bytes][128 rows]: a warp's store or copy of one chunk touches 512 contiguous bytes
        uint8_t* my_p = scratch + row * 16;                           // + tile * kSaScratchTileBytes + chunk * 2048
        uint8_t* my_alpha = scratch + 128 * kSaBK * 2 + row * 4;      // + tile * kSaScratchTileBytes: this row's factor
        // multiplies this thread's row of O by alpha (the caller has made sure that every earlier PV product is complete)
        auto scale_o = [&](float alpha, uint32_t col0) {
            tcgen05_fence_after_sync();
#pragma unroll 1
            for (int c = 0; c < 8; ++c) {
                uint32_t o[32];
                tmem_ld_32x32b_x32(lane_base + col0 + c * 32, o);
                tmem_ld_wait(o);
#pragma unroll
                for (int j = 0; j < 32; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * alpha);
                tmem_st_32x32b_x32(lane_base + col0 + c * 32, o);
            }
        };
        // Normalises this thread's row of O and writes 256 output columns: fp32 to this split's partial result when
        // several CTAs share the query (part_row != nullptr), else bf16 to the output. A thread holds 32 columns of one
        // row at a time, and storing them directly makes every warp store touch 32 lines; so the warp transposes them
        // through 2 KB of shared memory (the last block of a stage, which neither the value tiles of pass 2 nor the Q
        // staging use) and stores 8 rows x 64 contiguous bytes per instruction.
        uint8_t* const stg = stage_smem + 8 * kSaKBlockBytes + quarter * 2048;     // [32 rows][64 B], 16-byte chunks XORed by (row >> 1) & 3
        auto write_out = [&](__nv_bfloat16* dst_query, float* part_row, float inv, uint32_t col0, bool last) -> bool {   // dst_query: row 0 of the query, first column of the half
            // each of the two barriers completes once per query: the phase flips after the second half
            if (!__all_sync(0xFFFFFFFFu, mbar_wait(last ? bar_o2_full : bar_o_full, ph_o_full, abort_flag))) return false;
            if (last) ph_o_full ^= 1u;
            tcgen05_fence_after_sync();
#pragma unroll 1
            for (int c = 0; c < 8; ++c) {
                uint32_t o[32];
                tmem_ld_32x32b_x32(lane_base + col0 + c * 32, o);
                tmem_ld_wait(o);
                if (part_row != nullptr) {
                    if (row < p.H) {
                        float4* dst = reinterpret_cast<float4*>(part_row + c * 32);
#pragma unroll
                        for (int v = 0; v < 8; ++v)
                            dst[v] = make_float4(__uint_as_float(o[4 * v + 0]) * inv, __uint_as_float(o[4 * v + 1]) * inv,
                                                 __uint_as_float(o[4 * v + 2]) * inv, __uint_as_float(o[4 * v + 3]) * inv);
                    }
                } else {
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        uint4 w;
                        w.x = pack_bf16x2(__uint_as_float(o[8 * v + 0]) * inv, __uint_as_float(o[8 * v + 1]) * inv);
                        w.y = pack_bf16x2(__uint_as_float(o[8 * v + 2]) * inv, __uint_as_float(o[8 * v + 3]) * inv);
                        w.z = pack_bf16x2(__uint_as_float(o[8 * v + 4]) * inv, __uint_as_float(o[8 * v + 5]) * inv);
                        w.w = pack_bf16x2(__uint_as_float(o[8 * v + 6]) * inv, __uint_as_float(o[8 * v + 7]) * inv);
                        *reinterpret_cast<uint4*>(stg + lane * 64 + ((v ^ ((lane >> 1) & 3)) << 4)) = w;
                    }
                    __syncwarp();
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int rr = (lane >> 2) + 8 * k, ch = lane & 3;     // 8 rows per instruction, 4 lanes per row
                        const uint4 w = *reinterpret_cast<const uint4*>(stg + rr * 64 + ((ch ^ ((rr >> 1) & 3)) << 4));
                        if (quarter * 32 + rr < p.H)
                            st_global_v4_hint(dst_query + static_cast<int64_t>(quarter * 32 + rr) * 512 + c * 32 + ch * 8, w, pol_stream);
                    }
                    __syncwarp();
                }
            }
            tcgen05_fence_before_sync();
            __syncwarp();
            if (last && lane == 0) mbar_arrive(bar_o_free);    // both halves of O are read out: the next query may overwrite them
            return true;
        };
        for (int64_t item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
            int64_t t;
            int i0;
            const int nt = item_of(item, t, i0);
            __nv_bfloat16* out_row = p.out + (t * p.H + row) * 512;
            float* part_row = p.splits > 1 ? p.part_out + (item * p.H + row) * 512 : nullptr;
            if (nt == 0) {                              // nothing (usable) in this item's range: zeros, weight 0 in the merge
                if (row < p.H) {
                    if (part_row) {
                        for (int c = 0; c < 512 / 4; ++c) reinterpret_cast<float4*>(part_row)[c] = make_float4(0.f, 0.f, 0.f, 0.f);
                        p.part_lse[item * p.H + row] = -INFINITY;
                    } else {
                        for (int c = 0; c < 512 / 8; ++c) reinterpret_cast<uint4*>(out_row)[c] = make_uint4(0u, 0u, 0u, 0u);
                        if (p.lse) p.lse[t * p.H + row] = -INFINITY;
                    }
                }
                continue;
            }
            // ---- Q blocks 0..3: staging (swizzled rows) -> tensor memory, two bf16 per column
            ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar_q_full, ph_q_full, abort_flag));
            if (!ok) break;
            ph_q_full ^= 1u;
            // every reader of the previous query's flags is done (its last PV product was issued before this thread
            // wrote its output); the arrival on q_ready below orders the reset before this query's tiles
            if (quarter == 0 && lane < kSaFlagTiles / 32) resc_mask[lane] = 0u;
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

            // ---- pass 1
            float m_ref = -INFINITY, l = 0.f;
            for (int i = 0; i < nt; ++i) {
                const int sbuf = i & 1;
                ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar_s_full + 8 * sbuf, ph_s_full[sbuf], abort_flag));
                if (!ok) break;
                ph_s_full[sbuf] ^= 1u;
                tcgen05_fence_after_sync();
                const uint32_t s_tmem = lane_base + kColS + sbuf * 64;
                uint32_t mlo, mhi;                                  // explicit shared-memory load: a generic one queues behind the global traffic
                asm volatile("ld.volatile.shared.v2.u32 {%0, %1}, [%2];" : "=r"(mlo), "=r"(mhi) : "r"(smem_u32(const_cast<uint32_t*>(tile_mask) + stage * 2)) : "memory");
                // Both sweeps over the 64 scores are rolled loops over 16-column chunks, read from tensor memory
                // twice: the instruction footprint of the hot loop stays small.
                // (the load of the next chunk is in flight while a chunk is processed: a tensor-memory load takes ~200 cycles)
                float mt = -INFINITY;
                auto max16 = [&](const uint32_t (&r)[16], uint32_t m16) {
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        mt = fmaxf(mt, (m16 >> j) & 1u ? __uint_as_float(r[j]) * p.scale_log2 : -INFINITY);
                };
                {
                    uint32_t ra[16], rb[16];
                    tmem_ld_32x32b_x16(s_tmem, ra);
#pragma unroll 1
                    for (int h = 0; h < 2; ++h) {
                        const uint32_t m32 = h ? mhi : mlo;
                        tmem_ld_wait(ra);
                        tmem_ld_32x32b_x16(s_tmem + 32 * h + 16, rb);
                        max16(ra, m32);
                        tmem_ld_wait(rb);
                        if (h == 0) tmem_ld_32x32b_x16(s_tmem + 32, ra);
                        max16(rb, m32 >> 16);
                    }
                }
                // rows beyond the query's heads hold whatever the staging area held before (only H rows are loaded): they
                // must never ask for a rescale of O, which would cost every tile of the query an extra pass
                if (row >= p.H) mt = -INFINITY;
                // lazy reference maximum: move it only when the row maximum outgrew it by 2^8
                const bool move = mt > m_ref + kRescaleThreshold;      // also true for the first usable score (m_ref = -inf)
                float alpha = 1.f;
                if (move) {
                    alpha = m_ref == -INFINITY ? 0.f : fast_exp2(m_ref - mt);
                    m_ref = mt;
                    l *= alpha;
                }
                if (i > 0 && __any_sync(0xFFFFFFFFu, move)) {
                    if (lane == 0 && i < kSaFlagTiles) atomicOr(const_cast<uint32_t*>(resc_mask) + (i >> 5), 1u << (i & 31));
                    // PV(i-1) was issued before the second part of S(i), whose completion this thread has seen; the wait
                    // below (one phase per PV tile: the barrier is in phase pv_tiles-1 or pv_tiles) then passes at once
                    ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar_pv_done, (pv_tiles - 1u) & 1u, abort_flag));
                    if (!ok) break;
                    scale_o(alpha, kColO);
                }
                const float m_sub = m_ref == -INFINITY ? 0.f : m_ref;   // no usable score yet: every P is exp2(-inf) = 0
                // P(i) goes over the first half of S(i) chunk by chunk (columns 8c..8c+7 hold scores this thread has
                // already read) and, with the factor, to the scratch area for pass 2
                uint4* dst = reinterpret_cast<uint4*>(my_p + static_cast<size_t>(i) * kSaScratchTileBytes);
                float sum = 0.f;
                auto exp16 = [&](const uint32_t (&r)[16], uint32_t m16, int c) {
                    uint32_t pr[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const float x0 = (m16 >> (2 * j)) & 1u ? __uint_as_float(r[2 * j]) * p.scale_log2 : -INFINITY;
                        const float x1 = (m16 >> (2 * j + 1)) & 1u ? __uint_as_float(r[2 * j + 1]) * p.scale_log2 : -INFINITY;
                        const float p0 = fast_exp2(x0 - m_sub), p1 = fast_exp2(x1 - m_sub);
                        sum += p0 + p1;
                        pr[j] = pack_bf16x2(p0, p1);
                    }
                    tmem_st_32x32b_x8(s_tmem + 8 * c, pr);
                    st_global_v4_hint(dst + (2 * c) * 128, make_uint4(pr[0], pr[1], pr[2], pr[3]), pol_keep);
                    st_global_v4_hint(dst + (2 * c + 1) * 128, make_uint4(pr[4], pr[5], pr[6], pr[7]), pol_keep);
                };
                {
                    uint32_t ra[16], rb[16];
                    tmem_ld_32x32b_x16(s_tmem, ra);
#pragma unroll 1
                    for (int h = 0; h < 2; ++h) {
                        const uint32_t m32 = h ? mhi : mlo;
                        tmem_ld_wait(ra);
                        tmem_ld_32x32b_x16(s_tmem + 32 * h + 16, rb);
                        exp16(ra, m32, 2 * h);
                        tmem_ld_wait(rb);
                        if (h == 0) tmem_ld_32x32b_x16(s_tmem + 32, ra);   // columns 32..47: beyond the P columns written so far
                        exp16(rb, m32 >> 16, 2 * h + 1);
                    }
                }
                l += sum;
                tmem_st_wait();
                tcgen05_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_p_ready + 8 * sbuf);
                __stcg(reinterpret_cast<float*>(my_alpha + static_cast<size_t>(i) * kSaScratchTileBytes), alpha);
                ++pv_tiles;
                stage ^= 1;
            }
            if (!ok) break;
            // P and the factors of every tile are written: order them before the bulk copies of pass 2 (async proxy),
            // which the loader issues once all four warps have arrived. Every score product has completed by now, so
            // the shared memory that held Q is free for the ring.
            __threadfence();
            fence_proxy_async_global();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_p2_go);
            const float inv = l > 0.f ? 1.f / l : 0.f;
            ok = write_out(p.out + t * p.H * 512, part_row, inv, kColO, false);
            if (!ok) break;
            if (row < p.H) {
                const float lse_val = l > 0.f ? (m_ref + log2f(l)) * 0.6931471805599453f : -INFINITY;
                if (part_row) p.part_lse[item * p.H + row] = lse_val;
                else if (p.lse) p.lse[t * p.H + row] = lse_val;
            }

            // ---- pass 2: the MMA warp reads P from the ring itself; this thread only replays the rescales of its row
            // (the factor of tile i applies to the sum over the tiles before i) at the tiles flagged in pass 1: the MMA
            // warp signals when the products before such a tile are complete and waits for the arrival below
#pragma unroll 1
            for (int i = 1; i < nt && ok; ++i) {
                if (!tile_rescales(i)) continue;
                ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar_resc_go, ph_resc_go, abort_flag));
                if (!ok) break;
                ph_resc_go ^= 1u;
                const float alpha = __ldcg(reinterpret_cast<const float*>(my_alpha + static_cast<size_t>(i) * kSaScratchTileBytes));
                if (__any_sync(0xFFFFFFFFu, alpha != 1.f)) {
                    scale_o(alpha, kColO2);
                    tmem_st_wait();
                }
                tcgen05_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_p_ready + 8 * (i & (kSaPRing - 1)));
            }
            pv_tiles += static_cast<uint32_t>(nt);
            if (!ok) break;
            ok = write_out(p.out + t * p.H * 512 + 256, part_row ? part_row + 256 : nullptr, inv, kColO2, true);
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

// Merges the splits of a query: out = sum_s w_s out_s / sum_s w_s with w_s = exp(lse_s - max_s lse_s). One CTA per
// (query, head), 128 threads x 4 columns.
__global__ void __launch_bounds__(128)
sparse_attn_merge_kernel(const float* __restrict__ part_out, const float* __restrict__ part_lse, int H, int splits,
                         __nv_bfloat16* __restrict__ out, float* __restrict__ lse) {
    constexpr int kMaxSplits = 8;              // sparse_attn_splits never returns more
    const int64_t t = blockIdx.x / H;
    const int h = static_cast<int>(blockIdx.x - t * H);
    // all loads are issued before anything depends on them: one round trip to the L2 instead of one per split
    float ls[kMaxSplits];
    float4 v[kMaxSplits];
#pragma unroll
    for (int s = 0; s < kMaxSplits; ++s) {
        ls[s] = -INFINITY;
        v[s] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (s < splits) {
            ls[s] = __ldg(part_lse + (t * splits + s) * H + h);
            v[s] = __ldg(reinterpret_cast<const float4*>(part_out + ((t * splits + s) * H + h) * 512) + threadIdx.x);
        }
    }
    float m = -INFINITY;
#pragma unroll
    for (int s = 0; s < kMaxSplits; ++s) m = fmaxf(m, ls[s]);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float denom = 0.f;
    if (m > -INFINITY) {
#pragma unroll
        for (int s = 0; s < kMaxSplits; ++s) {
            const float w = __expf(ls[s] - m);     // 0 for a split with nothing usable (its result is all zeros)
            acc.x += w * v[s].x; acc.y += w * v[s].y; acc.z += w * v[s].z; acc.w += w * v[s].w;
            denom += w;
        }
    }
    const float inv = denom > 0.f ? 1.f / denom : 0.f;
    uint2 packed;
    packed.x = pack_bf16x2(acc.x * inv, acc.y * inv);
    packed.y = pack_bf16x2(acc.z * inv, acc.w * inv);
    reinterpret_cast<uint2*>(out + (t * H + h) * 512)[threadIdx.x] = packed;
    if (lse && threadIdx.x == 0) lse[t * H + h] = denom > 0.f ? m + logf(denom) : -INFINITY;
}

}  // namespace

bool sparse_attn_supported(int H, int d_qk, int d_v) { return H >= 1 && H <= 128 && d_qk == 64 * kSaNB && d_v == 128 * kSaNVH; }

// Few queries (a decode step) would leave most SMs idle: their selected rows are split over several CTAs.
int sparse_attn_splits(int64_t n_q) {
    if (n_q <= 0 || n_q >= 64) return 1;
    const int64_t s = 128 / n_q;
    return static_cast<int>(s > 8 ? 8 : s);
}
size_t sparse_attn_scratch_bytes(int64_t n_q, int k_top) {
    const int64_t items = n_q * sparse_attn_splits(n_q);
    const int64_t ctas = items < kSparseAttnMaxGrid ? items : kSparseAttnMaxGrid;
    return static_cast<size_t>(ctas) * ((k_top + kSaBK - 1) / kSaBK) * kSaScratchTileBytes;
}
size_t sparse_attn_partial_bytes(int64_t n_q) {        // sized for 128 heads
    const int splits = sparse_attn_splits(n_q);
    return splits > 1 ? static_cast<size_t>(n_q) * splits * 128 * (512 + 1) * sizeof(float) : 0;
}

cudaError_t launch_sparse_attn(const void* kv, const int32_t* topk, const int64_t* kv_base, int64_t n_q, int64_t n_kv, int H,
                               int k_top, float scale, void* out, float* lse, int32_t* n_eff, void* scratch, void* partial,
                               const CUtensorMap& q_map, unsigned int* status, int sm_count,
                               cudaStream_t stream) {
    if (n_q <= 0) return cudaSuccess;
    sparse_attn_count_kernel<<<static_cast<unsigned>(n_q), kSaCountThreads, 0, stream>>>(topk, kv_base, n_q, n_kv, k_top, n_eff);
    if (cudaError_t e = cudaGetLastError(); e != cudaSuccess) return e;
    if (cudaError_t e = ensure_max_dynamic_smem(reinterpret_cast<const void*>(sparse_attn_kernel), kSaSmemBytes); e != cudaSuccess) return e;
    const int splits = sparse_attn_splits(n_q);
    float* part_out = static_cast<float*>(partial);
    float* part_lse = part_out ? part_out + static_cast<size_t>(n_q) * splits * 128 * 512 : nullptr;
    SaParams p{static_cast<const uint8_t*>(kv), topk, kv_base, n_eff, static_cast<uint8_t*>(scratch), n_q, n_kv, H, k_top,
               scale * 1.4426950408889634f, static_cast<__nv_bfloat16*>(out), lse, splits, part_out, part_lse, status};
    const int64_t items = n_q * splits;
    const int cap = sm_count < kSparseAttnMaxGrid ? sm_count : kSparseAttnMaxGrid;
    const int grid = static_cast<int>(items < cap ? items : cap);
    sparse_attn_kernel<<<grid, kSaThreads, kSaSmemBytes, stream>>>(q_map, p);
    if (cudaError_t e = cudaGetLastError(); e != cudaSuccess) return e;
    if (splits > 1) {
        sparse_attn_merge_kernel<<<static_cast<unsigned>(n_q * H), 128, 0, stream>>>(part_out, part_lse, H, splits,
                                                                                      static_cast<__nv_bfloat16*>(out), lse);
        return cudaGetLastError();
    }
    return cudaSuccess;
}

}  // namespace idxc
