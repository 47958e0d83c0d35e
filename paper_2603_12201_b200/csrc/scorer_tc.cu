// tcgen05 / TMEM indexer scorers for sm_100a.
//
// Score (Sec. 2.1): I[t,s] = sum_h w[t,h] * max(q[t,h,:] . k[s,:], 0), s <= t.
// The dot products are one dense contraction [keys, d] x [d, (query, head)]. It is laid
// out with KEYS ON THE MMA's M axis (TMEM lanes) and (query, head) ON N (TMEM columns):
// an epilogue thread then owns a few keys and a quarter of the (query, head) columns, so
// the gate and the w-weighted head sum are register arithmetic with w held in registers,
// finished by a butterfly of three shuffles across the four threads that share a group of four keys.
//
// Prefill kernel (persistent, one CTA per SM, warp-specialised):
//   warp 0      TMA producer: a block of 2*256/H queries (two 256-column B tiles) is loaded
//               once per work item and stays in shared memory; 128-key A tiles stream
//               through a ring of stages. Per-CTA loads only.
//   warp 1      MMA issuer: per key tile, one 128 x 256 x d UMMA chain into each of the two
//               256-column TMEM accumulators, so accumulator A is drained while B is filled.
//   warps 2-9   epilogue: tcgen05.ld (16x256b), ReLU, FMA with w held in registers, three shuffles per four
//               scores to join the four threads of a key group, causal predicate, coalesced score store.
// Causal structure: a work item only visits key tiles up to its last query's position;
// items are handed out longest first in a boustrophedon order over the CTAs.
//
// Decode kernel: work item = (sequence, run of key tiles); the sequence's H x d query tile
// is the B operand (N = H), key tiles stream from HBM through a deep TMA ring; two groups of four
// epilogue warps drain alternate TMEM accumulator slots.
#include "kernels.h"
#include "ptx_sm100.cuh"
#include "topk_common.cuh"

namespace idxc {
namespace {

constexpr int kTileKeys = 128;          // UMMA M
constexpr int kTileCols = 256;          // UMMA N (prefill)
constexpr int kChunkBytes = 128;        // one swizzle row: 64 bf16 or 128 fp8 elements
constexpr int kQRegionBytes = kTileCols * kChunkBytes;   // 32 KB
constexpr int kKRegionBytes = kTileKeys * kChunkBytes;   // 16 KB
// 8 epilogue warps measured faster than 16 on B200 (6.5 ms vs 6.9 ms on config 2): the kernel runs at the
// board's power limit, and the extra warps cost more than the latency they hide.
#ifndef IDXC_EPI_WARPS
#define IDXC_EPI_WARPS 8
#endif
constexpr int kEpilogueWarp0 = 2;       // warps 0, 1: TMA producer, MMA issuer; no idle warps, so that the
                                        // registers left on the SM can host a top-k CTA next to this kernel
constexpr int kNumEpilogueWarps = IDXC_EPI_WARPS;       // 8 or 16: 2 or 4 per TMEM lane quarter
constexpr int kPrefillThreads = (kEpilogueWarp0 + kNumEpilogueWarps) * 32;
constexpr int kColsPerEpiWarp = kTileCols / (kNumEpilogueWarps / 4);   // 128 or 64 accumulator columns per warp
constexpr int kGroupsPerEpiWarp = kColsPerEpiWarp / 8;               // 8-column groups per warp
constexpr int kChunksPerEpiWarp = kColsPerEpiWarp / 32;              // 32-column TMEM loads per 16 lanes

// STREAM: streaming top-k (kernels.h, StreamTopk). The sample of a work item's rows lives in shared memory
// (kStreamSampleBytes over all rows of the item); with 256-byte operand rows the key ring gives up a stage for it.
constexpr int kStreamSampleBytes = 32 * 1024;
template <int NKH, int H, bool STREAM>
struct PrefillCfg {
    static constexpr int QB = 2 * (kTileCols / H);
    static constexpr int kStages = NKH == 2 ? (STREAM ? 2 : 3) : 4;
    static constexpr int kQBytes = 2 * NKH * kQRegionBytes;
    static constexpr int kKBytes = kStages * NKH * kKRegionBytes;
    static constexpr int kSampleBytes = STREAM ? kStreamSampleBytes : 0;
    static constexpr int kSampleMax = kStreamSampleBytes / 4 / QB;          // sample scores per row: 1024, 512, 256
    static constexpr int kSampleTiles = kSampleMax / kTileKeys;             // key tiles visited before the threshold exists
    static constexpr int kBarBytes = 256 + (STREAM ? 16 * QB + 1024 : 0);   // + per-row counter, threshold; 32 bins per epilogue warp
    static constexpr int kSmemBytes = kQBytes + kKBytes + kSampleBytes + kBarBytes + 1024;   // + alignment slack
    static constexpr bool kFits = kSmemBytes <= 227 * 1024 && kSampleTiles >= 2;
};

struct PrefillParams {
    const float* w;
    const float* q_scale;
    const float* k_scale;
    float* scores;
    int64_t ld;
    int64_t q_begin;
    int64_t n_rows;
    int64_t k_rows;
    unsigned int* status;
    StreamTopk st;
    const uint8_t* item_mask;
    int sub_per_block;      // work items per block of QB query rows: 1, or (few blocks, long rows) the block's key tiles in
    int key_split;          // ... sub_per_block runs of key_split tiles each, so that every SM gets work
};

// Order in which a work item of nkt key tiles is visited when the top-k streams: `ns` sample tiles 0, stride,
// 2 stride, ... first, then the others in ascending order. Without a sample (ns == nkt) the order is plain.
struct TileOrder {
    int nkt, stride, ns;
    __device__ TileOrder(int nkt_, int max_sample_tiles) : nkt(nkt_) {
        stride = (nkt + max_sample_tiles - 1) / max_sample_tiles;
        if (stride < 2) { stride = 1; ns = nkt; }
        else ns = (nkt + stride - 1) / stride;
    }
    __device__ int tile(int j) const {
        if (j < ns) return j * stride;
        const int r = j - ns;                       // r-th tile that is not a multiple of stride
        return r + r / (stride - 1) + 1;
    }
};

__device__ __forceinline__ void give_up(volatile uint32_t* abort_flag, unsigned int* status, unsigned int code) {
    *abort_flag = 1u;
    atomicCAS(status, 0u, code);
}

// NKH: 128-byte chunks per operand row (d * element size / 128). H: indexer heads.
template <int NKH, int H, bool FP8, bool STREAM, bool SPLIT>
__global__ void __launch_bounds__(kPrefillThreads, 1)
score_prefill_tc_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                        const PrefillParams p) {
    using Cfg = PrefillCfg<NKH, H, STREAM>;
    constexpr int kStages = Cfg::kStages;
    constexpr int QPA = kTileCols / H;       // queries per accumulator
    constexpr int QB = 2 * QPA;              // queries per work item
    constexpr int kElemsPerChunk = FP8 ? 128 : 64;
    constexpr uint32_t kIdesc = FP8 ? umma_idesc(0, 0, kTileKeys, kTileCols) : umma_idesc(1, 1, kTileKeys, kTileCols);

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t* q_smem = smem;                                   // [2][NKH][256 x 128 B]
    uint8_t* k_smem = q_smem + Cfg::kQBytes;                  // [kStages][NKH][128 x 128 B]
    float* sample = reinterpret_cast<float*>(k_smem + Cfg::kKBytes);          // STREAM: [QB][kSampleMax] scores of the sample tiles
    uint64_t* bars = reinterpret_cast<uint64_t*>(k_smem + Cfg::kKBytes + Cfg::kSampleBytes);
    // barrier map
    const uint32_t bar_q_full = smem_u32(bars + 0);           // [2]
    const uint32_t bar_q_empty = smem_u32(bars + 2);          // [2]
    const uint32_t bar_acc_full = smem_u32(bars + 4);         // [2]
    const uint32_t bar_acc_empty = smem_u32(bars + 6);        // [2]
    const uint32_t bar_k_full = smem_u32(bars + 8);           // [kStages]
    const uint32_t bar_k_empty = smem_u32(bars + 8 + kStages);
    const uint32_t bar_group = smem_u32(bars + 8 + 2 * kStages);   // STREAM: [2] the four warps that share a set of query rows
    uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(bars + 10 + 2 * kStages);
    volatile uint32_t* abort_flag = tmem_base_slot + 1;
    float* row_tau = reinterpret_cast<float*>(tmem_base_slot + 4);   // STREAM: [QB] the row's threshold
    uint32_t* warp_hist = reinterpret_cast<uint32_t*>(row_tau + QB);   // STREAM: [epilogue warps][32]
    static_assert((10 + 2 * kStages) * 8 + 16 + (STREAM ? 4 * QB + 128 * kNumEpilogueWarps : 0) <= Cfg::kBarBytes, "barrier area");

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar_q_full + 8 * i, 1);
            mbar_init(bar_q_empty + 8 * i, 1);
            mbar_init(bar_acc_full + 8 * i, 1);
            mbar_init(bar_acc_empty + 8 * i, kNumEpilogueWarps);
        }
        for (int i = 0; i < kStages; ++i) {
            mbar_init(bar_k_full + 8 * i, 1);
            mbar_init(bar_k_empty + 8 * i, 1);
        }
        mbar_init(bar_group, kNumEpilogueWarps / 2);
        mbar_init(bar_group + 8, kNumEpilogueWarps / 2);
        *abort_flag = 0u;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_base_slot), 512);
        tmem_relinquish_alloc_permit();
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    tcgen05_fence_after_sync();
    const uint32_t tmem_base = *tmem_base_slot;

    const int n_sub = SPLIT ? p.sub_per_block : 1;       // (a compile-time 1 keeps the unsplit kernel's code as it was)
    const int64_t n_items = (p.n_rows + QB - 1) / QB * n_sub;
    const int G = gridDim.x;
    const int cta = blockIdx.x;
    // key tiles a block of QB query rows visits: positions 0 .. q_begin + (its last row)
    auto key_tiles_of_block = [&](int64_t block) -> int {
        int64_t last = block * QB + QB;
        if (last > p.n_rows) last = p.n_rows;
        return static_cast<int>((p.q_begin + last + kTileKeys - 1) / kTileKeys);
    };
    // A work item is a block of QB query rows with all its key tiles, or (n_sub > 1) run number item % n_sub of key_split
    // of its key tiles. Work item of this CTA in round `rho` (longest first, boustrophedon), -1: none left,
    // -2: the item is masked out or its run lies beyond the block's last tile, and every role passes over it
    auto item_of_round = [&](int64_t rho) -> int64_t {
        const int64_t seq = rho * G + ((rho & 1) ? (G - 1 - cta) : cta);
        if (seq >= n_items) return -1;
        const int64_t item = n_items - 1 - seq;
        const int64_t block = n_sub == 1 ? item : item / n_sub;
        if (p.item_mask != nullptr && p.item_mask[block] == 0) return -2;
        if (n_sub > 1 && static_cast<int>(item % n_sub) * p.key_split >= key_tiles_of_block(block)) return -2;
        return item;
    };
    // first key tile and number of key tiles of a work item
    auto first_tile_of_item = [&](int64_t item) -> int { return n_sub == 1 ? 0 : static_cast<int>(item % n_sub) * p.key_split; };
    auto key_tiles_of_item = [&](int64_t item) -> int {
        const int all = key_tiles_of_block(n_sub == 1 ? item : item / n_sub);
        if (n_sub == 1) return all;
        const int left = all - first_tile_of_item(item);
        return left < p.key_split ? left : p.key_split;
    };

    if (warp == 0) {
        if (lane == 0) {
            // ------------------------------------------------------------ TMA producer
            tma_prefetch_desc(&q_map);
            tma_prefetch_desc(&k_map);
            int stage = 0;
            uint32_t k_phase = 0, q_phase = 0;
            bool ok = true;
            for (int64_t rho = 0; ok; ++rho) {
                const int64_t item_id = item_of_round(rho);
                if (item_id == -2) continue;
                if (item_id < 0) break;
                const int nkt = key_tiles_of_item(item_id);
                const int kt0 = first_tile_of_item(item_id);
                const int64_t item = n_sub == 1 ? item_id : item_id / n_sub;        // the block of query rows
                const TileOrder ord(nkt, STREAM ? Cfg::kSampleTiles : nkt);
                auto load_k = [&](int j) -> bool {
                    const int kt = STREAM ? ord.tile(j) : kt0 + j;
                    if (!mbar_wait(bar_k_empty + 8 * stage, k_phase ^ 1u, abort_flag)) return false;
                    mbar_arrive_expect_tx(bar_k_full + 8 * stage, NKH * kKRegionBytes);
                    for (int kh = 0; kh < NKH; ++kh)
                        tma_load_2d(smem_u32(k_smem + (stage * NKH + kh) * kKRegionBytes), &k_map, bar_k_full + 8 * stage,
                                    kh * kElemsPerChunk, kt * kTileKeys);
                    if (++stage == kStages) { stage = 0; k_phase ^= 1u; }
                    return true;
                };
                // The first key tiles of this item go out before the wait for the query buffers: their ring stages come
                // free while the previous item's last tiles are still being multiplied, the query buffers only after them.
                const int pre = nkt < kStages ? nkt : kStages;
                for (int kt = 0; kt < pre && ok; ++kt) ok = load_k(kt);
                for (int half = 0; half < 2 && ok; ++half) {
                    ok = mbar_wait(bar_q_empty + 8 * half, q_phase ^ 1u, abort_flag);
                    if (!ok) break;
                    mbar_arrive_expect_tx(bar_q_full + 8 * half, NKH * kQRegionBytes);
                    const int row0 = static_cast<int>((item * QB + half * QPA) * H);
                    for (int kh = 0; kh < NKH; ++kh)
                        tma_load_2d(smem_u32(q_smem + (half * NKH + kh) * kQRegionBytes), &q_map, bar_q_full + 8 * half,
                                    kh * kElemsPerChunk, row0);
                }
                for (int kt = pre; kt < nkt && ok; ++kt) ok = load_k(kt);
                q_phase ^= 1u;
            }
            if (!ok) give_up(abort_flag, p.status, DEV_TIMEOUT_PRODUCER);
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        // The whole warp runs this role with uniform control flow and one elected lane issues; descriptors are a base
        // plus 16-byte units.
        int stage = 0;
        uint32_t k_phase = 0, q_phase = 0;
        uint32_t acc_phase[2] = {0u, 0u};
        bool ok = true;
        const uint64_t a_desc0 = umma_smem_desc_sw128(smem_u32(k_smem));
        const uint64_t b_desc0 = umma_smem_desc_sw128(smem_u32(q_smem));
        auto wait_bar = [&](uint32_t bar, uint32_t parity) -> bool {
            return __all_sync(0xFFFFFFFFu, mbar_wait(bar, parity, abort_flag));
        };
        for (int64_t rho = 0; ok; ++rho) {
            const int64_t item_id = item_of_round(rho);
            if (item_id == -2) continue;
            if (item_id < 0) break;
            const int nkt = key_tiles_of_item(item_id);
            for (int kt = 0; kt < nkt && ok; ++kt) {
                ok = wait_bar(bar_k_full + 8 * stage, k_phase);
                if (!ok) break;
                const uint64_t a_stage = a_desc0 + static_cast<uint64_t>(stage * NKH * kKRegionBytes / 16);
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    if (kt == 0) {
                        ok = wait_bar(bar_q_full + 8 * half, q_phase);
                        if (!ok) break;
                    }
                    ok = wait_bar(bar_acc_empty + 8 * half, acc_phase[half] ^ 1u);
                    if (!ok) break;
                    acc_phase[half] ^= 1u;
                    tcgen05_fence_after_sync();
                    const uint32_t d_tmem = tmem_base + half * kTileCols;
                    const uint64_t b_half = b_desc0 + static_cast<uint64_t>(half * NKH * kQRegionBytes / 16);
#pragma unroll
                    for (int kh = 0; kh < NKH; ++kh) {
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) {   // 32 bytes of K per MMA: 16 bf16 or 32 fp8
                            const uint64_t a = a_stage + (kh * kKRegionBytes + ks * 32) / 16, b = b_half + (kh * kQRegionBytes + ks * 32) / 16;
                            if constexpr (FP8) {
                                if ((kh | ks) != 0) umma_f8_elect<true>(d_tmem, a, b, kIdesc);
                                else umma_f8_elect<false>(d_tmem, a, b, kIdesc);
                            } else {
                                if ((kh | ks) != 0) umma_f16_elect<true>(d_tmem, a, b, kIdesc);
                                else umma_f16_elect<false>(d_tmem, a, b, kIdesc);
                            }
                        }
                    }
                    umma_commit_elect(bar_acc_full + 8 * half);
                    if (kt == nkt - 1) umma_commit_elect(bar_q_empty + 8 * half);
                }
                if (!ok) break;
                umma_commit_elect(bar_k_empty + 8 * stage);
                if (++stage == kStages) { stage = 0; k_phase ^= 1u; }
            }
            q_phase ^= 1u;
        }
        if (!ok && lane == 0) give_up(abort_flag, p.status, DEV_TIMEOUT_MMA);
    } else if (warp >= kEpilogueWarp0) {
        // ---------------------------------------------------------------- epilogue
        // TMEM is read with the 16x256b shape: a thread owns 4 keys (TMEM lanes g, g+8, g+16, g+24 of
        // its warp's lane quarter, g = lane/4) and the columns 8i + 2j + {0,1} (j = lane%4) of every
        // 8-column group. Its share of w (64 values per work item) therefore lives in registers and
        // the gate/FMA loop issues no shared-memory loads; the four threads of a group add their
        // partial head sums with three shuffles per four scores at the end.
        constexpr int QPW = kColsPerEpiWarp / H;     // queries per warp per accumulator
        static_assert(QPW >= 1, "an epilogue warp must cover at least one query");
        const int ew = warp - kEpilogueWarp0;
        const int quarter = warp & 3;                // TMEM lane quarter this warp may read
        const int colhalf = ew >> 2;                 // which slice of kColsPerEpiWarp columns of the accumulator
        const int j = lane & 3, g = lane >> 2;
        const int key_written = quarter * 32 + g + 8 * j;    // the key (of the thread's four) this thread stores
        uint32_t acc_phase[2] = {0u, 0u};
        uint32_t grp_phase = 0;                      // STREAM: phase of this warp group's barrier
        bool ok = true;
        // STREAM: the four warps that hold the same columns (one per TMEM lane quarter) share 2 QPW query rows; they meet
        // at a barrier of their own (bounded like every other wait)
        auto group_sync = [&]() -> bool {
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_group + 8 * colhalf);
            const bool good = __all_sync(0xFFFFFFFFu, mbar_wait(bar_group + 8 * colhalf, grp_phase, abort_flag));
            grp_phase ^= 1u;
            return good;
        };
        for (int64_t rho = 0; ok; ++rho) {
            const int64_t item_id = item_of_round(rho);
            if (item_id == -2) continue;
            if (item_id < 0) break;
            const int nkt = key_tiles_of_item(item_id);
            const int kt0 = first_tile_of_item(item_id);
            const int64_t item = n_sub == 1 ? item_id : item_id / n_sub;            // the block of query rows
            const TileOrder ord(nkt, STREAM ? Cfg::kSampleTiles : nkt);
            const int64_t row_base = item * QB;
            // STREAM: every thread has a list of its own per row (it sees one key of each tile), so it appends at a position
            // it keeps in a register: no vote, no atomic, nothing to wait for
            uint32_t my_count[STREAM ? 2 * QPW : 1];
#pragma unroll
            for (int c = 0; c < (STREAM ? 2 * QPW : 1); ++c) my_count[c] = 0u;
            // this thread's list of the group's first row; row c of the group is c / QPW * QPA + c % QPW rows further
            uint2* const my_list = STREAM ? p.st.cand + (row_base + colhalf * QPW) * kStreamRowSlots + kStreamSampleCap +
                                                (quarter * 32 + lane) * kStreamLaneCap
                                          : nullptr;
            uint64_t wreg[2][kGroupsPerEpiWarp];       // (w of column 8g+2j, w of column 8g+2j+1), packed
#pragma unroll
            for (int half = 0; half < 2; ++half) {
#pragma unroll
                for (int grp = 0; grp < kGroupsPerEpiWarp; ++grp) {
                    const int col = 8 * grp + 2 * j;                       // column within this warp's slice
                    const int64_t row = row_base + half * QPA + colhalf * QPW + (8 * grp) / H;
                    float2 v = make_float2(0.f, 0.f);
                    if (row < p.n_rows) {
                        v = __ldg(reinterpret_cast<const float2*>(p.w + row * H + col % H));
                        if constexpr (FP8) {
                            const float qs = __ldg(p.q_scale + row);
                            v.x *= qs; v.y *= qs;
                        }
                    }
                    wreg[half][grp] = pack_f32x2(v.x, v.y);
                }
            }
            for (int jt = 0; jt < nkt && ok; ++jt) {
                const int kt = STREAM ? ord.tile(jt) : kt0 + jt;
                const int64_t s = static_cast<int64_t>(kt) * kTileKeys + key_written;
                float ksc = 1.f;
                if constexpr (FP8) ksc = s < p.k_rows ? __ldg(p.k_scale + s) : 0.f;
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar_acc_full + 8 * half, acc_phase[half], abort_flag));   // warp-uniform
                    if (!ok) break;
                    acc_phase[half] ^= 1u;
                    tcgen05_fence_after_sync();
                    const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                                           static_cast<uint32_t>(half * kTileCols + colhalf * kColsPerEpiWarp);
                    // acc[r][i]: partial sums of (key slot r, query i) over this thread's even / odd columns
                    uint64_t acc[4][QPW];
#pragma unroll
                    for (int r = 0; r < 4; ++r)
#pragma unroll
                        for (int i = 0; i < QPW; ++i) acc[r][i] = 0ull;
                    uint32_t ra[16], rb[16];
                    tmem_ld_16x256b_x4(taddr, ra);
                    tmem_ld_wait(ra);
                    constexpr int NL = 2 * kChunksPerEpiWarp;
#pragma unroll
                    for (int n = 0; n < NL; ++n) {         // n = lane half (16 TMEM lanes) * chunks + 32-column chunk
                        uint32_t (&cur)[16] = (n & 1) ? rb : ra;
                        uint32_t (&nxt)[16] = (n & 1) ? ra : rb;
                        if (n + 1 < NL)
                            tmem_ld_16x256b_x4(taddr + (static_cast<uint32_t>(((n + 1) / kChunksPerEpiWarp) * 16) << 16) +
                                                   ((n + 1) % kChunksPerEpiWarp) * 32, nxt);
                        const int lh = n / kChunksPerEpiWarp, c = n % kChunksPerEpiWarp;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int grp = 4 * c + i;
                            const int qi = (8 * grp) / H;
                            // gate, then one packed FMA per key slot: (even column, odd column) * (w_even, w_odd)
                            const uint64_t xa = pack_f32x2(fmaxf(__uint_as_float(cur[4 * i + 0]), 0.f),
                                                           fmaxf(__uint_as_float(cur[4 * i + 1]), 0.f));
                            const uint64_t xb = pack_f32x2(fmaxf(__uint_as_float(cur[4 * i + 2]), 0.f),
                                                           fmaxf(__uint_as_float(cur[4 * i + 3]), 0.f));
                            acc[2 * lh][qi] = fma_f32x2(xa, wreg[half][grp], acc[2 * lh][qi]);
                            acc[2 * lh + 1][qi] = fma_f32x2(xb, wreg[half][grp], acc[2 * lh + 1][qi]);
                        }
                        if (n + 1 < NL) tmem_ld_wait(nxt);
                    }
                    // this warp's TMEM reads of the accumulator are complete
                    tcgen05_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_acc_empty + 8 * half);
#pragma unroll
                    for (int i = 0; i < QPW; ++i) {
                        float mine = 0.f;
                        {
                            // The four threads of a group each hold partial sums of the group's four keys; thread j wants
                            // the whole sum of key j. A butterfly does it in three shuffles: with the neighbour (xor 1) a
                            // thread keeps the two keys of its own parity and gives away the other two, with the thread
                            // two further (xor 2) it keeps its own key. The sum is ((own + xor 1) + (xor 2 + xor 3)).
                            float v[4];
#pragma unroll
                            for (int r = 0; r < 4; ++r) {
                                float lo, hi;
                                unpack_f32x2(acc[r][i], lo, hi);
                                v[r] = lo + hi;
                            }
                            const bool odd = (j & 1) != 0, upper = (j & 2) != 0;
                            float keep0 = odd ? v[1] : v[0], give0 = odd ? v[0] : v[1];
                            float keep1 = odd ? v[3] : v[2], give1 = odd ? v[2] : v[3];
                            keep0 += __shfl_xor_sync(0xFFFFFFFFu, give0, 1);
                            keep1 += __shfl_xor_sync(0xFFFFFFFFu, give1, 1);
                            const float keep = upper ? keep1 : keep0, give = upper ? keep0 : keep1;
                            mine = keep + __shfl_xor_sync(0xFFFFFFFFu, give, 2);
                        }
                        const int r_item = half * QPA + colhalf * QPW + i;
                        const int64_t row = row_base + half * QPA + colhalf * QPW + i;
                        const int64_t t = p.q_begin + row;
                        if constexpr (!STREAM) {
                            if (row < p.n_rows && s <= t) {
                                if constexpr (FP8) mine *= ksc;
                                p.scores[row * p.ld + s] = mine;
                            }
                        } else if (jt < ord.ns) {
                            if constexpr (FP8) mine *= ksc;
                            // a sample tile: every score goes to the row's sample (which of them are real is worked out
                            // from their place when the sample is read)
                            sample[r_item * Cfg::kSampleMax + jt * kTileKeys + key_written] = mine;
                        } else {
                            if constexpr (FP8) mine *= ksc;
                            // past the sample: only scores that are not below the row's threshold (a NaN stays in)
                            if (row < p.n_rows && s <= t && !(mine < row_tau[r_item])) {
                                const uint32_t pos = my_count[half * QPW + i]++;
                                if (pos < static_cast<uint32_t>(kStreamLaneCap))
                                    my_list[(half * QPA + i) * kStreamRowSlots + pos] = make_uint2(__float_as_uint(mine), static_cast<uint32_t>(s));
                            }
                        }
                    }
                }
                if constexpr (STREAM) {
                    if (ok && jt == ord.ns - 1) {
                        // ---- the sample is complete: each warp of the group takes the thresholds of its share of the rows
                        ok = group_sync();
                        if (!ok) break;
                        for (int idx = quarter; idx < 2 * QPW; idx += 4) {
                            const int r_item = (idx / QPW) * QPA + colhalf * QPW + idx % QPW;
                            const int64_t row = row_base + r_item;
                            if (row >= p.n_rows) continue;                          // warp-uniform
                            const int64_t t = p.q_begin + row;
                            const float* smp = sample + r_item * Cfg::kSampleMax;
                            // place p of the sample is key (p / 128) * stride * 128 + p % 128; keys grow with the place, so
                            // the real scores (key <= t) are the first n_valid places
                            const int64_t tile_span = static_cast<int64_t>(ord.stride) * kTileKeys;
                            const int64_t j_last = t / tile_span;
                            int n_valid = ord.ns * kTileKeys;
                            if (j_last < ord.ns) {
                                const int64_t in_tile = t - j_last * tile_span + 1;
                                n_valid = static_cast<int>(j_last) * kTileKeys + static_cast<int>(in_tile < kTileKeys ? in_tile : kTileKeys);
                            }
                            // rank (from the top) of the sample score wanted as threshold: where the k_top-th largest of the
                            // t + 1 scores is expected in a sample of n_valid, plus 4.5 standard deviations of that count
                            const float frac = static_cast<float>(n_valid) / static_cast<float>(t + 1);
                            const float expect = static_cast<float>(p.st.k_top) * frac;
                            const float rank_f = ceilf(expect + 4.5f * sqrtf(expect * fmaxf(1.f - frac, 0.f)) + 2.f);
                            float tau = -INFINITY;
                            if (rank_f < static_cast<float>(n_valid)) {
                                const uint32_t rank = static_cast<uint32_t>(rank_f);
                                // mean and spread of the sample, then 32 bins of 3/32 spreads around where a normal sample
                                // has that rank; the threshold is the lower edge of the highest bin that, with the bins
                                // above it, holds `rank` scores (a sample score of at least that rank: never too high)
                                float s1 = 0.f, s2 = 0.f;
                                for (int place = lane; place < n_valid; place += 32) {
                                    const float x = smp[place];
                                    s1 += x;
                                    s2 = fmaf(x, x, s2);
                                }
#pragma unroll
                                for (int o = 16; o > 0; o >>= 1) {
                                    s1 += __shfl_xor_sync(0xFFFFFFFFu, s1, o);
                                    s2 += __shfl_xor_sync(0xFFFFFFFFu, s2, o);
                                }
                                const float inv_n = 1.f / static_cast<float>(n_valid);
                                const float mean = s1 * inv_n;
                                const float sd = sqrtf(fmaxf(s2 * inv_n - mean * mean, 0.f));
                                const float z = topk::upper_quantile_z(static_cast<float>(rank) * inv_n);
                                const float lo_edge = mean + (z - 1.5f) * sd;
                                const float scale = 32.f / (3.f * sd);
                                if (sd > 0.f && fabsf(scale) < 3.0e38f && fabsf(lo_edge) < 3.0e38f) {      // finite, not constant
                                    uint32_t* hist = warp_hist + (warp - kEpilogueWarp0) * 32;
                                    hist[lane] = 0u;
                                    __syncwarp();
                                    for (int place = lane; place < n_valid; place += 32) {
                                        const int bin = __float2int_rd((smp[place] - lo_edge) * scale);
                                        if (bin >= 0) atomicAdd(&hist[bin < 31 ? bin : 31], 1u);
                                    }
                                    __syncwarp();
                                    uint32_t from_top = hist[lane];                       // scores in bins lane .. 31
#pragma unroll
                                    for (int o = 1; o < 32; o <<= 1) {
                                        const uint32_t y = __shfl_down_sync(0xFFFFFFFFu, from_top, o);
                                        if (lane + o < 32) from_top += y;
                                    }
                                    const uint32_t reach = __ballot_sync(0xFFFFFFFFu, from_top >= rank);
                                    if (reach != 0u) tau = lo_edge + static_cast<float>(31 - __clz(reach)) / scale;
                                    __syncwarp();
                                }
                            }
                            // the sample's own scores that are not below the threshold open the row's list
                            uint32_t mine_mask = 0;                                   // bit e: place lane + 32 e passes
                            for (int e = 0; e < Cfg::kSampleMax / 32; ++e) {
                                const int place = lane + 32 * e;
                                if (place < n_valid && !(smp[place] < tau)) mine_mask |= 1u << e;
                            }
                            uint32_t total;
                            uint32_t pos = topk::warp_excl_scan(static_cast<uint32_t>(__popc(mine_mask)), lane, total);
                            while (mine_mask != 0u) {
                                const int e = __ffs(mine_mask) - 1;
                                mine_mask &= mine_mask - 1u;
                                const int place = lane + 32 * e;
                                if (pos < static_cast<uint32_t>(kStreamSampleCap))
                                    p.st.cand[row * kStreamRowSlots + pos] =
                                        make_uint2(__float_as_uint(smp[place]), static_cast<uint32_t>((place >> 7) * tile_span + (place & 127)));
                                ++pos;
                            }
                            if (lane == 0) p.st.sample_count[row] = total;       // (never above kStreamSampleCap: the sample is no larger)
                            if (lane == 0) row_tau[r_item] = tau;
                        }
                        ok = group_sync();
                        if (!ok) break;
                    }
                }
            }
            if constexpr (STREAM) {
                // ---- end of the item: this warp's sub-list lengths go out (and the thresholds of the rows it owns)
                if (!ok) break;
#pragma unroll
                for (int c = 0; c < 2 * QPW; ++c) {
                    const int r_item = (c / QPW) * QPA + colhalf * QPW + c % QPW;
                    const int64_t row = row_base + r_item;
                    if (row < p.n_rows) {
                        p.st.lane_count[row * kStreamLanes + quarter * 32 + lane] = static_cast<uint8_t>(my_count[c] < 255u ? my_count[c] : 255u);
                        if (lane == 0 && (c & 3) == quarter) p.st.tau[row] = row_tau[r_item];
                    }
                }
            }
        }
        if (!ok && lane == 0) give_up(abort_flag, p.status, DEV_TIMEOUT_EPILOGUE);
    }

    // ------------------------------------------------------------------- teardown
    __syncwarp();
    if (*abort_flag) {
        // a role gave up: give copies that may still be in flight time to land before
        // shared memory and TMEM are released (bounded: about a millisecond)
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tcgen05_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
}

template <int NKH, int H, bool FP8, bool STREAM, bool SPLIT>
cudaError_t launch_prefill_kernel(const PrefillParams& p, int grid, const CUtensorMap& q_map, const CUtensorMap& k_map, cudaStream_t stream) {
    using Cfg = PrefillCfg<NKH, H, STREAM>;
    auto kern = score_prefill_tc_kernel<NKH, H, FP8, STREAM, SPLIT>;
    if (cudaError_t e = ensure_max_dynamic_smem(reinterpret_cast<const void*>(kern), Cfg::kSmemBytes); e != cudaSuccess) return e;
    kern<<<grid, kPrefillThreads, Cfg::kSmemBytes, stream>>>(q_map, k_map, p);
    return cudaGetLastError();
}

template <int NKH, int H, bool FP8, bool STREAM>
cudaError_t launch_prefill_variant(const ScoreArgs& a, const CUtensorMap& q_map, const CUtensorMap& k_map,
                                   unsigned int* status, int sm_count, cudaStream_t stream) {
    constexpr int QB = 2 * (kTileCols / H);
    const int64_t n_blocks = (a.n_rows + QB - 1) / QB;
    // Few blocks of query rows (a short prompt, or a short chunk of queries against a long context) leave SMs idle and
    // the longest block sets the time: the blocks' key tiles are then cut into runs of key_split tiles (the scores of a
    // row's keys are independent, so any cut is exact; the query tile is loaded once per run). The split with the
    // shortest makespan rounds x run length among those that give the grid 1 to 4 items per SM; not with the streaming
    // top-k, whose threshold needs a row's sample before the rest of its tiles.
    int sub_per_block = 1, key_split = 0;
    if (!STREAM && n_blocks < 2 * static_cast<int64_t>(sm_count)) {
        const int64_t tiles_longest = (a.q_begin + a.n_rows + kTileKeys - 1) / kTileKeys;
        const int64_t tiles_first = (a.q_begin + (a.n_rows < QB ? a.n_rows : QB) + kTileKeys - 1) / kTileKeys;
        const int64_t total = (tiles_first + tiles_longest) * n_blocks / 2;          // the blocks' tile counts grow linearly
        int64_t best = ((n_blocks + sm_count - 1) / sm_count) * (tiles_longest + 1);
        for (int m = 1; m <= 4; ++m) {
            int64_t split = (total + static_cast<int64_t>(m) * sm_count - 1) / (static_cast<int64_t>(m) * sm_count);
            if (split < 4) split = 4;
            if (split >= tiles_longest) continue;
            const int64_t subs = (tiles_longest + split - 1) / split;
            // runs that are not empty: block b has ceil(tiles_b / split) of them; estimated from the linear growth
            const int64_t n_runs = n_blocks * ((tiles_first + tiles_longest) / 2 + split - 1) / split;
            const int64_t cost = ((n_runs + sm_count - 1) / sm_count) * (split + 1);
            if (cost < best) { best = cost; sub_per_block = static_cast<int>(subs); key_split = static_cast<int>(split); }
        }
    }
    const int64_t n_items = n_blocks * sub_per_block;
    const int grid = static_cast<int>(n_items < sm_count ? n_items : sm_count);
    PrefillParams p{a.w, a.q_scale, a.k_scale, a.scores, a.ld, a.q_begin, a.n_rows, a.k_rows, status, a.stream, a.item_mask,
                    sub_per_block, key_split};
    if constexpr (!STREAM) {
        if (sub_per_block > 1) return launch_prefill_kernel<NKH, H, FP8, false, true>(p, grid, q_map, k_map, stream);
    }
    return launch_prefill_kernel<NKH, H, FP8, STREAM, false>(p, grid, q_map, k_map, stream);
}

template <int NKH, int H, bool FP8>
cudaError_t launch_prefill_instance(const ScoreArgs& a, const CUtensorMap& q_map, const CUtensorMap& k_map,
                                    unsigned int* status, int sm_count, cudaStream_t stream) {
    if (a.stream.cand != nullptr) {
        if constexpr (PrefillCfg<NKH, H, true>::kFits)
            return launch_prefill_variant<NKH, H, FP8, true>(a, q_map, k_map, status, sm_count, stream);
        else
            return cudaErrorInvalidValue;
    }
    return launch_prefill_variant<NKH, H, FP8, false>(a, q_map, k_map, status, sm_count, stream);
}

}  // namespace

bool score_tc_supported(int H, int d, int fp8) {
    if (H != 16 && H != 32 && H != 64) return false;
    if (fp8) return d == 128;
    return d == 64 || d == 128;
}

bool score_prefill_stream_supported(int H, int d, int fp8) {
    if (!score_tc_supported(H, d, fp8)) return false;
    const int nkh = fp8 ? 1 : d / 64;
    switch (H) {
        case 16: return nkh == 2 ? PrefillCfg<2, 16, true>::kFits : PrefillCfg<1, 16, true>::kFits;
        case 32: return nkh == 2 ? PrefillCfg<2, 32, true>::kFits : PrefillCfg<1, 32, true>::kFits;
        default: return nkh == 2 ? PrefillCfg<2, 64, true>::kFits : PrefillCfg<1, 64, true>::kFits;
    }
}

int score_prefill_rows_per_item(int H) { return 2 * (kTileCols / H); }

cudaError_t launch_score_prefill_tc(const ScoreArgs& a, const CUtensorMap& q_map, const CUtensorMap& k_map,
                                    unsigned int* status, int sm_count, cudaStream_t stream) {
    if (a.n_rows <= 0) return cudaSuccess;
#define IDXC_DISPATCH_H(NKH, FP8)                                                                              \
    switch (a.H) {                                                                                             \
        case 16: return launch_prefill_instance<NKH, 16, FP8>(a, q_map, k_map, status, sm_count, stream);      \
        case 32: return launch_prefill_instance<NKH, 32, FP8>(a, q_map, k_map, status, sm_count, stream);      \
        case 64: return launch_prefill_instance<NKH, 64, FP8>(a, q_map, k_map, status, sm_count, stream);      \
        default: return cudaErrorInvalidValue;                                                                 \
    }
    if (a.fp8) {
        if (a.d == 128) { IDXC_DISPATCH_H(1, true) }
        return cudaErrorInvalidValue;
    }
    if (a.d == 64) { IDXC_DISPATCH_H(1, false) }
    if (a.d == 128) { IDXC_DISPATCH_H(2, false) }
#undef IDXC_DISPATCH_H
    return cudaErrorInvalidValue;
}

// ===================================================================== decode
namespace {

constexpr int kDecodeEpiWarps = 8;       // two groups of 4 (one warp per TMEM lane quarter); group g drains slots g, g+2
constexpr int kDecodeMmaWarps = 2;      // warp 1 and (if 2) the last warp: key tiles alternate between them
constexpr int kDecodeThreads = (1 + kDecodeMmaWarps + kDecodeEpiWarps) * 32;   // warp 0 producer, warp 1 MMA, warps 2-9 epilogue, warp 10 MMA
// Key tiles (of 128 keys, 256-byte rows) per work item; twice as many when a row is 128 bytes, so that an item is
// the same stretch of HBM. Measured on B200 (bf16, d = 128, B = 32, 16K-128K keys per sequence): 16 tiles stream
// at 6.1 TB/s; 6-8 tiles per item lose 20 % (all CTAs then walk HBM with the same 192-256 KB stride).
constexpr int kDecodeChunkTiles = 16;
constexpr int kDecodeAccSlots = 8;       // TMEM accumulators in flight (64 columns apart: all 512 columns)

template <int NKH, int H>
struct DecodeCfg {
    static constexpr int kStages = NKH == 2 ? 5 : 8;
    static constexpr int kQRegion = H * kChunkBytes;                  // one 128-byte chunk of the query tile
    static constexpr int kQBytes = 2 * NKH * kQRegion;                // double buffered
    static constexpr int kKBytes = kStages * NKH * kKRegionBytes;
    static constexpr int kWBytes = kDecodeEpiWarps * 64 * 4;          // per epilogue warp: w of the item's sequence
    static constexpr int kMaxChunk = kDecodeChunkTiles * 2 / NKH;     // key tiles per work item, at most
    static constexpr int kMaxOwn = (kMaxChunk + 1) / 2;               // ... of which one group of epilogue warps drains
    static constexpr int kScaleBytes = kDecodeEpiWarps * 2 * kMaxOwn * 32 * 4;   // FP8 key scales: [warp][2 items][own tile][lane]
    static constexpr int kBarBytes = 512;
    static constexpr int kSmemBytes = kQBytes + kKBytes + kWBytes + kScaleBytes + kBarBytes + 1024;
};

struct DecodeParams {
    const float* w;
    const float* q_scale;
    const float* k_scale;
    const int64_t* k_offsets;
    const int32_t* lens;
    float* scores;
    int64_t ld;
    int64_t max_len;
    int B;
    int chunk_tiles;       // key tiles per work item, at most kDecodeChunkTiles (chosen at launch for the grid's balance)
    unsigned int* status;
};

// Walks the (sequence, chunk) work items of one CTA: items are numbered sequence-major,
// sequence b having ceil(len_b / (128 * chunk_tiles)) of them; CTA c takes items
// c, c + G, c + 2G, ...
struct DecodeItemWalker {
    const int32_t* lens;
    int64_t max_len;
    int B, G, chunk;
    int64_t next;        // next item number of this CTA
    int b;               // sequence the cursor is in
    int64_t base;        // first item number of sequence b
    __device__ DecodeItemWalker(const DecodeParams& p, int cta, int grid)
        : lens(p.lens), max_len(p.max_len), B(p.B), G(grid), chunk(p.chunk_tiles), next(cta), b(0), base(0) {}
    __device__ int len_of(int bb) const {
        int64_t l = lens[bb];
        l = l < 0 ? 0 : (l > max_len ? max_len : l);
        return static_cast<int>(l);
    }
    // Fetches the next item: sequence, first key tile, number of key tiles, sequence length.
    __device__ bool pop(int& seq, int& tile0, int& ntiles, int& len) {
        while (b < B) {
            const int l = len_of(b);
            const int tiles = (l + kTileKeys - 1) / kTileKeys;
            const int chunks = (tiles + chunk - 1) / chunk;
            if (next < base + chunks) {
                const int c = static_cast<int>(next - base);
                seq = b;
                tile0 = c * chunk;
                ntiles = tiles - tile0 < chunk ? tiles - tile0 : chunk;
                len = l;
                next += G;
                return true;
            }
            base += chunks;
            ++b;
        }
        return false;
    }
};

template <int NKH, int H, bool FP8>
__global__ void __launch_bounds__(kDecodeThreads, 1)
score_decode_tc_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                       const DecodeParams p) {
    using Cfg = DecodeCfg<NKH, H>;
    constexpr int kStages = Cfg::kStages;
    constexpr int kElemsPerChunk = FP8 ? 128 : 64;
    constexpr uint32_t kIdesc = FP8 ? umma_idesc(0, 0, kTileKeys, H) : umma_idesc(1, 1, kTileKeys, H);
    // Two MMA warps only when the key ring has an even number of stages: a stage then always belongs to the same warp.
    // With an odd ring a warp would wait for every other phase of a stage's barrier, and a parity wait cannot tell the
    // phase it wants from the one two before it.
    constexpr int kMmaWarps = (kStages % 2 == 0 && kDecodeAccSlots % 2 == 0) ? kDecodeMmaWarps : 1;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t* k_smem = smem;                                  // [kStages][NKH][128 x 128 B]
    uint8_t* q_smem = k_smem + Cfg::kKBytes;                 // [2][NKH][H x 128 B]
    float* w_smem = reinterpret_cast<float*>(q_smem + Cfg::kQBytes);   // [4 warps][64]
    float* scale_smem = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(w_smem) + Cfg::kWBytes);
    uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(scale_smem) + Cfg::kScaleBytes);
    const uint32_t bar_q_full = smem_u32(bars + 0);          // [2]
    const uint32_t bar_q_empty = smem_u32(bars + 2);         // [2]
    const uint32_t bar_acc_full = smem_u32(bars + 4);        // [kDecodeAccSlots]
    const uint32_t bar_acc_empty = smem_u32(bars + 4 + kDecodeAccSlots);
    const uint32_t bar_k_full = smem_u32(bars + 4 + 2 * kDecodeAccSlots);         // [kStages]
    const uint32_t bar_k_empty = smem_u32(bars + 4 + 2 * kDecodeAccSlots + kStages);
    uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(bars + 4 + 2 * kDecodeAccSlots + 2 * kStages);
    static_assert((5 + 2 * kDecodeAccSlots + 2 * kStages) * 8 <= Cfg::kBarBytes && kDecodeAccSlots * 64 <= 512, "barrier area, tensor memory");
    volatile uint32_t* abort_flag = tmem_base_slot + 1;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar_q_full + 8 * i, 1);
            mbar_init(bar_q_empty + 8 * i, kMmaWarps);
        }
        for (int i = 0; i < kDecodeAccSlots; ++i) {
            mbar_init(bar_acc_full + 8 * i, 1);
            mbar_init(bar_acc_empty + 8 * i, 4);
        }
        for (int i = 0; i < kStages; ++i) {
            mbar_init(bar_k_full + 8 * i, 1);
            mbar_init(bar_k_empty + 8 * i, 1);
        }
        *abort_flag = 0u;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_base_slot), kDecodeAccSlots * 64);
        tmem_relinquish_alloc_permit();
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    tcgen05_fence_after_sync();
    const uint32_t tmem_base = *tmem_base_slot;

    DecodeItemWalker walk(p, blockIdx.x, gridDim.x);
    int seq, tile0, ntiles, len;

    if (warp == 0) {
        if (lane == 0) {
            tma_prefetch_desc(&q_map);
            tma_prefetch_desc(&k_map);
            int stage = 0, qbuf = 0;
            uint32_t k_phase = 0, q_phase[2] = {0u, 0u};
            bool ok = true;
            while (ok && walk.pop(seq, tile0, ntiles, len)) {
                ok = mbar_wait(bar_q_empty + 8 * qbuf, q_phase[qbuf] ^ 1u, abort_flag);
                if (!ok) break;
                q_phase[qbuf] ^= 1u;
                mbar_arrive_expect_tx(bar_q_full + 8 * qbuf, NKH * Cfg::kQRegion);
                for (int kh = 0; kh < NKH; ++kh)
                    tma_load_2d(smem_u32(q_smem + (qbuf * NKH + kh) * Cfg::kQRegion), &q_map, bar_q_full + 8 * qbuf,
                                kh * kElemsPerChunk, seq * H);
                const int64_t row0 = p.k_offsets[seq] + static_cast<int64_t>(tile0) * kTileKeys;
                for (int kt = 0; kt < ntiles && ok; ++kt) {
                    ok = mbar_wait(bar_k_empty + 8 * stage, k_phase ^ 1u, abort_flag);
                    if (!ok) break;
                    mbar_arrive_expect_tx(bar_k_full + 8 * stage, NKH * kKRegionBytes);
                    for (int kh = 0; kh < NKH; ++kh)
                        tma_load_2d(smem_u32(k_smem + (stage * NKH + kh) * kKRegionBytes), &k_map, bar_k_full + 8 * stage,
                                    kh * kElemsPerChunk, static_cast<int>(row0 + kt * kTileKeys));
                    if (++stage == kStages) { stage = 0; k_phase ^= 1u; }
                }
                qbuf ^= 1;
            }
            if (!ok) give_up(abort_flag, p.status, DEV_TIMEOUT_PRODUCER);
        }
    } else if (warp == 1 || (kMmaWarps == 2 && warp == 2 + kDecodeEpiWarps)) {
        // The whole warp runs this role with uniform control flow and one elected lane issues (a single diverged lane
        // issues the same instruction stream about 1.5x slower); descriptors are a base plus 16-byte units.
        // With two such warps the key tiles alternate between them (a tile is four to eight small MMAs, two commits and
        // two barrier waits, and one warp gets through that more slowly than 16 KB tiles arrive): warp m takes the tiles
        // whose running number has parity m, which are also the accumulator slots of parity m; both walk all tiles to
        // keep the ring position and the phases.
        const int mma_id = warp == 1 ? 0 : 1;
        int stage = 0, qbuf = 0, slot = 0;
        uint32_t k_phase = 0, q_phase[2] = {0u, 0u}, acc_phase = 0;   // acc_phase: one bit per accumulator slot
        bool ok = true;
        const uint64_t a_desc0 = umma_smem_desc_sw128(smem_u32(k_smem));
        const uint64_t b_desc0 = umma_smem_desc_sw128(smem_u32(q_smem));
        auto wait_bar = [&](uint32_t bar, uint32_t parity) -> bool {
            return __all_sync(0xFFFFFFFFu, mbar_wait(bar, parity, abort_flag));
        };
        while (ok && walk.pop(seq, tile0, ntiles, len)) {
            ok = wait_bar(bar_q_full + 8 * qbuf, q_phase[qbuf]);
            if (!ok) break;
            q_phase[qbuf] ^= 1u;
            const uint64_t b_desc = b_desc0 + static_cast<uint64_t>(qbuf * NKH * Cfg::kQRegion / 16);
            for (int kt = 0; kt < ntiles && ok; ++kt) {
                if (kMmaWarps == 1 || (slot & 1) == mma_id) {
                    ok = wait_bar(bar_k_full + 8 * stage, k_phase) && wait_bar(bar_acc_empty + 8 * slot, ((acc_phase >> slot) & 1u) ^ 1u);
                    if (!ok) break;
                    acc_phase ^= 1u << slot;
                    tcgen05_fence_after_sync();
                    const uint32_t d_tmem = tmem_base + slot * 64;
                    const uint64_t a_desc = a_desc0 + static_cast<uint64_t>(stage * NKH * kKRegionBytes / 16);
#pragma unroll
                    for (int kh = 0; kh < NKH; ++kh) {
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) {
                            const uint64_t a = a_desc + (kh * kKRegionBytes + ks * 32) / 16, b = b_desc + (kh * Cfg::kQRegion + ks * 32) / 16;
                            if constexpr (FP8) {
                                if ((kh | ks) != 0) umma_f8_elect<true>(d_tmem, a, b, kIdesc);
                                else umma_f8_elect<false>(d_tmem, a, b, kIdesc);
                            } else {
                                if ((kh | ks) != 0) umma_f16_elect<true>(d_tmem, a, b, kIdesc);
                                else umma_f16_elect<false>(d_tmem, a, b, kIdesc);
                            }
                        }
                    }
                    umma_commit_elect(bar_acc_full + 8 * slot);
                    umma_commit_elect(bar_k_empty + 8 * stage);
                }
                // the query buffer is free once the item's MMAs of BOTH warps are complete: each commits after its last
                // tile of the item (a commit with nothing outstanding arrives at once)
                if (kt == ntiles - 1) umma_commit_elect(bar_q_empty + 8 * qbuf);
                if (++stage == kStages) { stage = 0; k_phase ^= 1u; }
                slot = (slot + 1) & (kDecodeAccSlots - 1);
            }
            qbuf ^= 1;
        }
        if (!ok && lane == 0) give_up(abort_flag, p.status, DEV_TIMEOUT_MMA);
    } else if (warp < 2 + kDecodeEpiWarps) {
        const int quarter = warp & 3;
        const int grp = (warp - 2) >> 2;                 // which accumulator slots this warp drains
        const int key_in_tile = quarter * 32 + lane;
        float* my_w = w_smem + (warp - 2) * 64;
        int slot = 0;
        uint32_t acc_phase = 0;                          // one bit per accumulator slot
        bool ok = true;
        // What a work item needs besides its accumulators is fetched one item ahead, by a second walker: w of the item's
        // sequence (times its query scale) into registers and, FP8, the scales of this thread's keys in the tiles this
        // warp will drain, by 4-byte cp.async into a staging area of its own (two items deep, a slot per lane and tile).
        // Asked for tile by tile they cost the warp a memory latency each, and any per-tile bookkeeping is dear in a warp
        // that has its scheduler almost to itself (a dependent instruction every 4-6 cycles).
        constexpr int kWPerLane = (H + 31) / 32;
        constexpr int kMaxOwn = Cfg::kMaxOwn;
        float* my_scales = scale_smem + (warp - 2) * (2 * kMaxOwn * 32) + lane;
        DecodeItemWalker walk_next(p, blockIdx.x, gridDim.x);
        float w_next[kWPerLane];
        int next_slot0 = 0;                              // accumulator slot of the next item's first tile
        int stage_buf = 0;                               // staging buffer the next fetch goes to
        auto fetch_next = [&]() {                        // always commits one cp.async group
            int s2, t2, n2, l2;
            if (walk_next.pop(s2, t2, n2, l2)) {
                float qs = 1.f;
                if constexpr (FP8) qs = __ldg(p.q_scale + s2);
#pragma unroll
                for (int i = 0; i < kWPerLane; ++i) {
                    const int h = lane + 32 * i;
                    w_next[i] = h < H ? __ldg(p.w + static_cast<int64_t>(s2) * H + h) * qs : 0.f;
                }
                if constexpr (FP8) {
                    const int kt0 = ((next_slot0 & 1) != grp) ? 1 : 0;          // this group's first tile of the item
                    const int s_first = (t2 + kt0) * kTileKeys + key_in_tile;
                    const float* src = p.k_scale + p.k_offsets[s2] + s_first;
                    const uint32_t dst = smem_u32(my_scales + stage_buf * (kMaxOwn * 32));
#pragma unroll
                    for (int j = 0; j < kMaxOwn; ++j)
                        if (kt0 + 2 * j < n2 && s_first + 2 * kTileKeys * j < l2) cp_async_4(dst + j * 128, src + 2 * kTileKeys * j);
                }
                next_slot0 = (next_slot0 + n2) & (kDecodeAccSlots - 1);
            }
            if constexpr (FP8) cp_async_commit();
            stage_buf ^= 1;
        };
        fetch_next();
        while (ok && walk.pop(seq, tile0, ntiles, len)) {
            __syncwarp();
#pragma unroll
            for (int i = 0; i < kWPerLane; ++i)
                if (lane + 32 * i < H) my_w[lane + 32 * i] = w_next[i];
            const float* item_scales = my_scales + (stage_buf ^ 1) * (kMaxOwn * 32);   // where the last fetch went
            fetch_next();
            if constexpr (FP8) cp_async_wait_group<1>();   // this item's scales (the group before the one just committed) are in
            __syncwarp();
            const float4* w4 = reinterpret_cast<const float4*>(my_w);
            for (int kt = 0; kt < ntiles && ok; ++kt, slot = (slot + 1) & (kDecodeAccSlots - 1)) {
                if ((slot & 1) != grp) continue;         // the other group's tile
                const int s = (tile0 + kt) * kTileKeys + key_in_tile;
                float ksc = 1.f;
                if constexpr (FP8) {
                    if (s < len) ksc = *item_scales;       // (slots of keys past the end were not written)
                    item_scales += 32;
                }
                ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar_acc_full + 8 * slot, (acc_phase >> slot) & 1u, abort_flag));   // warp-uniform
                if (!ok) break;
                acc_phase ^= 1u << slot;
                tcgen05_fence_after_sync();
                const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + static_cast<uint32_t>(slot * 64);
                float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;    // four independent partial sums over the heads
                // the accumulator is in registers once its loads have completed: the slot goes back to the MMA warp
                // before the head sums, not after
                auto release_slot = [&]() {
                    tcgen05_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_acc_empty + 8 * slot);
                };
                if constexpr (H == 16) {
                    uint32_t r[16];
                    tmem_ld_32x32b_x16(taddr, r);
                    tmem_ld_wait(r);
                    release_slot();
#pragma unroll
                    for (int j4 = 0; j4 < 4; ++j4) {
                        const float4 wv = w4[j4];
                        a0 = fmaf(fmaxf(__uint_as_float(r[4 * j4 + 0]), 0.f), wv.x, a0);
                        a1 = fmaf(fmaxf(__uint_as_float(r[4 * j4 + 1]), 0.f), wv.y, a1);
                        a2 = fmaf(fmaxf(__uint_as_float(r[4 * j4 + 2]), 0.f), wv.z, a2);
                        a3 = fmaf(fmaxf(__uint_as_float(r[4 * j4 + 3]), 0.f), wv.w, a3);
                    }
                } else {
                    uint32_t ra[32], rb[32];
                    tmem_ld_32x32b_x32(taddr, ra);
                    if constexpr (H == 64) tmem_ld_32x32b_x32(taddr + 32, rb);
                    tmem_ld_wait(ra);                    // waits for every load issued so far
                    if constexpr (H == 64) tmem_ld_wait(rb);
                    release_slot();
#pragma unroll
                    for (int j4 = 0; j4 < 8; ++j4) {
                        const float4 wv = w4[j4];
                        a0 = fmaf(fmaxf(__uint_as_float(ra[4 * j4 + 0]), 0.f), wv.x, a0);
                        a1 = fmaf(fmaxf(__uint_as_float(ra[4 * j4 + 1]), 0.f), wv.y, a1);
                        a2 = fmaf(fmaxf(__uint_as_float(ra[4 * j4 + 2]), 0.f), wv.z, a2);
                        a3 = fmaf(fmaxf(__uint_as_float(ra[4 * j4 + 3]), 0.f), wv.w, a3);
                    }
                    if constexpr (H == 64) {
#pragma unroll
                        for (int j4 = 0; j4 < 8; ++j4) {
                            const float4 wv = w4[8 + j4];
                            a0 = fmaf(fmaxf(__uint_as_float(rb[4 * j4 + 0]), 0.f), wv.x, a0);
                            a1 = fmaf(fmaxf(__uint_as_float(rb[4 * j4 + 1]), 0.f), wv.y, a1);
                            a2 = fmaf(fmaxf(__uint_as_float(rb[4 * j4 + 2]), 0.f), wv.z, a2);
                            a3 = fmaf(fmaxf(__uint_as_float(rb[4 * j4 + 3]), 0.f), wv.w, a3);
                        }
                    }
                }
                if (s < len) {
                    float acc = (a0 + a1) + (a2 + a3);
                    if constexpr (FP8) acc *= ksc;
                    p.scores[static_cast<int64_t>(seq) * p.ld + s] = acc;
                }
            }
        }
        if (!ok && lane == 0) give_up(abort_flag, p.status, DEV_TIMEOUT_EPILOGUE);
    }

    __syncwarp();
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tcgen05_fence_after_sync();
        tmem_dealloc(tmem_base, kDecodeAccSlots * 64);
    }
}

template <int NKH, int H, bool FP8>
cudaError_t launch_decode_instance(const ScoreArgs& a, const CUtensorMap& q_map, const CUtensorMap& k_map,
                                   unsigned int* status, int sm_count, cudaStream_t stream) {
    using Cfg = DecodeCfg<NKH, H>;
    auto kern = score_decode_tc_kernel<NKH, H, FP8>;
    if (cudaError_t e = ensure_max_dynamic_smem(reinterpret_cast<const void*>(kern), Cfg::kSmemBytes); e != cudaSuccess) return e;
    const int64_t tiles = (a.max_len + kTileKeys - 1) / kTileKeys;
    // Tiles per work item, estimated with every sequence at max_len (the lengths live on the device): the size with the
    // lowest rounds x (size + one tile's worth of hand-over per item). 512 KB of keys streams best at a large batch
    // (shorter items cost about 5 %), but a small batch must be cut finer to give every SM an item (one sequence of
    // 131072 e4m3 keys in items of 28 tiles is 37 items for 148 SMs). Items of 192 to 256 KB count a quarter dearer: the CTAs
    // then walk HBM in lock-step at a stride that costs a fifth of the bandwidth. The larger size wins a tie.
    constexpr int kTileBytes = NKH * kKRegionBytes;
    const int cmax = Cfg::kMaxChunk;
    int chunk = cmax;
    int64_t best = -1;
    for (int c = cmax; c >= 2; --c) {
        const int item_bytes = c * kTileBytes;
        const bool bad_stride = item_bytes > 160 * 1024 && item_bytes < 320 * 1024;
        const int64_t n_items = a.n_rows * ((tiles + c - 1) / c);
        const int64_t cost = ((n_items + sm_count - 1) / sm_count) * (c + 1) * (bad_stride ? 5 : 4);   // (a quarter dearer)
        if (best < 0 || cost < best) { best = cost; chunk = c; }
    }
    const int64_t items = a.n_rows * ((tiles + chunk - 1) / chunk);
    if (items <= 0) return cudaSuccess;
    const int grid = static_cast<int>(items < sm_count ? items : sm_count);
    DecodeParams p{a.w, a.q_scale, a.k_scale, a.k_offsets, a.lens, a.scores, a.ld, a.max_len, static_cast<int>(a.n_rows), chunk, status};
    kern<<<grid, kDecodeThreads, Cfg::kSmemBytes, stream>>>(q_map, k_map, p);
    return cudaGetLastError();
}

}  // namespace

// Loads every decode scorer instance on the current device and raises its shared-memory limit, so that no later
// launch has to (a kernel's first use on a device makes the driver load its code).
cudaError_t preload_score_decode_tc() {
    cudaError_t e = cudaSuccess;
    auto one = [&](const void* kern, int smem) {
        cudaFuncAttributes fa;
        if (e == cudaSuccess) e = cudaFuncGetAttributes(&fa, kern);
        if (e == cudaSuccess) e = ensure_max_dynamic_smem(kern, smem);
    };
#define IDXC_PRELOAD(NKH, H, FP8) one(reinterpret_cast<const void*>(score_decode_tc_kernel<NKH, H, FP8>), DecodeCfg<NKH, H>::kSmemBytes);
    IDXC_PRELOAD(1, 16, false) IDXC_PRELOAD(1, 32, false) IDXC_PRELOAD(1, 64, false)
    IDXC_PRELOAD(2, 16, false) IDXC_PRELOAD(2, 32, false) IDXC_PRELOAD(2, 64, false)
    IDXC_PRELOAD(1, 16, true) IDXC_PRELOAD(1, 32, true) IDXC_PRELOAD(1, 64, true)
#undef IDXC_PRELOAD
    return e;
}

cudaError_t launch_score_decode_tc(const ScoreArgs& a, const CUtensorMap& q_map, const CUtensorMap& k_map,
                                   unsigned int* status, int sm_count, cudaStream_t stream) {
    if (a.n_rows <= 0 || a.max_len <= 0) return cudaSuccess;
#define IDXC_DISPATCH_H(NKH, FP8)                                                                             \
    switch (a.H) {                                                                                            \
        case 16: return launch_decode_instance<NKH, 16, FP8>(a, q_map, k_map, status, sm_count, stream);      \
        case 32: return launch_decode_instance<NKH, 32, FP8>(a, q_map, k_map, status, sm_count, stream);      \
        case 64: return launch_decode_instance<NKH, 64, FP8>(a, q_map, k_map, status, sm_count, stream);      \
        default: return cudaErrorInvalidValue;                                                                \
    }
    if (a.fp8) {
        if (a.d == 128) { IDXC_DISPATCH_H(1, true) }
        return cudaErrorInvalidValue;
    }
    if (a.d == 64) { IDXC_DISPATCH_H(1, false) }
    if (a.d == 128) { IDXC_DISPATCH_H(2, false) }
#undef IDXC_DISPATCH_H
    return cudaErrorInvalidValue;
}

}  // namespace idxc
