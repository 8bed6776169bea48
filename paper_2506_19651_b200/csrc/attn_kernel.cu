// Warp-specialised block-masked flash attention for sm_100a (Eq. 1 under the masks of Eq. 3-5).
//
// One CTA owns TWO query tiles of 128 rows that share a kv head and a key-tile list (two q
// heads of one GQA group at the same block position, or two neighbouring positions), so every
// K/V tile staged in shared memory feeds both.  Roles (12 warps):
//   warps 0-3   softmax and epilogue of query tile 0: one thread per row; the 128 scores of a key
//               tile are read from TMEM once, running max/sum kept in fp32, probabilities written
//               back over the scores as bf16; the rare rescale of the O accumulator (the reference
//               maximum moves only when a row's maximum grows by more than 2^8) is done in place
//               by the same threads.  After the item's last key tile the same thread reads its
//               row of the accumulator in one round trip, releases the accumulator, and writes
//               the normalised output and the LSE
//   warps 4-7   the same for query tile 1
//   warp 8      issues the tcgen05 MMAs: S = Q K^T (both operands from shared memory) and
//               O += P V (P from TMEM, V from shared memory), ping-ponging between the two
//               query tiles so one is in the tensor cores while the other is in its softmax
//   warp 9      work scheduler and TMA producer: takes the next work item from a global
//               counter, decodes it once into shared memory for the other roles (the decode is
//               a dozen integer divisions), loads its two Q tiles, then streams K/V tiles
//               through a 4-slot ring that runs on across items
//   warps 10-11 idle (they complete the third warpgroup for the register reallocation)
// The kernel is persistent (one CTA per SM): while the softmax threads write out item k, the
// producer and the MMA warp already work on item k+1.
// TMEM (512 columns): S0/P0 [0,128) S1/P1 [128,256) O0 [256,384) O1 [384,512).
// Every wait is bounded; an expired wait records PEVLM_ETIMEOUT and the CTA still runs to its
// normal end (waits become short), so TMEM is always released.
#include "internal.h"
#include "ptx.cuh"

namespace pevlm {

constexpr int kAttnThreads = 384;
constexpr int kRing = 4;
constexpr float kRescaleThresholdLog2 = 8.0f;  // rescale O only when the row maximum grew by > 2^8

enum WaitId : int {
    kWaitQ = 11, kWaitFull = 12, kWaitEmpty = 13, kWaitS = 14,
    kWaitPO = 16, kWaitPV = 17, kWaitItem = 19, kWaitItemFree = 20,
    kWaitQFree = 21, kWaitOFree = 22
};

template <int D>
struct AttnSmem {
    static constexpr int kPanels = D / 64;
    static constexpr int kPanelBytes = kTile * 128;
    static constexpr int kTileBytes = kPanels * kPanelBytes;
    static constexpr int kQ0 = 0;
    static constexpr int kQ1 = kTileBytes;
    static constexpr int kRing0 = 2 * kTileBytes;
    static constexpr int kTotal = kRing0 + kRing * kTileBytes;
};

size_t attn_smem_bytes(int head_dim) {
    return 1024 + (head_dim == 128 ? AttnSmem<128>::kTotal : AttnSmem<64>::kTotal);
}

// One query tile.  Row r of the tile is token q_tok0 + r / row_div, head q_head0 + r % row_div; it
// exists iff r / row_div < ntok and r % row_div < nheads.  Full prefill tiles have row_div = 1; the
// ragged last tile of a segment packs the tails of several q heads of the kv group (row_div heads,
// ntok = the tail's rows); question tiles pack all G heads of the group.
struct QSlot {
    int valid;
    int q_tok0, q_head0, row_div, ntok, nheads, qmap, box_rows, limit0, b_end, nt;
};
// Key tiles of an item: first the na tiles of the shared range [0, a_end) (the sink), then the tiles of the own
// range from global key row b_start on.  The own range is fetched through the block tensor map at row
// b_coord0 of that map, or, for the sink's own items, through the sink map (own_map = 1).
struct WorkItem {
    int kv_head, a_end, b_start, na, split, b_coord0, own_map;
    QSlot s[2];
};

// Optional time stamps (-DPEVLM_TRACE): clock64 at the hand-offs of CTA 0's first work item, key tiles
// [kTraceJ0, kTraceJ0 + 16), read back through pevlm_debug_trace (see timeline.py).  Events: 0/1 scores of
// tile 0/1 seen by the softmax, 2/3 probabilities handed over, 4 QK0 issue starts, 5 QK0 issued,
// 6 probabilities of tile 0 seen by the MMA warp, 7 PV0 issued.  A second table holds, for CTA 0's work items
// [kTraceK0, kTraceK0 + 16), the events of an item boundary: 0 item taken by the MMA warp, 1 its first QK goes
// out, 2 its last PV and commits are issued; query tile 0's thread 0: 3 first scores seen, 4 last probabilities
// handed over, 5 accumulator complete, 6 accumulator released, 7 output stored.
#ifdef PEVLM_TRACE
__device__ unsigned g_trace[8][16];
__device__ unsigned g_trace_item[8][16];
constexpr int kTraceK0 = 2;
#define PEVLM_STAMP_ITEM(ev, kk, cond)                                                          \
    do {                                                                                        \
        if ((cond) && blockIdx.x == 0 && (kk) >= kTraceK0 && (kk) < kTraceK0 + 16)              \
            g_trace_item[ev][(kk) - kTraceK0] = static_cast<unsigned>(clock64());               \
    } while (0)
constexpr int kTraceJ0 = 8;
#define PEVLM_STAMP(ev, j, cond)                                                                \
    do {                                                                                        \
        if ((cond) && blockIdx.x == 0 && k == 0 && (j) >= kTraceJ0 && (j) < kTraceJ0 + 16)      \
            g_trace[ev][(j) - kTraceJ0] = static_cast<unsigned>(clock64());                     \
    } while (0)
extern "C" int pevlm_debug_trace(unsigned* host_out) {
    return cudaMemcpyFromSymbol(host_out, g_trace, sizeof(g_trace)) == cudaSuccess ? 0 : -1;
}
extern "C" int pevlm_debug_trace_items(unsigned* host_out) {
    return cudaMemcpyFromSymbol(host_out, g_trace_item, sizeof(g_trace_item)) == cudaSuccess ? 0 : -1;
}
#else
#define PEVLM_STAMP(ev, j, cond) do {} while (0)
#define PEVLM_STAMP_ITEM(ev, kk, cond) do {} while (0)
#endif

// The probabilities of a key tile are handed to the MMA warp in two parts: after the first 32 * kPvSplit keys and
// at the end of the tile, so the first PV steps run while the softmax still forms the rest (0 = one hand-off).
// Measured on B200: 2 and 3 within 1 % of each other, both 1-3 % ahead of 0.
#ifndef PEVLM_PV_SPLIT
#define PEVLM_PV_SPLIT 2
#endif
constexpr int kPvSplit = PEVLM_PV_SPLIT;

__device__ __forceinline__ int cdiv(int a, int b) { return (a + b - 1) / b; }

__device__ __forceinline__ void decode_item(const AttnParams& p, int w, WorkItem& it) {
    it.split = 0;
    if (p.mode == 0) {
        int seg_start, seg_q0, seg_len, tiles, pi, g, tail_rows, tail_heads, tail_tiles, qmap_tail;
        if (w < p.items_block) {
            // Order of the items: the pair list of a (block, kv head), heaviest first, is cut into chunks of
            // pair_chunk pairs; chunk-major, then (block, kv head), then the pairs of the chunk.  CTAs that run
            // at the same time then share few K/V tiles' worth of L2 traffic, and the launch ends on the
            // lightest chunk of every (block, kv head) rather than on the last block's whole list.  A pair
            // index past the end of the list (padding of the last chunk) is an empty item.
            const int per_chunk = p.N * p.Hkv * p.pair_chunk;
            const int r = w % per_chunk;
            const int combo = r / p.pair_chunk;
            pi = (w / per_chunk) * p.pair_chunk + r % p.pair_chunk;
            const int blk = combo / p.Hkv;
            g = combo % p.Hkv;
            seg_start = p.blk_key0 + blk * p.B;  // key rows of the block
            seg_q0 = p.blk_q0 + blk * p.B;       // its rows in q / o
            seg_len = p.B;
            tiles = p.tiles_block;
            tail_rows = p.tail_rows_block; tail_heads = p.tail_heads_block; tail_tiles = p.tail_tiles_block;
            qmap_tail = 1;
            it.a_end = p.S;
            it.b_coord0 = blk * p.B;
            it.own_map = 0;
        } else {
            const int w2 = w - p.items_block;
            g = w2 / p.pairs_sink;
            pi = w2 % p.pairs_sink;
            seg_start = 0;
            seg_q0 = 0;
            seg_len = p.S;
            tiles = p.tiles_sink;
            tail_rows = p.tail_rows_sink; tail_heads = p.tail_heads_sink; tail_tiles = p.tail_tiles_sink;
            qmap_tail = 2;
            it.a_end = 0;
            it.b_coord0 = 0;
            it.own_map = 1;
        }
        it.kv_head = g;
        it.b_start = seg_start;
        it.na = cdiv(it.a_end, kTile);
        // entries of this (segment, kv head), heaviest first: the packed tail tiles (last tile position of
        // the segment, tail_heads q heads each), then (tile position, q head) for the full positions
        const int full_tiles = tiles - (tail_tiles > 0 ? 1 : 0);
        const int entries = tail_tiles + p.G * full_tiles;
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            const int e = 2 * pi + x;
            QSlot& s = it.s[x];
            s.valid = e < entries;
            int qt;
            if (e < tail_tiles) {
                qt = tiles - 1;
                s.q_head0 = g * p.G + e * tail_heads;
                s.row_div = tail_heads;
                s.ntok = tail_rows;
                s.nheads = min(tail_heads, p.G - e * tail_heads);
                s.qmap = qmap_tail;
                s.box_rows = tail_heads * tail_rows;
            } else {
                const int e2 = e - tail_tiles;
                qt = full_tiles - 1 - e2 / p.G;
                s.q_head0 = g * p.G + e2 % p.G;
                s.row_div = 1;
                s.ntok = min(kTile, seg_len - qt * kTile);
                s.nheads = 1;
                s.qmap = 0;
                s.box_rows = kTile;
            }
            s.q_tok0 = seg_q0 + qt * kTile;
            s.limit0 = seg_start + qt * kTile;
            s.b_end = min(s.limit0 + kTile, seg_start + seg_len);
            s.nt = s.valid ? it.na + cdiv(s.b_end - it.b_start, kTile) : 0;
        }
    } else {
        it.split = w % p.n_splits;
        const int rest = w / p.n_splits;
        const int q_pairs = cdiv(p.q_tiles, 2);
        const int pi = rest % q_pairs;
        const int g = rest / q_pairs;
        it.kv_head = g;
        it.a_end = 0;
        it.na = 0;
        const int split_lo = it.split * p.tiles_per_split * kTile;
        const int split_hi = split_lo + p.tiles_per_split * kTile;
        it.b_start = split_lo;
        it.b_coord0 = split_lo;
        it.own_map = 0;
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            const int qt = 2 * pi + x;
            QSlot& s = it.s[x];
            s.valid = qt < p.q_tiles;
            const int tok0 = qt * p.tok_per_tile;
            const int ntok = max(0, min(p.tok_per_tile, p.Q - tok0));
            s.q_tok0 = tok0;
            s.q_head0 = g * p.G;
            s.row_div = p.G;
            s.ntok = ntok;
            s.nheads = p.G;
            s.qmap = 0;
            s.box_rows = p.G * p.tok_per_tile;
            s.limit0 = p.n_video + tok0;
            const int kv_end = p.n_video + tok0 + ntok;  // keys past the last row's limit are never visible
            s.b_end = min(kv_end, split_hi);
            s.nt = (s.valid && s.b_end > split_lo) ? cdiv(s.b_end - split_lo, kTile) : 0;
        }
    }
}

template <int D>
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_kernel(const __grid_constant__ AttnParams p, const __grid_constant__ CUtensorMap tmap_q,
            const __grid_constant__ CUtensorMap tmap_q_tail_block, const __grid_constant__ CUtensorMap tmap_q_tail_sink,
            const __grid_constant__ CUtensorMap tmap_k_sink, const __grid_constant__ CUtensorMap tmap_v_sink,
            const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v) {
    using L = AttnSmem<D>;
    constexpr int NP = L::kPanels;
    extern __shared__ uint8_t smem_raw[];
    // barrier map (uint64 each): [0,2) item_full [2,4) item_free [4,6) q_full [6,8) q_free
    // [8,12) ring full [12,16) ring empty, then per slot x: [16,18) s_full [18,20) po
    // [24,26) o_free [26,28) o_done
    __shared__ uint64_t bars[30];  // [28,30) po_a: first part of a tile's probabilities written
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ int s_item[2];
    __shared__ WorkItem s_decoded[2];  // the producer decodes an item once; every role copies it from here

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bar0 = smem_u32(&bars[0]);
    const uint32_t bar_item_full = bar0, bar_item_free = bar0 + 16, bar_q_full = bar0 + 32, bar_q_free = bar0 + 48;
    const uint32_t bar_full = bar0 + 64, bar_empty = bar0 + 96;
    const uint32_t bar_s_full = bar0 + 128, bar_po = bar0 + 144;
    const uint32_t bar_o_free = bar0 + 192, bar_o_done = bar0 + 208, bar_po_a = bar0 + 224;
    constexpr int kItemConsumers = 1 + 2 * kTile;  // MMA warp + two softmax warpgroups

    if (tid == 0) {
        abort_flag = 0;
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar_item_full + 8 * i, 1);
            mbar_init(bar_item_free + 8 * i, kItemConsumers);
            mbar_init(bar_q_full + 8 * i, 1);
            mbar_init(bar_q_free + 8 * i, 1);
            mbar_init(bar_s_full + 8 * i, 1);
            mbar_init(bar_po + 8 * i, kTile);
            mbar_init(bar_po_a + 8 * i, kTile);
            mbar_init(bar_o_free + 8 * i, kTile);
            mbar_init(bar_o_done + 8 * i, 1);
        }
        for (int i = 0; i < kRing; ++i) {
            mbar_init(bar_full + 8 * i, 1);
            mbar_init(bar_empty + 8 * i, 1);
        }
        fence_mbar_init();
        tma_prefetch_desc(&tmap_q);
        tma_prefetch_desc(&tmap_q_tail_block);
        tma_prefetch_desc(&tmap_q_tail_sink);
        tma_prefetch_desc(&tmap_k_sink);
        tma_prefetch_desc(&tmap_v_sink);
        tma_prefetch_desc(&tmap_k);
        tma_prefetch_desc(&tmap_v);
    }
    if (warp == 8) {
        __syncwarp();
        tmem_alloc(smem_u32(&tmem_base_slot), 512);
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_base_slot;

    auto give_up = [&](int which) {
        if (atomicCAS(&p.hdr->status, 0, PEVLM_ETIMEOUT) == 0) p.hdr->detail = which * 1000000 + blockIdx.x;
    };
    auto wait = [&](uint32_t bar, uint32_t parity, int which) {
        if (!mbar_wait(bar, parity, &abort_flag, p.wait_limit_ns)) give_up(which);
    };
    // consumer side of the item queue: k-th item of this CTA, -1 = no more work
    auto next_item = [&](int k, WorkItem& it) {
        wait(bar_item_full + 8 * (k & 1), (k >> 1) & 1, kWaitItem);
        const int w = s_item[k & 1];
        if (w >= 0) it = s_decoded[k & 1];
        mbar_arrive(bar_item_free + 8 * (k & 1));
        return w;
    };

    // register budget per warpgroup: 2 x 216 (softmax + epilogue) + 56 (TMA/MMA) <= 384 x 168
    if (warp >= 8) {
        reg_dealloc<56>();
      if (warp == 9) {
        // ------------------------------------------------------------- scheduler + TMA producer
        if (lane == 0) {
            int ring_idx = 0;          // K/V tiles loaded so far (ring position), runs on across items
            int q_loads[2] = {0, 0};   // Q loads per slot so far
            for (int k = 0;; ++k) {
                int w = (k == 0) ? static_cast<int>(blockIdx.x)
                                 : static_cast<int>(gridDim.x) + atomicAdd(&p.hdr->work_counter, 1);
                if (w >= p.n_items || abort_flag != 0 || *reinterpret_cast<volatile int32_t*>(&p.hdr->status) != 0) w = -1;
                if (k >= 2) wait(bar_item_free + 8 * (k & 1), ((k >> 1) - 1) & 1, kWaitItemFree);
                s_item[k & 1] = w;
                WorkItem it;
                if (w >= 0) {
                    decode_item(p, w, it);
                    s_decoded[k & 1] = it;
                }
                mbar_arrive(bar_item_full + 8 * (k & 1));  // release: the item and its decoded form are visible
                if (w < 0) break;
                const int nt_max = max(it.s[0].nt, it.s[1].nt);
#pragma unroll
                for (int x = 0; x < 2; ++x) {
                    if (it.s[x].nt == 0) continue;
                    if (q_loads[x] > 0) wait(bar_q_free + 8 * x, (q_loads[x] - 1) & 1, kWaitQFree);
                    mbar_arrive_expect_tx(bar_q_full + 8 * x, static_cast<uint32_t>(NP * it.s[x].box_rows * 128));
                    const CUtensorMap* qmap = it.s[x].qmap == 0 ? &tmap_q : it.s[x].qmap == 1 ? &tmap_q_tail_block : &tmap_q_tail_sink;
                    for (int h = 0; h < NP; ++h)
                        tma_load_3d(smem_base + (x ? L::kQ1 : L::kQ0) + h * L::kPanelBytes, qmap, h * 64,
                                    it.s[x].q_head0, it.s[x].q_tok0, bar_q_full + 8 * x);
                    ++q_loads[x];
                }
                for (int j = 0; j < nt_max; ++j) {
                    // Rows past the end of the sink, and past the end of the block range, are outside their
                    // tensor map and arrive as zeros: a ragged last tile never brings in a neighbour's rows.
                    const bool shared_range = j < it.na || it.own_map != 0;
                    const int j0 = j < it.na ? j * kTile : it.b_coord0 + (j - it.na) * kTile;
#pragma unroll
                    for (int kv = 0; kv < 2; ++kv) {
                        const int slot = ring_idx % kRing, use = ring_idx / kRing;
                        if (use > 0) wait(bar_empty + 8 * slot, (use - 1) & 1, kWaitEmpty);
                        mbar_arrive_expect_tx(bar_full + 8 * slot, L::kTileBytes);
                        for (int h = 0; h < NP; ++h)
                            tma_load_3d(smem_base + L::kRing0 + slot * L::kTileBytes + h * L::kPanelBytes,
                                        shared_range ? (kv ? &tmap_v_sink : &tmap_k_sink) : (kv ? &tmap_v : &tmap_k),
                                        h * 64, it.kv_head, j0, bar_full + 8 * slot);
                        ++ring_idx;
                    }
                }
            }
        }
      } else if (warp == 8) {
        // ------------------------------------------------------------- MMA issuer
        // All 32 lanes run this loop with warp-uniform values (descriptors and addresses stay in
        // uniform registers); the MMA and commit instructions themselves go out from one elected lane.
        int ring_base = 0;        // ring position of this item's K(0)
        int cnt[2] = {0, 0};      // tiles per slot before this item (phase of s_full / po)
        int q_uses[2] = {0, 0};   // items in which the slot was active so far
        for (int k = 0;; ++k) {
            // every lane reads the item, one lane releases the queue slot
            wait(bar_item_full + 8 * (k & 1), (k >> 1) & 1, kWaitItem);
            const int w = s_item[k & 1];
            WorkItem it;
            if (w >= 0) it = s_decoded[k & 1];
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_item_free + 8 * (k & 1));
            if (w < 0) break;
            PEVLM_STAMP_ITEM(0, k, lane == 0);
            const int nt[2] = {it.s[0].nt, it.s[1].nt};
            const int nt_max = max(nt[0], nt[1]);
            // keys in the last tile of the shared range and of each slot's own range (every other
            // tile is full)
            const int na = it.na;
            const int a_last = it.a_end - (na - 1) * kTile;
            const int b_last[2] = {it.s[0].b_end - it.b_start - (nt[0] - na - 1) * kTile,
                                   it.s[1].b_end - it.b_start - (nt[1] - na - 1) * kTile};
            auto valid_of = [&](int x, int j) { return (j == na - 1) ? a_last : (j == nt[x] - 1) ? b_last[x] : kTile; };
            auto ring_addr = [&](int idx) { return smem_base + L::kRing0 + ((ring_base + idx) % kRing) * L::kTileBytes; };
            auto wait_full = [&](int idx) {
                const int g = ring_base + idx;
                wait(bar_full + 8 * (g % kRing), (g / kRing) & 1, kWaitFull);
            };
            auto commit_empty = [&](int idx) { mma_commit_elect(bar_empty + 8 * ((ring_base + idx) % kRing)); };
            // S_x = Q_x K(j)^T
            auto issue_qk = [&](int x, int j) {
                PEVLM_STAMP(4, j, lane == 0 && x == 0);
                const int n_mma = (valid_of(x, j) + 15) & ~15;
                const uint32_t idesc = make_idesc_bf16(kTile, n_mma, false);
                mma_ss_batch<D / 16>(tmem_base + x * 128, desc_lo(smem_base + (x ? L::kQ1 : L::kQ0), 16),
                                     desc_lo(ring_addr(2 * j), 16), idesc);
                PEVLM_STAMP(5, j, lane == 0 && x == 0);
                mma_commit_elect(bar_s_full + 8 * x);
                if (j == nt[x] - 1) mma_commit_elect(bar_q_free + 8 * x);  // last use of this Q tile
            };
            // O_x += P_x V(j)
            auto issue_pv = [&](int x, int j) {
                wait((kPvSplit > 0 ? bar_po_a : bar_po) + 8 * x, (cnt[x] + j) & 1, kWaitPO);
                PEVLM_STAMP(6, j, lane == 0 && x == 0);
                // the previous item's output must have left TMEM before O is overwritten
                if (j == 0 && q_uses[x] > 0) wait(bar_o_free + 8 * x, (q_uses[x] - 1) & 1, kWaitOFree);
                tc_fence_after_sync();
                const int nvalid = valid_of(x, j);
                const uint32_t idesc = make_idesc_bf16(kTile, D, true);
                const uint32_t sv = ring_addr(2 * j + 1);
                const uint32_t d_tmem = tmem_base + 256 + x * 128, a_tmem = tmem_base + x * 128;
                if (kPvSplit > 0) {
                    // first part (the wait above was for it), then the wait for the rest of the tile
                    const uint32_t b_lo = desc_lo(sv, L::kPanelBytes);
                    const int ksteps = (nvalid + 15) >> 4;
                    constexpr int kFirst = 2 * kPvSplit;
                    if (nvalid == kTile) {
                        if (kPvSplit == 1) mma_ts_batch2(d_tmem, a_tmem, b_lo, idesc, j > 0);
                        if (kPvSplit >= 2) mma_ts_batch4(d_tmem, a_tmem, b_lo, idesc, j > 0);
                        if (kPvSplit == 3) mma_ts_batch2(d_tmem, a_tmem + 32, b_lo + 512, idesc, 1);
                    } else {
                        for (int ks = 0; ks < min(ksteps, kFirst); ++ks)
                            mma_ts_elect(d_tmem, a_tmem + ks * 8, make_smem_desc_sw128(sv + ks * 2048, L::kPanelBytes, 1024), idesc,
                                         (j > 0) || (ks > 0));
                    }
                    wait(bar_po + 8 * x, (cnt[x] + j) & 1, kWaitPO);
                    tc_fence_after_sync();
                    if (nvalid == kTile) {
                        if (kPvSplit == 1) mma_ts_batch2(d_tmem, a_tmem + 16, b_lo + 256, idesc, 1);
                        if (kPvSplit <= 2) mma_ts_batch4(d_tmem, a_tmem + 32, b_lo + 512, idesc, 1);
                        if (kPvSplit == 3) mma_ts_batch2(d_tmem, a_tmem + 48, b_lo + 768, idesc, 1);
                    } else {
                        for (int ks = kFirst; ks < ksteps; ++ks)
                            mma_ts_elect(d_tmem, a_tmem + ks * 8, make_smem_desc_sw128(sv + ks * 2048, L::kPanelBytes, 1024), idesc, 1);
                    }
                } else if (nvalid == kTile) {
                    mma_ts_batch8(d_tmem, a_tmem, desc_lo(sv, L::kPanelBytes), idesc, j > 0);
                } else {
                    const int ksteps = (nvalid + 15) >> 4;
                    for (int ks = 0; ks < ksteps; ++ks)
                        mma_ts_elect(d_tmem, a_tmem + ks * 8, make_smem_desc_sw128(sv + ks * 2048, L::kPanelBytes, 1024), idesc,
                                     (j > 0) || (ks > 0));
                }
                PEVLM_STAMP(7, j, lane == 0 && x == 0);
                // o_done: the item's accumulator is complete (one phase per item, for the epilogue)
                if (j == nt[x] - 1) mma_commit_elect(bar_o_done + 8 * x);
            };
#pragma unroll
            for (int x = 0; x < 2; ++x)
                if (nt[x] > 0) wait(bar_q_full + 8 * x, q_uses[x] & 1, kWaitQ);
            tc_fence_after_sync();
            // Order on the tensor pipe: QK0(0) QK1(0), then per key tile j: PV0(j) QK0(j+1) PV1(j) QK1(j+1).
            // While one query tile is in its softmax the other one's MMAs run.  PV_x(j) and QK_x(j+1) go out
            // back to back: everything they wait for except the probabilities (V(j), K(j+1)) is waited for
            // before the wait on P_x(j), so the scores of the next tile follow the probabilities of this one
            // through the pipe without a gap.
            if (nt_max > 0) {
                wait_full(0);
                PEVLM_STAMP_ITEM(1, k, lane == 0);
                if (nt[0] > 0) issue_qk(0, 0);
                if (nt[1] > 0) issue_qk(1, 0);
                commit_empty(0);  // K(0) consumed
            }
            for (int j = 0; j < nt_max; ++j) {
                const bool more = j + 1 < nt_max;
                wait_full(2 * j + 1);             // V(j)
                if (more) wait_full(2 * j + 2);   // K(j+1)
                if (j < nt[0]) {
                    issue_pv(0, j);
                    if (j + 1 < nt[0]) issue_qk(0, j + 1);
                }
                if (j < nt[1]) {
                    issue_pv(1, j);
                    if (j + 1 < nt[1]) issue_qk(1, j + 1);
                }
                commit_empty(2 * j + 1);            // V(j) consumed
                if (more) commit_empty(2 * j + 2);  // K(j+1) consumed
            }
            PEVLM_STAMP_ITEM(2, k, lane == 0);
            ring_base += 2 * nt_max;
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                cnt[x] += nt[x];
                if (nt[x] > 0) ++q_uses[x];
            }
        }
      }
    } else {
        // ------------------------------------------------------------- softmax and epilogue of slot x
        reg_alloc<216>();
        const int x = warp >> 2;
        const int row = tid & 127;
        const uint32_t lane_off = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tS = tmem_base + x * 128 + lane_off;
        const uint32_t tO = tmem_base + 256 + x * 128 + lane_off;
        const uint32_t my_s_full = bar_s_full + 8 * x, my_po = bar_po + 8 * x;
        int cnt = 0;        // tiles of this slot processed so far (phase of s_full)
        int uses = 0;       // items in which this slot was active so far
        int ring_base = 0;  // ring position of this item's K(0)
        for (int k = 0;; ++k) {
            WorkItem it;
            const int w = next_item(k, it);
            if (w < 0) break;
            // this slot's scalars, in registers
            const int nt = x ? it.s[1].nt : it.s[0].nt;
            const int item_ring_base = ring_base;
            ring_base += 2 * max(it.s[0].nt, it.s[1].nt);
            const QSlot& qs = x ? it.s[1] : it.s[0];
            if (!qs.valid) continue;
            // this thread's row of the query tile
            // (row_div is 1 for all but packed tiles: no integer division on the way to the item's first scores)
            const int row_tok = qs.row_div == 1 ? row : row / qs.row_div;
            const int row_head = qs.row_div == 1 ? 0 : row - row_tok * qs.row_div;
            const bool row_ok = (row_tok < qs.ntok) && (row_head < qs.nheads);
            const int tok = qs.q_tok0 + row_tok;
            const int head = qs.q_head0 + row_head;
            if (nt == 0) {
                // question-mode tile with no visible key in this CTA's key range: neutral partial
                if (p.mode == 1 && row_ok) {
                    const size_t r = (static_cast<size_t>(it.split) * p.Q + tok) * p.Hq + head;
                    p.part_lse[r] = -INFINITY;
                    float4* dst = reinterpret_cast<float4*>(p.part_o + r * D);
                    for (int c = 0; c < D / 4; ++c) dst[c] = make_float4(0.f, 0.f, 0.f, 0.f);
                }
                continue;
            }
            const int limit0 = x ? it.s[1].limit0 : it.s[0].limit0;
            const int b_end = x ? it.s[1].b_end : it.s[0].b_end;
            const int na = it.na, a_end = it.a_end, b_start = it.b_start;
            const int my_limit = limit0 + row_tok;
            float m_ref = -INFINITY;  // reference maximum (raw score units) the probabilities are scaled by
            float l_run = 0.f;
            for (int j = 0; j < nt; ++j, ++cnt) {
                const int j0 = j < na ? j * kTile : b_start + (j - na) * kTile;
                const int nvalid = min(kTile, (j < na ? a_end : b_end) - j0);
                const bool need_mask = (nvalid < kTile) || (j0 + kTile - 1 > limit0);
                wait(my_s_full, cnt & 1, kWaitS);
                PEVLM_STAMP(0 + x, j, (tid & 127) == 0);
                PEVLM_STAMP_ITEM(3, k, tid == 0 && j == 0);
                tc_fence_after_sync();
                // all 128 scores of the row in registers: one round trip to TMEM
                uint32_t r[kTile];
#pragma unroll
                for (int c = 0; c < 4; ++c) tmem_ld32(tS + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&r[32 * c]));
                tmem_wait_ld();
                if (need_mask) {
                    const int max_col = min(nvalid, my_limit - j0 + 1);
#pragma unroll
                    for (int i = 0; i < kTile; ++i)
                        if (i >= max_col) r[i] = 0xff800000u;  // -inf
                }
                float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                for (int i = 0; i < kTile; i += 8) {
#pragma unroll
                    for (int a = 0; a < 4; ++a)
                        mx[a] = fmax3(mx[a], __uint_as_float(r[i + 2 * a]), __uint_as_float(r[i + 2 * a + 1]));
                }
                const float m_tile = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
                float alpha = 1.f;
                if ((m_tile - m_ref) * p.scale_log2 > kRescaleThresholdLog2 || m_ref == -INFINITY) {
                    const float m_new = fmaxf(m_ref, m_tile);
                    alpha = (m_new == -INFINITY) ? 1.f : fast_exp2((m_ref - m_new) * p.scale_log2);
                    m_ref = m_new;
                }
                if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
                    // rare: rescale this row of the O accumulator in place, once PV(j-1) has landed: the
                    // ring slot of V(j-1) is released by a commit issued after both slots' PV(j-1).
                    // (S(j) is complete, so that slot's previous release, two tiles back, is too.)
                    const int gv = item_ring_base + 2 * (j - 1) + 1;
                    wait(bar_empty + 8 * (gv % kRing), (gv / kRing) & 1, kWaitPV);
                    tc_fence_after_sync();
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t o[32];
                        tmem_ld32(tO + c * 32, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                        tmem_st32(tO + c * 32, o);
                    }
                }
                const float neg_ms = (m_ref == -INFINITY) ? 0.f : -m_ref * p.scale_log2;
                // probabilities, written over the scores as bf16 pairs (columns [0, 64) of the slot);
                // scale-and-shift and the row sum run as packed fp32 pairs
                const uint64_t scale2 = pack_f32x2(p.scale_log2, p.scale_log2);
                const uint64_t shift2 = pack_f32x2(neg_ms, neg_ms);
                uint64_t sm2[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const uint64_t t2 = fma_f32x2(pack_f32x2(__uint_as_float(r[c * 32 + 2 * i]),
                                                                 __uint_as_float(r[c * 32 + 2 * i + 1])), scale2, shift2);
                        float t0, t1;
                        unpack_f32x2(t2, t0, t1);
                        const float p0 = fast_exp2(t0), p1 = fast_exp2(t1);
                        sm2[i & 3] = add_f32x2(sm2[i & 3], pack_f32x2(p0, p1));
                        pk[i] = pack_bf16x2(p0, p1);
                    }
                    tmem_st16(tS + c * 16, pk);
                    if (kPvSplit > 0 && c == kPvSplit - 1) {  // first part of the probabilities is in TMEM
                        tmem_wait_st();
                        tc_fence_before_sync();
                        mbar_arrive(bar_po_a + 8 * x);
                    }
                }
                float sum;
                {
                    float a0, a1, b0, b1;
                    unpack_f32x2(add_f32x2(sm2[0], sm2[1]), a0, a1);
                    unpack_f32x2(add_f32x2(sm2[2], sm2[3]), b0, b1);
                    sum = (a0 + a1) + (b0 + b1);
                }
                tmem_wait_st();
                tc_fence_before_sync();
                mbar_arrive(my_po);
                PEVLM_STAMP(2 + x, j, (tid & 127) == 0);
                PEVLM_STAMP_ITEM(4, k, tid == 0 && j == nt - 1);
                l_run = l_run * alpha + sum;
            }
            // Epilogue, by the same thread (its registers are free now and it would only wait for the next
            // item's scores): once the last PV has landed, the whole accumulator row goes to registers in one
            // round trip and the accumulator is released for the next item; normalisation, conversion and the
            // stores follow while the next item's first QK is already in the tensor pipe.
            wait(bar_o_done + 8 * x, uses & 1, kWaitPV);
            PEVLM_STAMP_ITEM(5, k, tid == 0);
            tc_fence_after_sync();
            {
                uint32_t o[D];
#pragma unroll
                for (int c = 0; c < D / 32; ++c) tmem_ld32(tO + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&o[32 * c]));
                tmem_wait_ld();
                tc_fence_before_sync();
                mbar_arrive(bar_o_free + 8 * x);
                PEVLM_STAMP_ITEM(6, k, tid == 0);
                const float inv_l = (l_run > 0.f) ? 1.f / l_run : 0.f;
                const float lse_val = (l_run > 0.f) ? m_ref * p.scale + logf(l_run) : -INFINITY;
                if (row_ok) {
                    if (p.mode == 0) {
                        // 32 bytes per store: every lane writes whole sectors of its own row
                        __nv_bfloat16* dst = p.o + (static_cast<size_t>(tok) * p.Hq + head) * D;
#pragma unroll
                        for (int v = 0; v < D / 16; ++v) {
                            uint32_t wd[8];
#pragma unroll
                            for (int e = 0; e < 8; ++e)
                                wd[e] = pack_bf16x2(__uint_as_float(o[v * 16 + 2 * e]) * inv_l,
                                                    __uint_as_float(o[v * 16 + 2 * e + 1]) * inv_l);
                            st_global_v8(dst + v * 16, wd);
                        }
                        if (p.lse) st_global_stream_f32(p.lse + static_cast<size_t>(head) * p.q_rows + tok, lse_val);
                    } else {
                        const size_t r = (static_cast<size_t>(it.split) * p.Q + tok) * p.Hq + head;
                        float* dst = p.part_o + r * D;
#pragma unroll
                        for (int v = 0; v < D / 8; ++v) {
                            uint32_t wd[8];
#pragma unroll
                            for (int e = 0; e < 8; ++e) wd[e] = __float_as_uint(__uint_as_float(o[v * 8 + e]) * inv_l);
                            st_global_v8(dst + v * 8, wd);
                        }
                        st_global_stream_f32(p.part_lse + r, lse_val);
                    }
                }
            }
            PEVLM_STAMP_ITEM(7, k, tid == 0);
            ++uses;
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 8) {
        __syncwarp();
        tmem_dealloc(tmem_base, 512);
    }
}

cudaError_t launch_attn(const AttnParams& p, int head_dim, const AttnMaps& m, cudaStream_t stream) {
    if (p.n_items <= 0) return cudaSuccess;
    const size_t smem = attn_smem_bytes(head_dim);
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const int grid = p.n_items < sms ? p.n_items : sms;  // persistent: one CTA per SM
    if (head_dim == 128) {
        e = cudaFuncSetAttribute(attn_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e != cudaSuccess) return e;
        attn_kernel<128><<<grid, kAttnThreads, smem, stream>>>(p, m.q, m.q_tail_block, m.q_tail_sink, m.k_sink, m.v_sink, m.k, m.v);
    } else {
        e = cudaFuncSetAttribute(attn_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e != cudaSuccess) return e;
        attn_kernel<64><<<grid, kAttnThreads, smem, stream>>>(p, m.q, m.q_tail_block, m.q_tail_sink, m.k_sink, m.v_sink, m.k, m.v);
    }
    return cudaGetLastError();
}

}  // namespace pevlm
