// Block-masked flash attention for sm_100a (Eq. 1 under the masks of Eq. 3-5).
//
// One CTA computes one query tile of 128 rows against the key tiles that tile can see:
//   prefill rows of context block i : the sink's tiles, then block i's tiles up to the diagonal
//   sink rows / full-causal rows    : tiles up to the diagonal
//   question rows (split over keys) : a contiguous slice of the cache's tiles
// Key/value tiles arrive by TMA (128-byte swizzle) into a two-stage ring; S = Q K^T and
// O += P V run on the tensor cores (tcgen05.mma, accumulators in TMEM, P fed back from TMEM
// as the A operand); the online softmax runs in fp32 with one thread per query row.
#include "internal.h"
#include "ptx.cuh"

namespace pevlm {

constexpr int kAttnThreads = 128;
constexpr int kStages = 2;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kTmemS = 0;    // 128 fp32 columns: scores
constexpr uint32_t kTmemP = 128;  // 64 columns: probabilities, two bf16 per column
constexpr uint32_t kTmemO = 256;  // d fp32 columns: output accumulator

// wait identifiers recorded in the workspace header when a bounded wait expires
enum WaitId : int { kWaitQ = 1, kWaitK = 2, kWaitV = 3, kWaitS = 4, kWaitO = 5 };

template <int D>
struct SmemLayout {
    static constexpr int kHalves = D / 64;                 // 64-element (128-byte) column panels
    static constexpr int kPanelBytes = kTile * 128;        // 128 rows x 128 bytes
    static constexpr int kTileBytes = kHalves * kPanelBytes;
    static constexpr int kQ = 0;
    static constexpr int kK = kTileBytes;
    static constexpr int kV = kK + kStages * kTileBytes;
    static constexpr int kTotal = kV + kStages * kTileBytes;
};

size_t attn_smem_bytes(int head_dim) {
    return 1024 + (head_dim == 128 ? SmemLayout<128>::kTotal : SmemLayout<64>::kTotal);
}

struct Item {
    int q_tok0;      // first token of the query tile (row of the q tensor)
    int q_head0;     // first head of the TMA box
    int kv_head;
    int rows_valid;  // rows of the tile that exist
    int row_div;     // rows per token (1 prefill, G question)
    int limit0;      // key index visible limit of row r: limit0 + r / row_div (inclusive)
    int a_start, a_end;  // first key range  [a_start, a_end)
    int b_start, b_end;  // second key range [b_start, b_end)
    int split;       // question mode
};

__device__ __forceinline__ int ceil_div(int a, int b) { return (a + b - 1) / b; }

__device__ __forceinline__ Item decode_item(const AttnParams& p, int w) {
    Item it;
    it.split = 0;
    if (p.mode == 0) {
        it.row_div = 1;
        if (w < p.items_block) {
            // context-block rows, heaviest query tiles (largest index in the block) first
            const int per_qt = p.N * p.Hq;
            const int qt = p.tiles_block - 1 - w / per_qt;
            const int rem = w % per_qt;
            const int blk = rem / p.Hq;
            const int h = rem % p.Hq;
            const int blk_start = p.S + blk * p.B;
            it.q_tok0 = blk_start + qt * kTile;
            it.q_head0 = h;
            it.kv_head = h / p.G;
            it.rows_valid = min(kTile, p.B - qt * kTile);
            it.limit0 = it.q_tok0;
            it.a_start = 0;
            it.a_end = p.S;
            it.b_start = blk_start;
            it.b_end = min(it.q_tok0 + kTile, blk_start + p.B);
        } else {
            const int w2 = w - p.items_block;
            const int qt = p.tiles_sink - 1 - w2 / p.Hq;
            const int h = w2 % p.Hq;
            it.q_tok0 = qt * kTile;
            it.q_head0 = h;
            it.kv_head = h / p.G;
            it.rows_valid = min(kTile, p.S - qt * kTile);
            it.limit0 = it.q_tok0;
            it.a_start = 0;
            it.a_end = 0;
            it.b_start = 0;
            it.b_end = min(it.q_tok0 + kTile, p.S);
        }
    } else {
        it.split = w % p.n_splits;
        const int rest = w / p.n_splits;
        const int qt = rest % p.q_tiles;
        const int g = rest / p.q_tiles;
        const int tok0 = qt * p.tok_per_tile;
        const int ntok = min(p.tok_per_tile, p.Q - tok0);
        it.q_tok0 = tok0;
        it.q_head0 = g * p.G;
        it.kv_head = g;
        it.rows_valid = ntok * p.G;
        it.row_div = p.G;
        it.limit0 = p.n_video + tok0;
        const int kv_end = p.n_video + tok0 + ntok;  // keys beyond the last row's limit are never visible
        it.a_start = 0;
        it.a_end = 0;
        it.b_start = min(kv_end, it.split * p.tiles_per_split * kTile);
        it.b_end = min(kv_end, (it.split + 1) * p.tiles_per_split * kTile);
    }
    return it;
}

template <int D>
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_kernel(const __grid_constant__ AttnParams p, const __grid_constant__ CUtensorMap tmap_q,
            const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v) {
    using L = SmemLayout<D>;
    constexpr int NH = L::kHalves;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[3 + 2 * kStages];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base + L::kQ;
    const uint32_t sK = smem_base + L::kK;
    const uint32_t sV = smem_base + L::kV;
    const uint32_t bar_q = smem_u32(&bars[0]);
    const uint32_t bar_s = smem_u32(&bars[1]);
    const uint32_t bar_o = smem_u32(&bars[2]);
    const uint32_t bar_k0 = smem_u32(&bars[3]);
    const uint32_t bar_v0 = smem_u32(&bars[3 + kStages]);

    // an earlier CTA of this launch gave up on a wait: do no work (decided once per CTA)
    if (tid == 0) abort_flag = p.hdr->status;
    __syncthreads();
    if (abort_flag != 0) return;

    const Item it = decode_item(p, blockIdx.x);
    const int na = ceil_div(it.a_end - it.a_start, kTile);
    const int nb = ceil_div(it.b_end - it.b_start, kTile);
    const int nt = na + nb;

    if (nt == 0) {
        // question-mode split with no visible key: neutral partial (weight 0 in the merge)
        if (p.mode == 1 && tid < it.rows_valid) {
            const int tok = it.q_tok0 + tid / it.row_div;
            const int head = it.q_head0 + tid % it.row_div;
            const size_t row = (static_cast<size_t>(it.split) * p.Q + tok) * p.Hq + head;
            p.part_lse[row] = -INFINITY;
            float4* dst = reinterpret_cast<float4*>(p.part_o + row * D);
            for (int c = 0; c < D / 4; ++c) dst[c] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        return;
    }

    if (tid == 0) {
        for (int i = 0; i < 3 + 2 * kStages; ++i) mbar_init(smem_u32(&bars[i]), 1);
        fence_mbar_init();
        tma_prefetch_desc(&tmap_q);
        tma_prefetch_desc(&tmap_k);
        tma_prefetch_desc(&tmap_v);
    }
    if (warp == 0) {
        __syncwarp();
        tmem_alloc(smem_u32(&tmem_base_slot), kTmemCols);
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_base_slot;
    const uint32_t lane_off = static_cast<uint32_t>(warp * 32) << 16;
    const uint32_t tS = tmem_base + kTmemS, tP = tmem_base + kTmemP, tO = tmem_base + kTmemO;

    auto tile_start = [&](int i) { return i < na ? it.a_start + i * kTile : it.b_start + (i - na) * kTile; };
    auto tile_valid = [&](int i) {
        return i < na ? min(kTile, it.a_end - (it.a_start + i * kTile)) : min(kTile, it.b_end - (it.b_start + (i - na) * kTile));
    };
    auto issue_kv_loads = [&](int i) {
        const int s = i % kStages;
        const int j0 = tile_start(i);
        mbar_arrive_expect_tx(bar_k0 + 8 * s, L::kTileBytes);
        for (int h = 0; h < NH; ++h)
            tma_load_3d(sK + s * L::kTileBytes + h * L::kPanelBytes, &tmap_k, h * 64, it.kv_head, j0, bar_k0 + 8 * s);
        mbar_arrive_expect_tx(bar_v0 + 8 * s, L::kTileBytes);
        for (int h = 0; h < NH; ++h)
            tma_load_3d(sV + s * L::kTileBytes + h * L::kPanelBytes, &tmap_v, h * 64, it.kv_head, j0, bar_v0 + 8 * s);
    };
    auto issue_qk = [&](int i) {
        const int s = i % kStages;
        const int n_mma = (tile_valid(i) + 15) & ~15;
        const uint32_t idesc = make_idesc_bf16(kTile, n_mma, false);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
            const uint32_t off = (ks / 4) * L::kPanelBytes + (ks % 4) * 32;
            const uint64_t a = make_smem_desc_sw128(sQ + off, 16, 1024);
            const uint64_t b = make_smem_desc_sw128(sK + s * L::kTileBytes + off, 16, 1024);
            mma_ss(tS, a, b, idesc, ks > 0);
        }
        mma_commit(bar_s);
    };
    auto issue_pv = [&](int i) {
        const int s = i % kStages;
        const int ksteps = (tile_valid(i) + 15) >> 4;
        const uint32_t idesc = make_idesc_bf16(kTile, D, true);
        for (int ks = 0; ks < ksteps; ++ks) {
            // V tile is [key][d] with d contiguous: MN-major B operand; 16 keys = 2048 bytes
            const uint64_t b = make_smem_desc_sw128(sV + s * L::kTileBytes + ks * 2048, L::kPanelBytes, 1024);
            mma_ts(tO, tP + ks * 8, b, idesc, (i > 0) || (ks > 0));
        }
        mma_commit(bar_o);
    };
    auto give_up = [&](int which) {
        if (atomicCAS(&p.hdr->status, 0, PEVLM_ETIMEOUT) == 0) p.hdr->detail = which * 1000000 + blockIdx.x;
    };

    if (tid == 0) {
        mbar_arrive_expect_tx(bar_q, static_cast<uint32_t>(NH * p.q_box_rows * 128));
        for (int h = 0; h < NH; ++h)
            tma_load_3d(sQ + h * L::kPanelBytes, &tmap_q, h * 64, it.q_head0, it.q_tok0, bar_q);
        issue_kv_loads(0);
        if (nt > 1) issue_kv_loads(1);
    }
    if (!mbar_wait(bar_q, 0, &abort_flag)) give_up(kWaitQ);
    if (!mbar_wait(bar_k0, 0, &abort_flag)) give_up(kWaitK);
    tc_fence_after_sync();
    if (tid == 0) issue_qk(0);

    const int my_limit = it.limit0 + tid / it.row_div;
    float m_run = -INFINITY;  // running maximum of the raw scores
    float l_run = 0.f;        // running sum of exp2((s - m) * scale_log2)

    for (int i = 0; i < nt; ++i) {
        const int s = i % kStages;
        const int j0 = tile_start(i);
        const int nvalid = tile_valid(i);
        const bool need_mask = (nvalid < kTile) || (j0 + kTile - 1 > it.limit0);

        if (!mbar_wait(bar_s, i & 1, &abort_flag)) give_up(kWaitS);
        tc_fence_after_sync();

        uint32_t sr[4][32];
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_ld32(tS + lane_off + c * 32, sr[c]);
        tmem_wait_ld();

        float m_tile = -INFINITY;
        if (need_mask) {
            const int max_col = min(nvalid, my_limit - j0 + 1);  // columns [0, max_col) are visible
#pragma unroll
            for (int c = 0; c < 4; ++c)
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const float v = (c * 32 + j < max_col) ? __uint_as_float(sr[c][j]) : -INFINITY;
                    sr[c][j] = __float_as_uint(v);
                    m_tile = fmaxf(m_tile, v);
                }
        } else {
#pragma unroll
            for (int c = 0; c < 4; ++c)
#pragma unroll
                for (int j = 0; j < 32; ++j) m_tile = fmaxf(m_tile, __uint_as_float(sr[c][j]));
        }
        const float m_new = fmaxf(m_run, m_tile);
        const float m_safe = (m_new == -INFINITY) ? 0.f : m_new;
        const float alpha = fast_exp2((m_run - m_safe) * p.scale_log2);  // m_run = -inf -> 0
        const float neg_ms = -m_safe * p.scale_log2;

        uint32_t pk[64];
        float sum = 0.f;
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const float p0 = fast_exp2(fmaf(__uint_as_float(sr[c][2 * j]), p.scale_log2, neg_ms));
                const float p1 = fast_exp2(fmaf(__uint_as_float(sr[c][2 * j + 1]), p.scale_log2, neg_ms));
                sum += p0 + p1;
                pk[c * 16 + j] = pack_bf16x2(p0, p1);
            }
        l_run = l_run * alpha + sum;
        m_run = m_new;

        if (i > 0) {
            // PV(i-1) must be complete before O is rescaled, P overwritten, or its stage refilled
            if (!mbar_wait(bar_o, (i - 1) & 1, &abort_flag)) give_up(kWaitO);
            tc_fence_after_sync();
            if (tid == 0 && i + 1 < nt) issue_kv_loads(i + 1);
            if (__any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t orow[32];
                    tmem_ld32(tO + lane_off + c * 32, orow);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j) orow[j] = __float_as_uint(__uint_as_float(orow[j]) * alpha);
                    tmem_st32(tO + lane_off + c * 32, orow);
                }
            }
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_st16(tP + lane_off + c * 16, pk + c * 16);
        tmem_wait_st();
        tc_fence_before_sync();
        __syncthreads();
        if (tid == 0) {
            tc_fence_after_sync();
            if (!mbar_wait(bar_v0 + 8 * s, (i / kStages) & 1, &abort_flag)) give_up(kWaitV);
            issue_pv(i);
            if (i + 1 < nt) {
                if (!mbar_wait(bar_k0 + 8 * ((i + 1) % kStages), ((i + 1) / kStages) & 1, &abort_flag)) give_up(kWaitK);
                issue_qk(i + 1);
            }
        }
    }

    if (!mbar_wait(bar_o, (nt - 1) & 1, &abort_flag)) give_up(kWaitO);
    tc_fence_after_sync();

    // epilogue: O / l -> bf16 (prefill) or fp32 partial (question), LSE = m * scale + ln l
    const bool row_ok = tid < it.rows_valid;
    const int tok = it.q_tok0 + tid / it.row_div;
    const int head = it.q_head0 + tid % it.row_div;
    const float inv_l = (l_run > 0.f) ? 1.f / l_run : 0.f;
    const float lse_val = (l_run > 0.f) ? m_run * p.scale + logf(l_run) : -INFINITY;
#pragma unroll
    for (int c = 0; c < D / 32; ++c) {
        uint32_t orow[32];
        tmem_ld32(tO + lane_off + c * 32, orow);
        tmem_wait_ld();
        if (row_ok) {
            if (p.mode == 0) {
                uint4* dst = reinterpret_cast<uint4*>(p.o + (static_cast<size_t>(tok) * p.Hq + head) * D + c * 32);
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    uint32_t w[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        w[e] = pack_bf16x2(__uint_as_float(orow[v * 8 + 2 * e]) * inv_l,
                                           __uint_as_float(orow[v * 8 + 2 * e + 1]) * inv_l);
                    dst[v] = make_uint4(w[0], w[1], w[2], w[3]);
                }
            } else {
                const size_t row = (static_cast<size_t>(it.split) * p.Q + tok) * p.Hq + head;
                float4* dst = reinterpret_cast<float4*>(p.part_o + row * D + c * 32);
#pragma unroll
                for (int v = 0; v < 8; ++v)
                    dst[v] = make_float4(__uint_as_float(orow[v * 4]) * inv_l, __uint_as_float(orow[v * 4 + 1]) * inv_l,
                                         __uint_as_float(orow[v * 4 + 2]) * inv_l, __uint_as_float(orow[v * 4 + 3]) * inv_l);
            }
        }
    }
    if (row_ok) {
        if (p.mode == 0) {
            if (p.lse) p.lse[static_cast<size_t>(head) * p.n_video + tok] = lse_val;
        } else {
            p.part_lse[(static_cast<size_t>(it.split) * p.Q + tok) * p.Hq + head] = lse_val;
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, kTmemCols);
}

// Merge of key-range partials: lse = log sum_s exp(lse_s), o = sum_s exp(lse_s - lse) o_s.
// One thread per (row, 4 output columns).
__global__ void merge_kernel(const __grid_constant__ MergeParams p) {
    const int vec_per_row = p.d / 4;
    const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const int64_t rows = static_cast<int64_t>(p.Q) * p.Hq;
    if (idx >= rows * vec_per_row) return;
    const int64_t row = idx / vec_per_row;  // = tok * Hq + head
    const int v = static_cast<int>(idx % vec_per_row);
    float m = -INFINITY;
    for (int s = 0; s < p.n_splits; ++s) m = fmaxf(m, p.part_lse[s * rows + row]);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float l = 0.f;
    if (m != -INFINITY) {
        for (int s = 0; s < p.n_splits; ++s) {
            const float ls = p.part_lse[s * rows + row];
            if (ls == -INFINITY) continue;
            const float w = __expf(ls - m);
            l += w;
            const float4 o = reinterpret_cast<const float4*>(p.part_o + (s * rows + row) * p.d)[v];
            acc.x += w * o.x; acc.y += w * o.y; acc.z += w * o.z; acc.w += w * o.w;
        }
    }
    const float inv = (l > 0.f) ? 1.f / l : 0.f;
    uint2 out;
    out.x = pack_bf16x2(acc.x * inv, acc.y * inv);
    out.y = pack_bf16x2(acc.z * inv, acc.w * inv);
    reinterpret_cast<uint2*>(p.o + row * p.d)[v] = out;
    if (p.lse && v == 0) {
        const int tok = static_cast<int>(row / p.Hq), head = static_cast<int>(row % p.Hq);
        p.lse[static_cast<int64_t>(head) * p.Q + tok] = (l > 0.f) ? m + logf(l) : -INFINITY;
    }
}

cudaError_t launch_attn(const AttnParams& p, int head_dim, const CUtensorMap& tq, const CUtensorMap& tk,
                        const CUtensorMap& tv, cudaStream_t stream) {
    if (p.n_items <= 0) return cudaSuccess;
    const size_t smem = attn_smem_bytes(head_dim);
    cudaError_t e;
    if (head_dim == 128) {
        e = cudaFuncSetAttribute(attn_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e != cudaSuccess) return e;
        attn_kernel<128><<<p.n_items, kAttnThreads, smem, stream>>>(p, tq, tk, tv);
    } else {
        e = cudaFuncSetAttribute(attn_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e != cudaSuccess) return e;
        attn_kernel<64><<<p.n_items, kAttnThreads, smem, stream>>>(p, tq, tk, tv);
    }
    return cudaGetLastError();
}

cudaError_t launch_merge(const MergeParams& p, cudaStream_t stream) {
    const int64_t n = static_cast<int64_t>(p.Q) * p.Hq * (p.d / 4);
    if (n <= 0) return cudaSuccess;
    merge_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace pevlm
