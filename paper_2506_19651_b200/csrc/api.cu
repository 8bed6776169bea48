// C ABI of the library: argument checking, TMA tensor-map encoding and kernel launches.
// Everything here runs on the host; no device memory is allocated and nothing synchronises
// except pevlm_read_status.
#include <cmath>
#include <cstdio>
#include <cstring>

#include "internal.h"
#include "ptx.cuh"

namespace pevlm {

static thread_local char g_cuda_error[256] = "";

int cuda_fail(cudaError_t e, const char* what) {
    snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s", what, cudaGetErrorString(e));
    return PEVLM_ECUDA;
}

int fail_with_text(int code, const char* text) {
    snprintf(g_cuda_error, sizeof(g_cuda_error), "%s", text);
    return code;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static bool aligned32(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 31u) == 0; }
static bool aligned256(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }

static int check_shape(const pevlm_shape_t* s) {
    if (!s) return PEVLM_EINVAL;
    if (s->batch < 1 || s->sink_len < 0 || s->num_blocks < 0 || s->query_len < 0) return PEVLM_EINVAL;
    if (s->num_blocks > 0 && s->block_len < 1) return PEVLM_EINVAL;
    if (s->block_len < 0) return PEVLM_EINVAL;
    if (s->num_q_heads < 1 || s->num_kv_heads < 1 || s->num_q_heads % s->num_kv_heads != 0) return PEVLM_EINVAL;
    if (s->mask_mode != PEVLM_MASK_PEVLM && s->mask_mode != PEVLM_MASK_FULL_CAUSAL) return PEVLM_EINVAL;
    if (!(s->rope_theta > 0.f) || !(s->softmax_scale >= 0.f)) return PEVLM_EINVAL;
    const int64_t L = static_cast<int64_t>(s->sink_len) + static_cast<int64_t>(s->num_blocks) * s->block_len + s->query_len;
    if (L < 1 || L > (1ll << 30)) return PEVLM_EINVAL;
    if (s->head_dim != 64 && s->head_dim != 128) return PEVLM_EUNSUPPORTED;
    if (s->num_q_heads / s->num_kv_heads > kTile) return PEVLM_EUNSUPPORTED;
    return PEVLM_OK;
}

static int64_t n_video(const pevlm_shape_t* s) {
    return static_cast<int64_t>(s->sink_len) + static_cast<int64_t>(s->num_blocks) * s->block_len;
}

static int check_device() {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    int major = 0;
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute");
    if (major != 10) return PEVLM_EUNSUPPORTED;
    return PEVLM_OK;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// Tensor map over a [tokens, heads, d] bf16 tensor (d contiguous) with a box of
// 64 elements x box_heads x box_tokens and the 128-byte swizzle the MMA descriptors expect.
// Rows past the end of the tensor read as zero.
static int make_tmap(CUtensorMap* m, const void* base, int64_t tokens, int heads, int d, int box_heads, int box_tokens) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) {
        snprintf(g_cuda_error, sizeof(g_cuda_error), "cuTensorMapEncodeTiled entry point not found");
        return PEVLM_ECUDA;
    }
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(heads), static_cast<cuuint64_t>(tokens)};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(d) * 2, static_cast<cuuint64_t>(d) * 2 * heads};
    cuuint32_t box[3] = {64, static_cast<cuuint32_t>(box_heads), static_cast<cuuint32_t>(box_tokens)};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(g_cuda_error, sizeof(g_cuda_error), "cuTensorMapEncodeTiled failed with CUresult %d", static_cast<int>(r));
        return PEVLM_ECUDA;
    }
    return PEVLM_OK;
}

static float resolve_scale(const pevlm_shape_t* s) {
    return s->softmax_scale > 0.f ? s->softmax_scale : 1.0f / sqrtf(static_cast<float>(s->head_dim));
}

// ---- query tiles of one prefill segment (sink or context block) per kv head, shared by the launch and
// the stats.  A segment of `len` tokens has ceil(len/128) tile positions; if the last one is ragged with
// at most 64 rows, the tails of `tail_heads` q heads of the kv group share one 128-row tile.
struct SegPlan {
    int tiles, tail_rows, tail_heads, tail_tiles, full_tiles, entries, pairs;
};

static SegPlan plan_segment(int len, int G) {
    SegPlan s;
    s.tiles = (len + kTile - 1) / kTile;
    s.tail_rows = 0; s.tail_heads = 0; s.tail_tiles = 0;
    const int rem = len % kTile;
    if (rem > 0 && rem <= kTile / 2 && G > 1) {
        s.tail_rows = rem;
        s.tail_heads = kTile / rem < G ? kTile / rem : G;
        s.tail_tiles = (G + s.tail_heads - 1) / s.tail_heads;
    }
    s.full_tiles = s.tiles - (s.tail_tiles > 0 ? 1 : 0);
    s.entries = s.tail_tiles + G * s.full_tiles;
    s.pairs = (s.entries + 1) / 2;
    return s;
}

// ---- question-attention decomposition (shared by the launch, the workspace size and the stats)
struct QueryPlan {
    int tok_per_tile, q_tiles, total_kv_tiles, n_splits, tiles_per_split;
};

static QueryPlan plan_query(const pevlm_shape_t* s) {
    QueryPlan q;
    const int G = s->num_q_heads / s->num_kv_heads;
    const int64_t L = n_video(s) + s->query_len;
    q.tok_per_tile = kTile / G;
    q.q_tiles = (s->query_len + q.tok_per_tile - 1) / q.tok_per_tile;
    q.total_kv_tiles = static_cast<int>((L + kTile - 1) / kTile);
    // Work items are (kv head, pair of query tiles, key split).  The kernel is persistent with one
    // CTA per SM, so the split count is chosen to give one full wave of the 148 SMs of a B200:
    // as many splits as fit, never more than there are key tiles.
    const int pairs = (q.q_tiles + 1) / 2;
    const int groups = s->num_kv_heads * (pairs > 0 ? pairs : 1);
    int want = kNumSms / groups;
    if (want < 1) want = 1;
    if (want > q.total_kv_tiles) want = q.total_kv_tiles;
    q.tiles_per_split = (q.total_kv_tiles + want - 1) / want;
    q.n_splits = (q.total_kv_tiles + q.tiles_per_split - 1) / q.tiles_per_split;
    return q;
}

static size_t query_partial_floats(const pevlm_shape_t* s, const QueryPlan& q) {
    return static_cast<size_t>(q.n_splits) * s->query_len * s->num_q_heads * (s->head_dim + 1);
}

// Host-side argument checks of the question attention, shared by its two entry points.
int check_query_args(const pevlm_shape_t* s, const void* q_question, const void* k_cache, const void* v_cache,
                     const void* o, const float* lse) {
    const int rc = check_shape(s);
    if (rc != PEVLM_OK) return rc;
    if (!q_question || !k_cache || !v_cache || !o) return PEVLM_EINVAL;
    if (!aligned16(q_question) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned32(o) || !aligned16(lse))
        return PEVLM_EALIGN;
    return PEVLM_OK;
}

}  // namespace pevlm

using namespace pevlm;

extern "C" {

const char* pevlm_strerror(int code) {
    switch (code) {
        case PEVLM_OK: return "ok";
        case PEVLM_EINVAL: return "invalid shape or NULL pointer";
        case PEVLM_EALIGN: return "pointer not 16-byte aligned (attention outputs: 32-byte, workspace: 256-byte)";
        case PEVLM_EUNSUPPORTED: return "unsupported head_dim / group size, or device is not sm_100";
        case PEVLM_EWORKSPACE: return "workspace missing or too small";
        case PEVLM_ECUDA: return "CUDA error (see pevlm_last_cuda_error)";
        case PEVLM_ETIMEOUT: return "a bounded device-side wait expired";
        default: return "unknown pevlm status";
    }
}

const char* pevlm_last_cuda_error(void) { return g_cuda_error; }

size_t pevlm_workspace_bytes(const pevlm_shape_t* s, int which) {
    if (check_shape(s) != PEVLM_OK) return 0;
    if (which == PEVLM_WS_PREFILL) return kStatusBytes;
    if (which == PEVLM_WS_QUERY) {
        const QueryPlan q = plan_query(s);
        return kStatusBytes + static_cast<size_t>(s->batch) * ((query_partial_floats(s, q) * sizeof(float) + 255) / 256 * 256);
    }
    return 0;
}

static int rope_common(const pevlm_shape_t* s, const void* q_in, const void* k_in, void* q_out, void* k_out,
                       int64_t first_token, int64_t n_tokens, const int32_t* pos_ids, const int32_t* pos3,
                       const int32_t* sections, void* stream) {
    int rc = check_shape(s);
    if (rc != PEVLM_OK) return rc;
    if (n_tokens < 0 || first_token < 0 || first_token + n_tokens > (1ll << 31)) return PEVLM_EINVAL;
    if ((q_in == nullptr) != (q_out == nullptr) || (k_in == nullptr) != (k_out == nullptr)) return PEVLM_EINVAL;
    if (!q_in && !k_in) return PEVLM_EINVAL;
    if (!aligned16(q_in) || !aligned16(k_in) || !aligned16(q_out) || !aligned16(k_out)) return PEVLM_EALIGN;
    if (pos_ids && (reinterpret_cast<uintptr_t>(pos_ids) & 3u)) return PEVLM_EALIGN;
    if (pos3 && (reinterpret_cast<uintptr_t>(pos3) & 3u)) return PEVLM_EALIGN;
    const int d = s->head_dim;
    if (sections) {
        if (sections[0] < 0 || sections[1] < 0 || sections[2] < 0 || sections[0] + sections[1] + sections[2] != d / 2)
            return PEVLM_EINVAL;
    }
    if (n_tokens == 0) return PEVLM_OK;
    RopeParams p;
    for (int i = 0; i < d / 2; ++i) p.inv_freq[i] = pow(static_cast<double>(s->rope_theta), -2.0 * i / d);
    for (int i = d / 2; i < 64; ++i) p.inv_freq[i] = 0.0;
    p.first_token = first_token;
    p.n_tokens = n_tokens;
    p.Hq = q_in ? s->num_q_heads : 0;
    p.Hkv = k_in ? s->num_kv_heads : 0;
    p.head_split = 1;
    p.sec_end0 = sections ? sections[0] : 0;
    p.sec_end1 = sections ? sections[0] + sections[1] : 0;
    for (int b = 0; b < s->batch; ++b) {
        const int64_t qo = static_cast<int64_t>(b) * n_tokens * s->num_q_heads * d;
        const int64_t ko = static_cast<int64_t>(b) * n_tokens * s->num_kv_heads * d;
        p.q_in = q_in ? static_cast<const __nv_bfloat16*>(q_in) + qo : nullptr;
        p.q_out = q_out ? static_cast<__nv_bfloat16*>(q_out) + qo : nullptr;
        p.k_in = k_in ? static_cast<const __nv_bfloat16*>(k_in) + ko : nullptr;
        p.k_out = k_out ? static_cast<__nv_bfloat16*>(k_out) + ko : nullptr;
        p.pos_ids = pos_ids ? pos_ids + static_cast<int64_t>(b) * n_tokens : nullptr;
        p.pos3 = pos3 ? pos3 + static_cast<int64_t>(b) * 3 * n_tokens : nullptr;
        cudaError_t e = launch_rope(p, d, static_cast<cudaStream_t>(stream));
        if (e != cudaSuccess) return cuda_fail(e, "rope launch");
    }
    return PEVLM_OK;
}

int pevlm_rope_qk(const pevlm_shape_t* s, const void* q_in, const void* k_in, void* q_out, void* k_out,
                  int64_t first_token, int64_t n_tokens, const int32_t* pos_ids, void* stream) {
    return rope_common(s, q_in, k_in, q_out, k_out, first_token, n_tokens, pos_ids, nullptr, nullptr, stream);
}

int pevlm_rope_qk_mrope(const pevlm_shape_t* s, const void* q_in, const void* k_in, void* q_out, void* k_out,
                        int64_t n_tokens, const int32_t* pos_ids3, const int32_t* sections, void* stream) {
    if (!pos_ids3 || !sections) return PEVLM_EINVAL;
    return rope_common(s, q_in, k_in, q_out, k_out, 0, n_tokens, nullptr, pos_ids3, sections, stream);
}

int pevlm_assemble_kv(const pevlm_shape_t* s, const void* k_video, const void* v_video, const void* k_question,
                      const void* v_question, void* k_cache, void* v_cache, void* stream) {
    int rc = check_shape(s);
    if (rc != PEVLM_OK) return rc;
    if ((k_video || k_question) && !k_cache) return PEVLM_EINVAL;
    if ((v_video || v_question) && !v_cache) return PEVLM_EINVAL;
    if (!aligned16(k_video) || !aligned16(v_video) || !aligned16(k_question) || !aligned16(v_question) ||
        !aligned16(k_cache) || !aligned16(v_cache))
        return PEVLM_EALIGN;
    const int64_t nv = n_video(s);
    const int64_t row_vec = static_cast<int64_t>(s->num_kv_heads) * s->head_dim * 2 / 16;  // 16-byte vectors per token
    const int64_t L = nv + s->query_len;
    for (int b = 0; b < s->batch; ++b) {
        CopySegments seg;
        const void* srcs[4] = {k_video, k_question, v_video, v_question};
        void* dsts[4] = {k_cache, k_cache, v_cache, v_cache};
        const int64_t rows[4] = {nv, s->query_len, nv, s->query_len};
        const int64_t dst_row0[4] = {0, nv, 0, nv};
        seg.total = 0;
        for (int i = 0; i < 4; ++i) {
            const int64_t n = srcs[i] ? rows[i] * row_vec : 0;
            seg.n_vec[i] = n;
            seg.src[i] = srcs[i] ? static_cast<const uint4*>(srcs[i]) + static_cast<int64_t>(b) * rows[i] * row_vec : nullptr;
            seg.dst[i] = dsts[i] ? static_cast<uint4*>(dsts[i]) + (static_cast<int64_t>(b) * L + dst_row0[i]) * row_vec : nullptr;
            seg.total += n;
        }
        cudaError_t e = launch_copy_segments(seg, static_cast<cudaStream_t>(stream));
        if (e != cudaSuccess) return cuda_fail(e, "assemble launch");
    }
    return PEVLM_OK;
}

// Prefill attention launches.  blocks_only = false: the whole video stream [sink | N blocks] (or full causal).
// blocks_only = true: N blocks whose K/V sit at rows [first_key_row, first_key_row + N*B) of a cache of cache_rows
// rows whose first S rows are the sink; q / o / lse cover the N*B block rows only and the sink rows are not computed.
static int prefill_common(const pevlm_shape_t* s, const void* q, const void* k, const void* v, void* o, float* lse,
                          void* workspace, size_t workspace_bytes, void* stream, bool blocks_only,
                          int64_t first_key_row, int64_t cache_rows) {
    int rc = check_shape(s);
    if (rc != PEVLM_OK) return rc;
    if (!q || !k || !v || !o) return PEVLM_EINVAL;
    // the output rows are written with 32-byte vector stores
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned32(o) || !aligned16(lse)) return PEVLM_EALIGN;
    if (!workspace || workspace_bytes < pevlm_workspace_bytes(s, PEVLM_WS_PREFILL)) return PEVLM_EWORKSPACE;
    if (!aligned256(workspace)) return PEVLM_EALIGN;
    const int64_t nv = n_video(s);
    const int64_t block_rows = static_cast<int64_t>(s->num_blocks) * s->block_len;
    if (blocks_only) {
        if (s->mask_mode != PEVLM_MASK_PEVLM) return PEVLM_EINVAL;
        if (first_key_row < s->sink_len || first_key_row + block_rows > cache_rows || cache_rows > (1ll << 30))
            return PEVLM_EINVAL;
        if (block_rows == 0) return PEVLM_OK;
    } else if (nv == 0) {
        return PEVLM_OK;
    }
    rc = check_device();
    if (rc != PEVLM_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemsetAsync(workspace, 0, kStatusBytes, st);
    if (e != cudaSuccess) return cuda_fail(e, "workspace memset");

    const int d = s->head_dim;
    const int64_t q_rows = blocks_only ? block_rows : nv;   // rows of q, o, lse
    const int64_t kv_rows = blocks_only ? cache_rows : nv;  // rows of k, v
    AttnParams p;
    memset(&p, 0, sizeof(p));
    p.mode = 0;
    if (s->mask_mode == PEVLM_MASK_FULL_CAUSAL) {
        p.S = 0; p.B = static_cast<int>(nv); p.N = 1;
    } else {
        p.S = s->sink_len; p.B = s->num_blocks > 0 ? s->block_len : 0; p.N = s->num_blocks;
    }
    p.n_video = static_cast<int>(nv);
    p.blk_key0 = blocks_only ? static_cast<int>(first_key_row) : p.S;
    p.blk_q0 = blocks_only ? 0 : p.S;
    p.q_rows = static_cast<int>(q_rows);
    p.Q = s->query_len;
    p.L = static_cast<int>(nv + s->query_len);
    p.Hq = s->num_q_heads; p.Hkv = s->num_kv_heads; p.G = p.Hq / p.Hkv;
    p.tiles_sink = (p.S + kTile - 1) / kTile;
    p.tiles_block = p.N > 0 ? (p.B + kTile - 1) / kTile : 0;
    const SegPlan pb = plan_segment(p.N > 0 ? p.B : 0, p.G), ps = plan_segment(blocks_only ? 0 : p.S, p.G);
    p.pairs_block = pb.pairs;
    p.pairs_sink = ps.pairs;
    p.tail_rows_block = pb.tail_rows; p.tail_heads_block = pb.tail_heads; p.tail_tiles_block = pb.tail_tiles;
    p.tail_rows_sink = ps.tail_rows; p.tail_heads_sink = ps.tail_heads; p.tail_tiles_sink = ps.tail_tiles;
    // How many pairs of one (block, kv head) are handed out together (decode_item): the whole list keeps the CTAs
    // that run at the same time on few K/V tiles (best for long blocks); short blocks (at most 4 query tiles)
    // run faster when pairs of equal length are handed out together across all blocks, and a launch with few
    // items per SM balances best with single pairs, heaviest first.  Thresholds from measurements on B200.
    int want_pc = p.pairs_block;
    if (p.tiles_block <= 4) want_pc = p.G / 2 > 0 ? p.G / 2 : 1;
    else if (static_cast<int64_t>(p.N) * p.Hkv * p.pairs_block < 16 * kNumSms) want_pc = 1;
    p.pair_chunk = p.pairs_block > 0 ? (want_pc < p.pairs_block ? want_pc : p.pairs_block) : 1;
    const int n_chunks = p.pairs_block > 0 ? (p.pairs_block + p.pair_chunk - 1) / p.pair_chunk : 0;
    p.items_block = p.N * p.Hkv * p.pair_chunk * n_chunks;
    p.n_items = p.items_block + p.Hkv * p.pairs_sink;
    p.scale = resolve_scale(s);
    p.scale_log2 = p.scale * 1.4426950408889634f;
    p.wait_limit_ns = kDefaultWaitLimitNs;
    p.hdr = static_cast<WorkspaceHeader*>(workspace);
    const int64_t block_rows_launch = static_cast<int64_t>(p.N) * p.B;  // full causal: the whole stream as one block
    for (int b = 0; b < s->batch; ++b) {
        const int64_t qoff = static_cast<int64_t>(b) * q_rows * p.Hq * d, koff = static_cast<int64_t>(b) * kv_rows * p.Hkv * d;
        AttnMaps m;
        const __nv_bfloat16* qb = static_cast<const __nv_bfloat16*>(q) + qoff;
        if ((rc = make_tmap(&m.q, qb, q_rows, p.Hq, d, 1, kTile)) != PEVLM_OK) return rc;
        m.q_tail_block = m.q;
        m.q_tail_sink = m.q;
        if (pb.tail_tiles > 0 && (rc = make_tmap(&m.q_tail_block, qb, q_rows, p.Hq, d, pb.tail_heads, pb.tail_rows)) != PEVLM_OK) return rc;
        if (ps.tail_tiles > 0 && (rc = make_tmap(&m.q_tail_sink, qb, q_rows, p.Hq, d, ps.tail_heads, ps.tail_rows)) != PEVLM_OK) return rc;
        // K and V: one map over the sink rows [0, S) and one over the block rows, so that the ragged last key
        // tile of either range reads zeros past its end (a map needs at least one row; an empty range is never read)
        const __nv_bfloat16* kb = static_cast<const __nv_bfloat16*>(k) + koff;
        const __nv_bfloat16* vb = static_cast<const __nv_bfloat16*>(v) + koff;
        const int64_t blk_off = static_cast<int64_t>(p.blk_key0) * p.Hkv * d;
        const int64_t sink_rows = p.S > 0 ? p.S : 1, blk_rows = block_rows_launch > 0 ? block_rows_launch : 1;
        if ((rc = make_tmap(&m.k_sink, kb, sink_rows, p.Hkv, d, 1, kTile)) != PEVLM_OK) return rc;
        if ((rc = make_tmap(&m.v_sink, vb, sink_rows, p.Hkv, d, 1, kTile)) != PEVLM_OK) return rc;
        if ((rc = make_tmap(&m.k, kb + blk_off, blk_rows, p.Hkv, d, 1, kTile)) != PEVLM_OK) return rc;
        if ((rc = make_tmap(&m.v, vb + blk_off, blk_rows, p.Hkv, d, 1, kTile)) != PEVLM_OK) return rc;
        p.o = static_cast<__nv_bfloat16*>(o) + qoff;
        p.lse = lse ? lse + static_cast<int64_t>(b) * p.Hq * q_rows : nullptr;
        if (b > 0) {  // every launch starts its work counter at zero; the status word is kept
            e = cudaMemsetAsync(&p.hdr->work_counter, 0, sizeof(int32_t), st);
            if (e != cudaSuccess) return cuda_fail(e, "work counter memset");
        }
        e = launch_attn(p, d, m, st);
        if (e != cudaSuccess) return cuda_fail(e, "prefill attention launch");
    }
    return PEVLM_OK;
}

int pevlm_parallel_prefill_attn(const pevlm_shape_t* s, const void* q, const void* k, const void* v, void* o, float* lse,
                                void* workspace, size_t workspace_bytes, void* stream) {
    return prefill_common(s, q, k, v, o, lse, workspace, workspace_bytes, stream, false, 0, 0);
}

int pevlm_block_attn(const pevlm_shape_t* s, const void* q_blocks, const void* k_cache, const void* v_cache,
                     int64_t first_key_row, int64_t cache_rows, void* o, float* lse, void* workspace,
                     size_t workspace_bytes, void* stream) {
    return prefill_common(s, q_blocks, k_cache, v_cache, o, lse, workspace, workspace_bytes, stream, true,
                          first_key_row, cache_rows);
}

int pevlm_query_attn(const pevlm_shape_t* s, const void* q_question, const void* k_cache, const void* v_cache, void* o,
                     float* lse, void* workspace, size_t workspace_bytes, void* stream) {
    int rc = check_query_args(s, q_question, k_cache, v_cache, o, lse);
    if (rc != PEVLM_OK) return rc;
    if (!workspace || workspace_bytes < pevlm_workspace_bytes(s, PEVLM_WS_QUERY)) return PEVLM_EWORKSPACE;
    if (!aligned256(workspace)) return PEVLM_EALIGN;
    if (s->query_len == 0) return PEVLM_OK;
    rc = check_device();
    if (rc != PEVLM_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemsetAsync(workspace, 0, kStatusBytes, st);
    if (e != cudaSuccess) return cuda_fail(e, "workspace memset");

    const int d = s->head_dim;
    const int64_t nv = n_video(s);
    const int64_t L = nv + s->query_len;
    const QueryPlan qp = plan_query(s);
    AttnParams p;
    memset(&p, 0, sizeof(p));
    p.mode = 1;
    p.n_video = static_cast<int>(nv);
    p.Q = s->query_len;
    p.L = static_cast<int>(L);
    p.Hq = s->num_q_heads; p.Hkv = s->num_kv_heads; p.G = p.Hq / p.Hkv;
    p.tok_per_tile = qp.tok_per_tile;
    p.q_tiles = qp.q_tiles;
    p.n_splits = qp.n_splits;
    p.tiles_per_split = qp.tiles_per_split;
    p.n_items = p.Hkv * ((p.q_tiles + 1) / 2) * p.n_splits;
    p.scale = resolve_scale(s);
    p.scale_log2 = p.scale * 1.4426950408889634f;
    p.wait_limit_ns = kDefaultWaitLimitNs;
    p.hdr = static_cast<WorkspaceHeader*>(workspace);
    const size_t part_floats = query_partial_floats(s, qp);
    const size_t part_stride = (part_floats * sizeof(float) + 255) / 256 * 256;
    for (int b = 0; b < s->batch; ++b) {
        float* part = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + kStatusBytes + b * part_stride);
        p.part_o = part;
        p.part_lse = part + static_cast<size_t>(p.n_splits) * p.Q * p.Hq * d;
        const int64_t qoff = static_cast<int64_t>(b) * p.Q * p.Hq * d, koff = static_cast<int64_t>(b) * L * p.Hkv * d;
        if (b > 0) {
            e = cudaMemsetAsync(&p.hdr->work_counter, 0, sizeof(int32_t), st);
            if (e != cudaSuccess) return cuda_fail(e, "work counter memset");
        }
        AttnMaps maps;
        if ((rc = make_tmap(&maps.q, static_cast<const __nv_bfloat16*>(q_question) + qoff, p.Q, p.Hq, d, p.G, p.tok_per_tile)) != PEVLM_OK) return rc;
        if ((rc = make_tmap(&maps.k, static_cast<const __nv_bfloat16*>(k_cache) + koff, L, p.Hkv, d, 1, kTile)) != PEVLM_OK) return rc;
        if ((rc = make_tmap(&maps.v, static_cast<const __nv_bfloat16*>(v_cache) + koff, L, p.Hkv, d, 1, kTile)) != PEVLM_OK) return rc;
        maps.q_tail_block = maps.q; maps.q_tail_sink = maps.q; maps.k_sink = maps.k; maps.v_sink = maps.v;
        e = launch_attn(p, d, maps, st);
        if (e != cudaSuccess) return cuda_fail(e, "question attention launch");
        MergeParams m;
        m.Q = p.Q; m.Hq = p.Hq; m.d = d; m.n_splits = p.n_splits;
        m.part_o = p.part_o; m.part_lse = p.part_lse;
        m.o = static_cast<__nv_bfloat16*>(o) + qoff;
        m.lse = lse ? lse + static_cast<int64_t>(b) * p.Hq * p.Q : nullptr;
        e = launch_merge(m, st);
        if (e != cudaSuccess) return cuda_fail(e, "merge launch");
    }
    return PEVLM_OK;
}

int pevlm_selftest_wait_expiry(void* workspace, size_t workspace_bytes, int64_t limit_ns, void* stream) {
    if (!workspace || workspace_bytes < kStatusBytes) return PEVLM_EWORKSPACE;
    if (!aligned256(workspace)) return PEVLM_EALIGN;
    if (limit_ns < 1000 || limit_ns > 100ll * 1000 * 1000) return PEVLM_EINVAL;  // 1 us .. 100 ms
    int rc = check_device();
    if (rc != PEVLM_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemsetAsync(workspace, 0, kStatusBytes, st);
    if (e != cudaSuccess) return cuda_fail(e, "workspace memset");
    e = launch_wait_selftest(static_cast<WorkspaceHeader*>(workspace), static_cast<uint64_t>(limit_ns), st);
    if (e != cudaSuccess) return cuda_fail(e, "wait self-test launch");
    return PEVLM_OK;
}

int pevlm_read_status(const void* workspace, void* stream, int32_t* status, int32_t* detail) {
    if (!status) return PEVLM_EINVAL;
    if (!workspace) {  // the built-in array of pevlm_query_attn_noalloc on the current device
        void* scratch = nullptr;
        const int rc = noalloc_scratch_for_current_device(&scratch);
        if (rc != PEVLM_OK) return rc;
        workspace = scratch;
    }
    cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
    int32_t words[2] = {0, 0};
    e = cudaMemcpy(words, workspace, sizeof(words), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpy(status)");
    *status = words[0];
    if (detail) *detail = words[1];
    return PEVLM_OK;
}

int pevlm_tile_stats(const pevlm_shape_t* s, int which, int64_t* tiles, double* flops) {
    int rc = check_shape(s);
    if (rc != PEVLM_OK) return rc;
    if (!tiles || !flops) return PEVLM_EINVAL;
    const int d = s->head_dim;
    int64_t n_tiles = 0;
    double cols = 0.0;  // sum over visited tiles of issued key columns (each over 128 query rows)
    auto add_range = [&](int64_t len) {  // a key range visited from its start in 128-key tiles
        for (int64_t j = 0; j < len; j += kTile) {
            const int64_t valid = len - j < kTile ? len - j : kTile;
            n_tiles += 1;
            cols += static_cast<double>((valid + 15) / 16 * 16);
        }
    };
    const int64_t nv = n_video(s);
    if (which == PEVLM_WS_PREFILL) {
        int64_t S = s->sink_len, B = s->num_blocks > 0 ? s->block_len : 0, N = s->num_blocks;
        if (s->mask_mode == PEVLM_MASK_FULL_CAUSAL) { S = 0; B = nv; N = nv > 0 ? 1 : 0; }
        const int G = s->num_q_heads / s->num_kv_heads;
        // query tiles of one segment per kv head: G per full tile position, tail_tiles for a packed ragged tail
        auto add_segment = [&](int64_t len, int64_t shared) {
            const SegPlan sp = plan_segment(static_cast<int>(len), G);
            for (int qt = 0; qt < sp.tiles; ++qt) {
                const int64_t q0 = static_cast<int64_t>(qt) * kTile;
                const int q_tiles = (sp.tail_tiles > 0 && qt == sp.tiles - 1) ? sp.tail_tiles : G;
                const int64_t t0 = n_tiles; const double c0 = cols;
                add_range(shared);
                add_range(q0 + kTile < len ? q0 + kTile : len);
                n_tiles = t0 + (n_tiles - t0) * q_tiles;
                cols = c0 + (cols - c0) * q_tiles;
            }
        };
        add_segment(S, 0);
        const int64_t t0 = n_tiles; const double c0 = cols;
        add_segment(B, S);
        n_tiles = t0 + (n_tiles - t0) * N;   // the block part repeats for each of the N blocks
        cols = c0 + (cols - c0) * static_cast<double>(N);
        n_tiles *= s->num_kv_heads;
        cols *= s->num_kv_heads;
    } else if (which == PEVLM_WS_QUERY) {
        const QueryPlan qp = plan_query(s);
        for (int qt = 0; qt < qp.q_tiles; ++qt) {
            const int tok0 = qt * qp.tok_per_tile;
            const int ntok = s->query_len - tok0 < qp.tok_per_tile ? s->query_len - tok0 : qp.tok_per_tile;
            const int64_t kv_end = nv + tok0 + ntok;
            for (int sp = 0; sp < qp.n_splits; ++sp) {
                int64_t a = static_cast<int64_t>(sp) * qp.tiles_per_split * kTile, e = a + static_cast<int64_t>(qp.tiles_per_split) * kTile;
                if (a > kv_end) a = kv_end;
                if (e > kv_end) e = kv_end;
                add_range(e - a);
            }
        }
        n_tiles *= s->num_kv_heads;
        cols *= s->num_kv_heads;
    } else {
        return PEVLM_EINVAL;
    }
    *tiles = n_tiles * s->batch;
    *flops = 4.0 * d * kTile * cols * s->batch;
    return PEVLM_OK;
}

}  // extern "C"
