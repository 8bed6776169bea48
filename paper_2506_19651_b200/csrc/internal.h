// Internal declarations shared by the library's translation units (not part of the C ABI).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/pevlm.h"

namespace pevlm {

constexpr int kTile = 128;        // query-tile rows (MMA M) and key-tile columns (MMA N max)
constexpr int kStatusBytes = 256; // first bytes of every workspace: status word + detail + counters
constexpr int kNumSms = 148;      // B200; used only to size the key splits of the question attention

// Workspace header (device memory, first kStatusBytes of the workspace).
struct WorkspaceHeader {
    int32_t status;  // 0 or PEVLM_ETIMEOUT
    int32_t detail;  // which wait expired (kernel-specific code)
    int32_t work_counter;
    int32_t pad[61];
};

// What one launch of the attention kernel does.  mode 0: prefill rows (sink + blocks, or
// full causal); mode 1: question rows against the assembled cache, split over keys.
struct AttnParams {
    int32_t mode;
    int32_t S, B, N;        // prefill geometry (full causal: S = 0, B = n_video, N = 1)
    int32_t n_video;        // S + N*B
    int32_t blk_key0;       // mode 0: K/V row of the first context block (S, or the cache row of a block range)
    int32_t blk_q0;         // mode 0: row of q / o where the first context block starts (S, or 0 for a block range)
    int32_t q_rows;         // mode 0: rows of q / o = row stride of lse
    int32_t Q, L;           // question length, total length
    int32_t Hq, Hkv, G;
    int32_t tiles_sink;     // ceil(S / 128)
    int32_t tiles_block;    // ceil(B / 128)
    int32_t pairs_block;    // ceil(G * tiles_block / 2) query-tile pairs per (block, kv head)
    int32_t pairs_sink;     // ceil(G * tiles_sink / 2) query-tile pairs per kv head
    int32_t pair_chunk;     // pairs of one (block, kv head) handed out together (see decode_item)
    int32_t items_block;    // work items over the context blocks, padded: N * Hkv * pair_chunk * chunks
    int32_t n_items;        // all work items of the launch
    // ragged last query tile of a segment (len % 128 rows): the tails of tail_heads q heads of one kv
    // group are packed into one 128-row tile, tail_tiles such tiles per (segment, kv head); 0 = no packing
    int32_t tail_rows_block, tail_heads_block, tail_tiles_block;
    int32_t tail_rows_sink, tail_heads_sink, tail_tiles_sink;
    int32_t tok_per_tile;   // mode 1: question tokens per query tile = 128 / G
    int32_t q_tiles;        // mode 1: ceil(Q / tok_per_tile)
    int32_t n_splits;       // mode 1
    int32_t tiles_per_split;// mode 1
    uint64_t wait_limit_ns; // longest a single device-side wait may last before the launch reports PEVLM_ETIMEOUT
    float scale;            // softmax scale
    float scale_log2;       // scale * log2(e)
    __nv_bfloat16* o;       // mode 0: [n_video, Hq, d]
    float* lse;             // mode 0: [Hq, n_video] or NULL
    float* part_o;          // mode 1: [n_splits, Q, Hq, d] fp32
    float* part_lse;        // mode 1: [n_splits, Q, Hq]
    WorkspaceHeader* hdr;
};

struct MergeParams {
    int32_t Q, Hq, d, n_splits;
    const float* part_o;
    const float* part_lse;
    __nv_bfloat16* o;  // [Q, Hq, d]
    float* lse;        // [Hq, Q] or NULL
};

struct RopeParams {
    double inv_freq[64];  // theta^(-2i/d), i < d/2, computed on the host in fp64
    const __nv_bfloat16* q_in;
    const __nv_bfloat16* k_in;
    __nv_bfloat16* q_out;
    __nv_bfloat16* k_out;
    const int32_t* pos_ids;
    int64_t first_token;
    int64_t n_tokens;
    int32_t Hq, Hkv;  // heads to process of each tensor (0 = skip tensor)
    int32_t head_split;  // slots sharing one token's heads (set by launch_rope)
    // multimodal RoPE: pos3 != NULL selects it; rotary pair i takes its position from component 0 for
    // i < sec_end0, component 1 for i < sec_end1, else component 2; pos3 is [3, n_tokens]
    const int32_t* pos3;
    int32_t sec_end0, sec_end1;
};

struct CopySegments {
    const uint4* src[4];
    uint4* dst[4];
    int64_t n_vec[4];  // 16-byte vectors per segment
    int64_t total;
};

cudaError_t launch_rope(const RopeParams& p, int head_dim, cudaStream_t stream);
cudaError_t launch_copy_segments(const CopySegments& s, cudaStream_t stream);
// Tensor maps of one attention launch.  q: [rows, Hq, d] with a 128-token box; q_tail_*: the same tensor with the
// box of a packed ragged tail (heads x tail rows).  K and V each have two maps so that a ragged last key tile
// reads zeros past the end of its range instead of a neighbour's rows: *_sink covers cache rows [0, S), k / v
// cover the context blocks of the call (base at the first block's row) or, for the question attention, the cache.
struct AttnMaps {
    CUtensorMap q, q_tail_block, q_tail_sink, k_sink, v_sink, k, v;
};
cudaError_t launch_attn(const AttnParams& p, int head_dim, const AttnMaps& m, cudaStream_t stream);
cudaError_t launch_wait_selftest(WorkspaceHeader* hdr, uint64_t limit_ns, cudaStream_t stream);
// device address of the built-in scratch array of pevlm_query_attn_noalloc on the current device
int noalloc_scratch_for_current_device(void** out);
int check_query_args(const pevlm_shape_t* s, const void* q_question, const void* k_cache, const void* v_cache,
                     const void* o, const float* lse);
cudaError_t launch_merge(const MergeParams& p, cudaStream_t stream);
size_t attn_smem_bytes(int head_dim);
// error reporting shared by the host-side translation units: both record a text that
// pevlm_last_cuda_error returns on the calling thread
int cuda_fail(cudaError_t e, const char* what);      // returns PEVLM_ECUDA
int fail_with_text(int code, const char* text);      // returns code

}  // namespace pevlm
