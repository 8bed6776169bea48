/*
 * pevlm.h -- C ABI of the B200 (sm_100a) PEVLM prefill-attention library.
 *
 * The method (paper sections in brackets): a long video token stream is laid out as
 *   [ sink | c_0 | c_1 | ... | c_{N-1} | question ]          lengths S, B, .., B, Q
 * with L = S + N*B + Q [Sec. 3.2.1, Sec. 3.2.3].  Every token keeps its original global
 * position for RoPE [Sec. 3.2.2].  With f = softmax(Q K^T / sqrt(d)) V [Eq. 1]:
 *   sink rows      attend causally to the sink                         [Eq. 3]
 *   rows of c_i    attend to the whole sink and causally to c_i        [Eq. 4, Eq. 8]
 *   question rows  attend causally to every token                      [Eq. 5]
 * The sink's K/V are computed once and shared by all blocks [Sec. 1, Sec. 3.1].
 *
 * Conventions the paper leaves open and this library fixes: the diagonal is visible;
 * RoPE rotates the pairs (i, i + d/2); q head h uses kv head h / (Hq/Hkv); LSE is the
 * natural log of the sum of exp(scaled score).
 *
 * General rules for every entry point
 *   - All tensor pointers are DEVICE pointers, contiguous, bf16 (2-byte brain float) unless
 *     stated, and 16-byte aligned; the attention OUTPUT `o` of pevlm_parallel_prefill_attn,
 *     pevlm_block_attn and pevlm_query_attn(_noalloc) must be 32-byte aligned (its rows are
 *     written with 32-byte vector stores), workspaces 256-byte aligned.  A pointer that misses
 *     its alignment is refused with PEVLM_EALIGN before any launch.  `stream` is a
 *     cudaStream_t passed as void* (NULL = the legacy default stream).  `shape` is a HOST
 *     pointer.  Input values must be finite.
 *   - The caller owns every buffer and the stream.  The library allocates no device
 *     memory, never synchronises the device (pevlm_read_status excepted) and never frees
 *     anything.  Calls are asynchronous on `stream`.  No state is kept between calls, with
 *     one exception: pevlm_query_attn_noalloc owns a fixed device array per GPU and
 *     remembers its address (see there).
 *   - batch > 1 means `batch` independent sequences of the same shape, stored one after
 *     another (the leading dimension of every tensor, and of the workspace partials).
 *   - Return value: PEVLM_OK (0) or a negative pevlm_status_t.  All argument checking
 *     happens before any launch; nothing aborts, traps or throws.  Device-side waits are
 *     bounded: if one expires the kernel records PEVLM_ETIMEOUT in the first word of the
 *     workspace and finishes; read it with pevlm_read_status after the stream is idle.
 */
#ifndef PEVLM_H_
#define PEVLM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    PEVLM_OK = 0,
    PEVLM_EINVAL = -1,       /* bad shape or NULL pointer */
    PEVLM_EALIGN = -2,       /* a pointer misses its alignment (16 bytes; attention outputs 32; workspaces 256) */
    PEVLM_EUNSUPPORTED = -3, /* head_dim not in {64,128}, device is not sm_100, ... */
    PEVLM_EWORKSPACE = -4,   /* workspace NULL or too small */
    PEVLM_ECUDA = -5,        /* a CUDA call failed; text via pevlm_last_cuda_error */
    PEVLM_ETIMEOUT = -6      /* a bounded device-side wait expired (see pevlm_read_status) */
} pevlm_status_t;

typedef enum {
    PEVLM_MASK_PEVLM = 0,      /* Eq. 3-5: sink + own block */
    PEVLM_MASK_FULL_CAUSAL = 1 /* plain causal attention over the video tokens (Eq. 1-2) */
} pevlm_mask_mode_t;

typedef struct {
    int32_t batch;         /* >= 1 */
    int32_t sink_len;      /* S >= 0 tokens  [Sec. 3.2.1 "Sink Block"] */
    int32_t block_len;     /* B >= 1 if num_blocks > 0  [uniform "Context Blocks"] */
    int32_t num_blocks;    /* N >= 0 */
    int32_t query_len;     /* Q >= 0  ["Question Block"] */
    int32_t num_q_heads;   /* Hq */
    int32_t num_kv_heads;  /* Hkv, Hq % Hkv == 0 */
    int32_t head_dim;      /* d in {64, 128} */
    float rope_theta;      /* RoPE base, e.g. 1e4 or 1e6 */
    float softmax_scale;   /* 0 => 1/sqrt(d)  [Eq. 1] */
    int32_t mask_mode;     /* pevlm_mask_mode_t */
} pevlm_shape_t;

typedef enum {
    PEVLM_WS_PREFILL = 0, /* workspace of pevlm_parallel_prefill_attn */
    PEVLM_WS_QUERY = 1    /* workspace of pevlm_query_attn */
} pevlm_workspace_kind_t;

/*
 * RoPE at global positions [Sec. 3.2.2].  Rotates every head vector of q_in
 * [n_tokens, Hq, d] and k_in [n_tokens, Hkv, d] by the angles pos * theta^(-2i/d),
 * i < d/2, pairing elements (i, i+d/2), where pos = pos_ids[t] if pos_ids != NULL (device
 * int32[n_tokens]) else first_token + t.  Angle, sine/cosine and rotation are evaluated in
 * fp64; the result is rounded once, fp64 -> fp32 -> bf16, round-to-nearest-even.  Results
 * go to q_out / k_out (same shapes); out may equal in (in place) or be any other buffer
 * (for K: the slot of these tokens in the KV cache).  Either (q_in,q_out) or (k_in,k_out)
 * may both be NULL to skip that tensor.  batch applies to all four tensors and to pos_ids.
 */
int pevlm_rope_qk(const pevlm_shape_t* shape, const void* q_in, const void* k_in, void* q_out,
                  void* k_out, int64_t first_token, int64_t n_tokens, const int32_t* pos_ids,
                  void* stream);

/*
 * Multimodal RoPE: the model family the paper evaluates encodes temporal and spatial coordinates in its
 * position embedding (Sec. 3.1), so every token has three position
 * components, pos_ids3 = device int32 [3, n_tokens] (temporal, height, width).  Rotary pair i < d/2 takes
 * its position from component 0 for i < sections[0], from component 1 for the next sections[1] pairs and
 * from component 2 for the last sections[2] (host int32[3], sum = d/2; the split itself is the model's,
 * not the paper's, e.g. {16, 24, 24} at d = 128).  Sequential positions in the sense of Sec. 3.2.2 means
 * the ids are those of the unpartitioned stream.  Everything else as pevlm_rope_qk (fp64 evaluation, one
 * rounding, in place or out of place, NULL pairs skipped); batch applies to pos_ids3 as [batch, 3, n_tokens].
 */
int pevlm_rope_qk_mrope(const pevlm_shape_t* shape, const void* q_in, const void* k_in, void* q_out,
                        void* k_out, int64_t n_tokens, const int32_t* pos_ids3, const int32_t* sections,
                        void* stream);

/*
 * Prefill attention of the video tokens [Eq. 3, Eq. 4]: rows [0, S + N*B).
 *   q [S+N*B, Hq, d], k, v [S+N*B, Hkv, d]  (q, k already roped), read only
 *   o [S+N*B, Hq, d] bf16, lse [Hq, S+N*B] fp32 (may be NULL), written
 * With mask_mode = PEVLM_MASK_FULL_CAUSAL the same kernel computes plain causal
 * attention over the S+N*B tokens.  Only the tiles a query tile can see are visited.
 * workspace: >= pevlm_workspace_bytes(shape, PEVLM_WS_PREFILL) bytes, 256-byte aligned.
 */
int pevlm_parallel_prefill_attn(const pevlm_shape_t* shape, const void* q, const void* k,
                                const void* v, void* o, float* lse, void* workspace,
                                size_t workspace_bytes, void* stream);

/*
 * Attention of a range of context blocks against a resident cache [Eq. 4 for those blocks alone]: the
 * num_blocks blocks of block_len tokens whose roped K and V sit at rows [first_key_row, first_key_row + N*B)
 * of k_cache / v_cache [cache_rows, Hkv, d]; rows [0, S) of the cache are the sink.  Each block sees the
 * sink and itself causally, exactly as in pevlm_parallel_prefill_attn; the sink rows are not recomputed.
 *   q_blocks [N*B, Hq, d] roped, o [N*B, Hq, d], lse [Hq, N*B] (may be NULL): the block rows only.
 * Because blocks do not attend to one another (Sec. 1), this one call serves (i) a video whose length is
 * not a multiple of the block length (Sec. 3.2.1 partitions uniformly and is silent on a remainder: the
 * remainder is taken as one shorter last block, run with block_len = its length), (ii) a streaming window
 * that encodes one new block against the fixed sink into any free slot of the cache (the paper's
 * future work, Sec. 5), (iii) per-sequence shapes, one call per shape.  mask_mode must be
 * PEVLM_MASK_PEVLM; first_key_row >= S and first_key_row + N*B <= cache_rows, else PEVLM_EINVAL.
 * batch strides: N*B rows for q / o / lse, cache_rows rows for the caches.  Workspace as for
 * pevlm_parallel_prefill_attn.  Only cache rows [0, S) and the block range are read: a ragged last key tile
 * takes zeros, not the neighbouring rows, past the end of either range, so the rest of the cache may hold
 * anything (uninitialised slots of a streaming window included).
 */
int pevlm_block_attn(const pevlm_shape_t* shape, const void* q_blocks, const void* k_cache,
                     const void* v_cache, int64_t first_key_row, int64_t cache_rows, void* o, float* lse,
                     void* workspace, size_t workspace_bytes, void* stream);

/*
 * KV-cache assembly [Eq. 5's key set s + c_all + q]: k_cache, v_cache [L, Hkv, d] receive
 * the video rows [0, S+N*B) from k_video / v_video and the question rows from k_question /
 * v_question [Q, Hkv, d].  K inputs are roped.  A source pointer may be NULL to skip that
 * part (for instance when pevlm_rope_qk already wrote K into the cache).
 */
int pevlm_assemble_kv(const pevlm_shape_t* shape, const void* k_video, const void* v_video,
                      const void* k_question, const void* v_question, void* k_cache,
                      void* v_cache, void* stream);

/*
 * Question attention [Eq. 5]: the Q question rows attend to cache rows [0, S+N*B) and
 * causally to the question rows themselves (cache rows S+N*B ..).  Split over the key
 * range; partials are merged by their log-sum-exp.
 *   q_question [Q, Hq, d] roped; k_cache, v_cache [L, Hkv, d]
 *   o [Q, Hq, d] bf16, lse [Hq, Q] fp32 (may be NULL)
 * workspace: >= pevlm_workspace_bytes(shape, PEVLM_WS_QUERY) bytes, 256-byte aligned.
 */
int pevlm_query_attn(const pevlm_shape_t* shape, const void* q_question, const void* k_cache,
                     const void* v_cache, void* o, float* lse, void* workspace,
                     size_t workspace_bytes, void* stream);

/*
 * Question attention without a caller workspace.  (The paper has no counterpart to this entry
 * point; it exists for deployment.)
 *
 * For callers that cannot allocate device memory where they need this step -- code inside a
 * memory-planned or real-time region that must not call cudaMalloc or any allocating library
 * routine, or a plug-in that is handed inputs and outputs but owns no memory pool.  Same
 * arguments, results and errors as pevlm_query_attn, minus the workspace: the split-KV partials
 * go to a fixed array of PEVLM_NOALLOC_SCRATCH_BYTES that is part of the library image, so
 * every GPU that loads the library holds that much device memory until the process exits.
 *   - Shapes whose pevlm_workspace_bytes(shape, PEVLM_WS_QUERY) exceeds that size are rejected
 *     with PEVLM_EWORKSPACE before any launch (text via pevlm_last_cuda_error).
 *   - The call itself performs no cudaMalloc / cudaFree and uses no allocating routine.
 *   - The first call on each device resolves the array's device address
 *     (cudaGetSymbolAddress, with that device current); make that first call outside any
 *     stream capture.
 *   - All calls on one device share the one array, which keeps the previous call's contents:
 *     each call clears the status header it needs on the stream and overwrites the partials it
 *     reads.  Two calls whose kernels overlap on the GPU (different streams, no ordering
 *     between them) race on the array; order them.
 *   - A device-side timeout is left in the array's header; pevlm_read_status with
 *     workspace = NULL reads it back (for the current device).
 */
#define PEVLM_NOALLOC_SCRATCH_BYTES (32u << 20)
int pevlm_query_attn_noalloc(const pevlm_shape_t* shape, const void* q_question, const void* k_cache,
                             const void* v_cache, void* o, float* lse, void* stream);

/* Bytes of workspace the given call needs for this shape (0 if the shape is invalid). */
size_t pevlm_workspace_bytes(const pevlm_shape_t* shape, int which /* pevlm_workspace_kind_t */);

/*
 * Reads the status word a kernel may have left in `workspace` (device pointer; NULL = the
 * built-in array of pevlm_query_attn_noalloc on the current device).  Blocks the calling host
 * thread until `stream` is idle.  *status = PEVLM_OK or PEVLM_ETIMEOUT; *detail (may be NULL)
 * = wait id * 1000000 + index of the thread block whose wait expired.
 */
int pevlm_read_status(const void* workspace, void* stream, int32_t* status, int32_t* detail);

/*
 * Self-test of the failure path (the paper has no counterpart): launches one thread block that
 * waits, with the library's bounded wait, on a barrier nothing ever arrives on.  After limit_ns
 * (1 us .. 100 ms) the wait gives up, the kernel records PEVLM_ETIMEOUT with wait id 99 in the
 * header of `workspace` (>= 256 bytes, 256-byte aligned) and ends normally; the context stays
 * usable and the next call on the same workspace clears the status.  Nothing traps or faults.
 */
int pevlm_selftest_wait_expiry(void* workspace, size_t workspace_bytes, int64_t limit_ns, void* stream);

/*
 * Executed tensor-core work of a call for this shape, for throughput accounting:
 * *tiles = number of (query tile, key tile) MMAs pairs visited over all heads and batch,
 * *flops = 4 * d * sum over visited tiles of (tile rows * tile key columns issued).
 */
int pevlm_tile_stats(const pevlm_shape_t* shape, int which, int64_t* tiles, double* flops);

const char* pevlm_strerror(int code);
/* Text of the last CUDA error seen by this thread inside the library ("" if none). */
const char* pevlm_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* PEVLM_H_ */
