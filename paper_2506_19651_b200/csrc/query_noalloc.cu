// pevlm_query_attn_noalloc: question attention for callers that cannot allocate device memory.
//
// Some hosts of this library are not allowed to call cudaMalloc (or any allocating library
// routine) at the point where they need the question attention: code running inside a
// framework's memory-planned region, a real-time serving loop that must not touch the driver's
// allocator, or a plug-in that is handed inputs and outputs but owns no memory pool of its own.
// For them the split-KV partials live in a fixed array that is part of the loaded library
// image on every GPU, instead of a caller-provided workspace.
#include <cstdio>
#include <mutex>

#include "internal.h"

namespace {

constexpr size_t kScratchBytes = PEVLM_NOALLOC_SCRATCH_BYTES;
constexpr int kMaxDevices = 64;

// File-scope device array: every GPU that loads the library holds these bytes until the
// process exits.  In HOST code this name is only a stand-in for the symbol; the device address
// comes from cudaGetSymbolAddress below and is what the kernels receive.
static __device__ __align__(256) unsigned char g_query_scratch[kScratchBytes];

std::mutex g_setup_mutex;
void* g_scratch_ptr[kMaxDevices] = {};

}  // namespace

// Once per device, with that device current: resolve the device address of the scratch array.
int pevlm::noalloc_scratch_for_current_device(void** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return pevlm::cuda_fail(e, "cudaGetDevice");
    if (dev < 0 || dev >= kMaxDevices) return pevlm::fail_with_text(PEVLM_EUNSUPPORTED, "device ordinal beyond 63");
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_ptr[dev]) {
        void* ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_query_scratch);
        if (e != cudaSuccess) return pevlm::cuda_fail(e, "cudaGetSymbolAddress(no-alloc scratch)");
        g_scratch_ptr[dev] = ptr;
    }
    *out = g_scratch_ptr[dev];
    return PEVLM_OK;
}

extern "C" int pevlm_query_attn_noalloc(const pevlm_shape_t* shape, const void* q_question, const void* k_cache,
                                        const void* v_cache, void* o, float* lse, void* stream) {
    // Everything that can be refused on the host is refused before the device is touched: a bad shape or
    // pointer by the same checks as the workspace entry point, then a shape beyond the array.
    const int bad = pevlm::check_query_args(shape, q_question, k_cache, v_cache, o, lse);
    if (bad != PEVLM_OK) return bad;
    const size_t need = pevlm_workspace_bytes(shape, PEVLM_WS_QUERY);
    if (need > kScratchBytes) {
        char text[160];
        snprintf(text, sizeof(text), "pevlm_query_attn_noalloc: this shape needs %zu scratch bytes, the built-in array holds %zu",
                 need, kScratchBytes);
        return pevlm::fail_with_text(PEVLM_EWORKSPACE, text);
    }
    void* scratch = nullptr;
    const int rc = pevlm::noalloc_scratch_for_current_device(&scratch);
    if (rc != PEVLM_OK) return rc;
    // Same kernels as pevlm_query_attn, with the built-in array as the workspace.  The status
    // header at its start is cleared on the stream by that call; the partials are fully
    // overwritten before the merge reads them, so nothing else has to start at zero.
    return pevlm_query_attn(shape, q_question, k_cache, v_cache, o, lse, scratch, kScratchBytes, stream);
}
