// LSE merge of the key-range partials of the question attention (Eq. 5): each split s left
// a locally normalised output o_s and lse_s for every question row; the whole-range result is
//   lse = log sum_s exp(lse_s),   o = sum_s exp(lse_s - lse) o_s.
// A split with no visible key for a row has lse_s = -inf and contributes nothing.
#include "internal.h"
#include "ptx.cuh"

namespace pevlm {

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

cudaError_t launch_merge(const MergeParams& p, cudaStream_t stream) {
    const int64_t n = static_cast<int64_t>(p.Q) * p.Hq * (p.d / 4);
    if (n <= 0) return cudaSuccess;
    merge_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace pevlm
