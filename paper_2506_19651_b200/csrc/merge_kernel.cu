// LSE merge of the key-range partials of the question attention (Eq. 5): each split s left
// a locally normalised output o_s and lse_s for every question row; the whole-range result is
//   lse = log sum_s exp(lse_s),   o = sum_s exp(lse_s - lse) o_s.
// A split with no visible key for a row has lse_s = -inf and contributes nothing.
#include "internal.h"
#include "ptx.cuh"

namespace pevlm {

constexpr int kMergeThreads = 256;
constexpr int kMergeChunk = 16;      // partial rows whose loads are in flight together
constexpr int kMergeMaxParts = 160;  // >= the largest split count (one split per SM at most)

// Many rows (a prefill-sized question block): one thread per (row, 4 output columns), the splits one after
// another; tens of thousands of threads hide the latency of the dependent loads.
__global__ void merge_kernel(const __grid_constant__ MergeParams p) {
    const int vec_per_row = p.d / 4;
    const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const int64_t rows = static_cast<int64_t>(p.Q) * p.Hq;
    if (idx >= rows * vec_per_row) return;
    const int64_t row = idx / vec_per_row;  // = tok * Hq + head
    const int v = static_cast<int>(idx % vec_per_row);
    const int n = p.n_splits;
    float m = -INFINITY;
    for (int s = 0; s < n; ++s) m = fmaxf(m, p.part_lse[s * rows + row]);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float l = 0.f;
    if (m != -INFINITY) {
        for (int s = 0; s < n; ++s) {
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

// Few rows (a decode step has Hq of them): one warp per question row (token, head).  Lane l owns output columns [4l, 4l + 4) (d = 128; lanes 0-15 at
// d = 64).  With few rows (a decode step has Hq of them) the time is the chain of dependent L2 round trips, so
// everything that can be fetched side by side is: the first chunk of partial rows and all of the row's lse_s
// (lane l takes splits l, l + 32, ...) are requested together; the lanes reduce the maximum and the sum, leave
// the normalised weights in shared memory, and the partial rows follow in chunks of kMergeChunk, all loads of a
// chunk issued before the first is used.
__global__ void __launch_bounds__(kMergeThreads) merge_rows_kernel(const __grid_constant__ MergeParams p) {
    __shared__ float weights[kMergeThreads / 32][kMergeMaxParts];
    const int lane = threadIdx.x & 31;
    float* w = weights[threadIdx.x >> 5];
    const int64_t row = static_cast<int64_t>(blockIdx.x) * (kMergeThreads / 32) + (threadIdx.x >> 5);
    const int64_t rows = static_cast<int64_t>(p.Q) * p.Hq;
    if (row >= rows) return;
    const int n = p.n_splits;
    const bool col_ok = lane * 4 < p.d;
    auto load_chunk = [&](int s0, float4 (&o)[kMergeChunk]) {
#pragma unroll
        for (int u = 0; u < kMergeChunk; ++u) {
            o[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (s0 + u < n && col_ok)
                o[u] = __ldcg(reinterpret_cast<const float4*>(p.part_o + ((s0 + u) * rows + row) * p.d) + lane);
        }
    };
    float4 o[kMergeChunk];
    load_chunk(0, o);
    float m = -INFINITY;
    for (int s = lane; s < n; s += 32) {
        const float ls = __ldcg(p.part_lse + s * rows + row);
        w[s] = ls;
        m = fmaxf(m, ls);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
    float l = 0.f;
    for (int s = lane; s < n; s += 32) {
        const float e = (m == -INFINITY) ? 0.f : __expf(w[s] - m);  // exp(-inf) = 0 for an empty split
        w[s] = e;
        l += e;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) l += __shfl_xor_sync(0xffffffffu, l, off);
    __syncwarp();
    const float inv = (l > 0.f) ? 1.f / l : 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s0 = 0; s0 < n; s0 += kMergeChunk) {
        if (s0 > 0) load_chunk(s0, o);
#pragma unroll
        for (int u = 0; u < kMergeChunk; ++u) {
            if (s0 + u >= n) break;
            const float wt = w[s0 + u];
            if (wt == 0.f) continue;  // an empty split's partial row is zero anyway
            acc.x += wt * o[u].x; acc.y += wt * o[u].y; acc.z += wt * o[u].z; acc.w += wt * o[u].w;
        }
    }
    if (col_ok) {
        uint2 out;
        out.x = pack_bf16x2(acc.x * inv, acc.y * inv);
        out.y = pack_bf16x2(acc.z * inv, acc.w * inv);
        reinterpret_cast<uint2*>(p.o + row * p.d)[lane] = out;
    }
    if (p.lse && lane == 0) {
        const int tok = static_cast<int>(row / p.Hq), head = static_cast<int>(row % p.Hq);
        p.lse[static_cast<int64_t>(head) * p.Q + tok] = (l > 0.f) ? m + logf(l) : -INFINITY;
    }
}

cudaError_t launch_merge(const MergeParams& p, cudaStream_t stream) {
    const int64_t rows = static_cast<int64_t>(p.Q) * p.Hq;
    if (rows <= 0) return cudaSuccess;
    const int rows_per_cta = kMergeThreads / 32;
    if (rows <= static_cast<int64_t>(kNumSms) * rows_per_cta && p.n_splits <= kMergeMaxParts) {
        // at most one CTA per SM of warp-per-row work: the latency-oriented form
        merge_rows_kernel<<<static_cast<unsigned>((rows + rows_per_cta - 1) / rows_per_cta), kMergeThreads, 0, stream>>>(p);
    } else {
        const int64_t n = rows * (p.d / 4);
        merge_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, stream>>>(p);
    }
    return cudaGetLastError();
}

}  // namespace pevlm
