// KV-cache assembly (the key/value set s + c_all + q of Eq. 5): a coalesced 16-byte-vector
// copy of up to four segments (K video, K question, V video, V question) into the two
// contiguous caches, one launch.  Pure HBM traffic: reads and writes each byte once.
#include "internal.h"

namespace pevlm {

constexpr int kCopyThreads = 256;
constexpr int kCopyUnroll = 4;

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream(uint4* p, const uint4& v) {
    asm volatile("st.global.L1::no_allocate.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}

__global__ void __launch_bounds__(kCopyThreads) copy_segments_kernel(const __grid_constant__ CopySegments s) {
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kCopyThreads * kCopyUnroll;
    for (int64_t base = static_cast<int64_t>(blockIdx.x) * kCopyThreads * kCopyUnroll + threadIdx.x; base < s.total;
         base += stride) {
        uint4 v[kCopyUnroll];
        uint4* dst[kCopyUnroll];
#pragma unroll
        for (int u = 0; u < kCopyUnroll; ++u) {
            int64_t i = base + static_cast<int64_t>(u) * kCopyThreads;
            dst[u] = nullptr;
            if (i < s.total) {
                int seg = 0;
#pragma unroll
                for (int k = 0; k < 3; ++k) {
                    if (seg == k && i >= s.n_vec[k]) {
                        i -= s.n_vec[k];
                        seg = k + 1;
                    }
                }
                v[u] = ld_stream(s.src[seg] + i);
                dst[u] = s.dst[seg] + i;
            }
        }
#pragma unroll
        for (int u = 0; u < kCopyUnroll; ++u)
            if (dst[u]) st_stream(dst[u], v[u]);
    }
}

cudaError_t launch_copy_segments(const CopySegments& s, cudaStream_t stream) {
    if (s.total <= 0) return cudaSuccess;
    const int64_t per_cta = static_cast<int64_t>(kCopyThreads) * kCopyUnroll;
    int64_t ctas = (s.total + per_cta - 1) / per_cta;
    const int64_t cap = 148 * 16;  // a few waves of the 148 SMs; the loop strides over the rest
    if (ctas > cap) ctas = cap;
    copy_segments_kernel<<<static_cast<unsigned>(ctas), kCopyThreads, 0, stream>>>(s);
    return cudaGetLastError();
}

}  // namespace pevlm
