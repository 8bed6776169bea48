// RoPE at global positions (Sec. 3.2.2): every token keeps its original sequential position.
// HBM-bound elementwise kernel; angle, sine/cosine and rotation in fp64, one rounding
// fp64 -> fp32 -> bf16 (round to nearest even).  No fused multiply-add in the rotation, so
// every fp64 operation rounds exactly once.
#include "internal.h"

namespace pevlm {

constexpr int kRopeThreads = 256;
constexpr int kRopeTokensPerCta = 4;

__device__ __forceinline__ double bf16_bits_to_f64(uint32_t bits16) {
    return static_cast<double>(__uint_as_float(bits16 << 16));
}
__device__ __forceinline__ uint32_t f64_to_bf16_bits(double x) {
    const float f = __double2float_rn(x);
    return static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(f)));
}

// One CTA handles kRopeTokensPerCta consecutive tokens: phase 1 evaluates the d/2 angles of
// each token once (shared by all heads), phase 2 rotates 8 pairs per thread from two 16-byte
// loads (elements i..i+7 and i+d/2..i+d/2+7) and writes two 16-byte stores.
template <int D>
__global__ void __launch_bounds__(kRopeThreads) rope_kernel(const __grid_constant__ RopeParams p) {
    constexpr int HALF = D / 2;
    constexpr int VEC_PER_HEAD = HALF / 8;
    __shared__ double s_cos[kRopeTokensPerCta][HALF];
    __shared__ double s_sin[kRopeTokensPerCta][HALF];

    const int64_t tok0 = static_cast<int64_t>(blockIdx.x) * kRopeTokensPerCta;
    const int ntok = static_cast<int>(min(static_cast<int64_t>(kRopeTokensPerCta), p.n_tokens - tok0));

    for (int idx = threadIdx.x; idx < ntok * HALF; idx += kRopeThreads) {
        const int t = idx / HALF, i = idx % HALF;
        const int64_t pos = p.pos_ids ? static_cast<int64_t>(p.pos_ids[tok0 + t]) : p.first_token + tok0 + t;
        const double ang = __dmul_rn(static_cast<double>(pos), p.inv_freq[i]);
        double s, c;
        sincos(ang, &s, &c);
        s_cos[t][i] = c;
        s_sin[t][i] = s;
    }
    __syncthreads();

    const int heads = p.Hq + p.Hkv;
    const int units_per_tok = heads * VEC_PER_HEAD;
    for (int idx = threadIdx.x; idx < ntok * units_per_tok; idx += kRopeThreads) {
        const int t = idx / units_per_tok;
        const int u = idx % units_per_tok;
        const int h = u / VEC_PER_HEAD;
        const int i0 = (u % VEC_PER_HEAD) * 8;
        const int64_t tok = tok0 + t;
        const __nv_bfloat16* src;
        __nv_bfloat16* dst;
        if (h < p.Hq) {
            const int64_t off = (tok * p.Hq + h) * D;
            src = p.q_in + off;
            dst = p.q_out + off;
        } else {
            const int64_t off = (tok * p.Hkv + (h - p.Hq)) * D;
            src = p.k_in + off;
            dst = p.k_out + off;
        }
        const uint4 lo = *reinterpret_cast<const uint4*>(src + i0);
        const uint4 hi = *reinterpret_cast<const uint4*>(src + i0 + HALF);
        const uint32_t lo_w[4] = {lo.x, lo.y, lo.z, lo.w};
        const uint32_t hi_w[4] = {hi.x, hi.y, hi.z, hi.w};
        uint32_t out_lo[4], out_hi[4];
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            uint32_t ra_bits[2], rb_bits[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int i = i0 + 2 * w + e;
                const double a = bf16_bits_to_f64((lo_w[w] >> (16 * e)) & 0xFFFFu);
                const double b = bf16_bits_to_f64((hi_w[w] >> (16 * e)) & 0xFFFFu);
                const double c = s_cos[t][i], s = s_sin[t][i];
                const double ra = __dsub_rn(__dmul_rn(a, c), __dmul_rn(b, s));
                const double rb = __dadd_rn(__dmul_rn(b, c), __dmul_rn(a, s));
                ra_bits[e] = f64_to_bf16_bits(ra);
                rb_bits[e] = f64_to_bf16_bits(rb);
            }
            out_lo[w] = ra_bits[0] | (ra_bits[1] << 16);
            out_hi[w] = rb_bits[0] | (rb_bits[1] << 16);
        }
        *reinterpret_cast<uint4*>(dst + i0) = make_uint4(out_lo[0], out_lo[1], out_lo[2], out_lo[3]);
        *reinterpret_cast<uint4*>(dst + i0 + HALF) = make_uint4(out_hi[0], out_hi[1], out_hi[2], out_hi[3]);
    }
}

cudaError_t launch_rope(const RopeParams& p, int head_dim, cudaStream_t stream) {
    if (p.n_tokens <= 0 || p.Hq + p.Hkv == 0) return cudaSuccess;
    const unsigned grid = static_cast<unsigned>((p.n_tokens + kRopeTokensPerCta - 1) / kRopeTokensPerCta);
    if (head_dim == 128) {
        rope_kernel<128><<<grid, kRopeThreads, 0, stream>>>(p);
    } else {
        rope_kernel<64><<<grid, kRopeThreads, 0, stream>>>(p);
    }
    return cudaGetLastError();
}

}  // namespace pevlm
