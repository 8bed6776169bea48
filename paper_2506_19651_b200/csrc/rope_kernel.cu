// RoPE at global positions (Sec. 3.2.2): every token keeps its original sequential position.
// HBM-bound elementwise kernel; angle, sine/cosine and rotation in fp64, one rounding
// fp64 -> fp32 -> bf16 (round to nearest even).  No fused multiply-add in the rotation, so
// every fp64 operation rounds exactly once.
#include "internal.h"

namespace pevlm {

constexpr int kRopeThreads = 256;

constexpr int kRopeCtasPerSm = 4;  // resident CTAs per SM of the long-range form (its register budget: 64)

// 16-byte accesses that do not allocate in L1 (every byte is touched once)
__device__ __forceinline__ uint4 ld_stream(const __nv_bfloat16* p) {
    uint4 v;
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream(__nv_bfloat16* p, const uint4& v) {
    asm volatile("st.global.L1::no_allocate.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// bf16 -> fp64 is exact (widen through fp32).
__device__ __forceinline__ double bf16_bits_to_f64(uint32_t bits16) {
    return static_cast<double>(__uint_as_float(bits16 << 16));
}
// fp64 -> fp32 (round to nearest even) -> bf16 (round to nearest even): two roundings, in this order;
// the second one is done for two values at once by the packed conversion
__device__ __forceinline__ uint32_t f64x2_to_bf16x2_bits(double lo, double hi) {
    const float flo = __double2float_rn(lo), fhi = __double2float_rn(hi);
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(fhi), "f"(flo));
    return r;
}

// A SLOT is a group of d/16 threads that handles one token: a thread owns 8 rotation pairs (elements i0..i0+7
// and i0+d/2..i0+d/2+7), evaluates their 8 angles once in fp64 (sincos) and then walks over the token's
// Hq + Hkv head vectors, two 16-byte loads and two 16-byte stores per head; the d/16 threads of a slot read 128
// contiguous bytes per half head vector, the 16 slots of a CTA take 16 neighbouring tokens (a contiguous 256 KB
// at 28/4 heads of 128: slots that each streamed a region of their own ran 25 % slower), and CTAs stride over
// these groups.  The kernel is bound by the bytes it keeps in flight (resident warps x outstanding loads) and
// registers bound the resident warps, so the (cos, sin) pairs sit in a thread-private column of shared memory
// rather than in 32 registers (4 resident CTAs per SM instead of 3) and the loads of the next two heads are
// issued before a head is rotated (template flag LONG).  Short ranges (the question block, a streamed block)
// take the other form, which keeps the pairs in registers, uses no shared memory and fetches one head at a time:
// a launch that uses shared memory made the attention launch that follows two launches later start about 9 us
// later (the SMs change their shared-memory configuration), which a short range cannot pay back.
// No block-level synchronisation.  The heads of a token can be split over
// `head_split` slots, each evaluating the token's angles itself, for short token ranges (the question block),
// so that the launch still fills the machine.
// MODE 0: one position per token.  MODE 1, 2: the multimodal form, where a rotary pair's section picks the
// position component; 1 when the section boundaries are multiples of 8 pairs (16/24/24 at d = 128), so that a
// thread's 8 pairs share one component, 2 in general (a component per pair).
template <int D, int MODE, bool LONG>
__global__ void __launch_bounds__(kRopeThreads, LONG ? kRopeCtasPerSm : 1) rope_kernel(const __grid_constant__ RopeParams p) {
    constexpr int kPrefetch = LONG ? 2 : 0;  // heads whose loads are in flight while one head is rotated
    constexpr int HALF = D / 2;
    constexpr int TPT = HALF / 8;                  // threads per slot
    constexpr int SLOTS_PER_CTA = kRopeThreads / TPT;
    // [pair of the thread][thread]: conflict-free 16-byte accesses (one dummy element in the short form)
    __shared__ double2 cs_sn[LONG ? 8 : 1][LONG ? kRopeThreads : 1];
    double cs[LONG ? 1 : 8], sn[LONG ? 1 : 8];
    const int v = threadIdx.x % TPT;
    const int i0 = v * 8;
    const int heads = p.Hq + p.Hkv;
    const int64_t n_slots = p.n_tokens * p.head_split;
    const int64_t n_groups = (n_slots + SLOTS_PER_CTA - 1) / SLOTS_PER_CTA;
    for (int64_t grp = blockIdx.x; grp < n_groups; grp += gridDim.x) {
        const int64_t slot = grp * SLOTS_PER_CTA + threadIdx.x / TPT;
        if (slot >= n_slots) continue;
        const int64_t tok = slot / p.head_split;
        // this slot's share of the token's heads: a contiguous range
        const int part = static_cast<int>(slot % p.head_split);
        const int h_first = part * heads / p.head_split, h_end = (part + 1) * heads / p.head_split;
        int64_t pos = 0;
        if (MODE == 0) pos = p.pos_ids ? static_cast<int64_t>(p.pos_ids[tok]) : p.first_token + tok;
        if (MODE == 1) {
            const int comp = i0 < p.sec_end0 ? 0 : i0 < p.sec_end1 ? 1 : 2;
            pos = static_cast<int64_t>(p.pos3[comp * p.n_tokens + tok]);
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            int64_t pe = pos;
            if (MODE == 2) {  // multimodal: the pair's section picks the temporal, height or width position
                const int i = i0 + e;
                const int comp = i < p.sec_end0 ? 0 : i < p.sec_end1 ? 1 : 2;
                pe = static_cast<int64_t>(p.pos3[comp * p.n_tokens + tok]);
            }
            const double ang = __dmul_rn(static_cast<double>(pe), p.inv_freq[i0 + e]);
            double sv, cv;
            sincos(ang, &sv, &cv);
            if (LONG) {
                cs_sn[e][threadIdx.x] = make_double2(cv, sv);
            } else {
                cs[e] = cv;
                sn[e] = sv;
            }
        }
        auto addr_of = [&](int h, const __nv_bfloat16*& src, __nv_bfloat16*& dst) {
            if (h < p.Hq) {
                const int64_t off = (tok * p.Hq + h) * D;
                src = p.q_in + off;
                dst = p.q_out + off;
            } else {
                const int64_t off = (tok * p.Hkv + (h - p.Hq)) * D;
                src = p.k_in + off;
                dst = p.k_out + off;
            }
        };
        uint4 lo_q[kPrefetch + 1], hi_q[kPrefetch + 1];
#pragma unroll
        for (int n = 0; n < kPrefetch; ++n) {
            const int h = h_first + n;
            if (h < h_end) {
                const __nv_bfloat16* src;
                __nv_bfloat16* dst;
                addr_of(h, src, dst);
                lo_q[n] = ld_stream(src + i0);
                hi_q[n] = ld_stream(src + i0 + HALF);
            }
        }
        for (int h = h_first; h < h_end; ++h) {
            const __nv_bfloat16* src;
            __nv_bfloat16* dst;
            if (h + kPrefetch < h_end) {
                addr_of(h + kPrefetch, src, dst);
                lo_q[kPrefetch] = ld_stream(src + i0);
                hi_q[kPrefetch] = ld_stream(src + i0 + HALF);
            }
            addr_of(h, src, dst);
            const uint4 lo = lo_q[0], hi = hi_q[0];
#pragma unroll
            for (int n = 0; n < kPrefetch; ++n) {
                lo_q[n] = lo_q[n + 1];
                hi_q[n] = hi_q[n + 1];
            }
            const uint32_t lo_w[4] = {lo.x, lo.y, lo.z, lo.w};
            const uint32_t hi_w[4] = {hi.x, hi.y, hi.z, hi.w};
            uint32_t out_lo[4], out_hi[4];
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                double ra[2], rb[2];
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const double a = bf16_bits_to_f64((lo_w[w] >> (16 * e)) & 0xFFFFu);
                    const double b = bf16_bits_to_f64((hi_w[w] >> (16 * e)) & 0xFFFFu);
                    double c, s;
                    if (LONG) {
                        const double2 t = cs_sn[2 * w + e][threadIdx.x];
                        c = t.x;
                        s = t.y;
                    } else {
                        c = cs[2 * w + e];
                        s = sn[2 * w + e];
                    }
                    ra[e] = __dsub_rn(__dmul_rn(a, c), __dmul_rn(b, s));
                    rb[e] = __dadd_rn(__dmul_rn(b, c), __dmul_rn(a, s));
                }
                out_lo[w] = f64x2_to_bf16x2_bits(ra[0], ra[1]);
                out_hi[w] = f64x2_to_bf16x2_bits(rb[0], rb[1]);
            }
            st_stream(dst + i0, make_uint4(out_lo[0], out_lo[1], out_lo[2], out_lo[3]));
            st_stream(dst + i0 + HALF, make_uint4(out_hi[0], out_hi[1], out_hi[2], out_hi[3]));
        }
    }
}

cudaError_t launch_rope(const RopeParams& p, int head_dim, cudaStream_t stream) {
    if (p.n_tokens <= 0 || p.Hq + p.Hkv == 0) return cudaSuccess;
    const int slots_per_cta = kRopeThreads / (head_dim / 16);
    const int64_t resident = static_cast<int64_t>(kNumSms) * kRopeCtasPerSm;  // CTAs the GPU holds at once
    RopeParams q = p;
    // short ranges: split a token's heads until the launch has about two CTAs per SM
    q.head_split = 1;
    while (q.head_split < 32 && q.head_split * 2 <= p.Hq + p.Hkv && p.n_tokens * q.head_split < 2 * kNumSms * slots_per_cta)
        q.head_split *= 2;
    const int64_t groups = (p.n_tokens * q.head_split + slots_per_cta - 1) / slots_per_cta;
    const int64_t cap = 2 * resident;  // CTAs stride over the remaining groups
    const unsigned grid = static_cast<unsigned>(groups < cap ? groups : cap);
    const int mode = !q.pos3 ? 0 : ((q.sec_end0 | q.sec_end1) & 7) == 0 ? 1 : 2;
    const bool long_range = q.head_split == 1 && groups >= resident;  // at least one full round of resident CTAs
#define PEVLM_ROPE_LAUNCH(D_, M_)                                                                   \
    do {                                                                                            \
        if (long_range) rope_kernel<D_, M_, true><<<grid, kRopeThreads, 0, stream>>>(q);            \
        else rope_kernel<D_, M_, false><<<grid, kRopeThreads, 0, stream>>>(q);                      \
    } while (0)
    if (head_dim == 128) {
        if (mode == 0) PEVLM_ROPE_LAUNCH(128, 0);
        else if (mode == 1) PEVLM_ROPE_LAUNCH(128, 1);
        else PEVLM_ROPE_LAUNCH(128, 2);
    } else {
        if (mode == 0) PEVLM_ROPE_LAUNCH(64, 0);
        else if (mode == 1) PEVLM_ROPE_LAUNCH(64, 1);
        else PEVLM_ROPE_LAUNCH(64, 2);
    }
#undef PEVLM_ROPE_LAUNCH
    return cudaGetLastError();
}

}  // namespace pevlm
