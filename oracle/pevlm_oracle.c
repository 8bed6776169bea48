/*
 * CPU oracle for PEVLM prefill attention.  TEST INFRASTRUCTURE ONLY: the product path
 * (the CUDA library) never links, imports or calls anything in this directory; only
 * tests, the smoke check and the benchmark's cpu_baseline / reference legs do.
 *
 * Plain, slow, obviously-correct fp64 evaluation of the definition, written from the
 * paper's statement of the method.  It shares no code, header, table or constant with
 * the CUDA path.
 *
 * What it computes, with the passages it follows:
 *   - Token stream [sink | c_0 .. c_{N-1} | question], lengths S, B, N, Q,
 *     L = S + N*B + Q                                           (Sec. 3.2.1, Sec. 3.2.3)
 *   - Sequential position embedding: every token keeps its original global position,
 *     RoPE is applied there and never re-encoded per block             (Sec. 3.2.2)
 *   - f(Q,K,V) = softmax(Q K^T / sqrt(d)) V                                  (Eq. 1)
 *   - Attn_s   = f(Q_s, K_s, V_s)            causal inside the sink          (Eq. 3)
 *   - Attn_c_i = f(Q_c_i, K_{s + c_i}, ..)   all sink keys + own block, causal
 *                inside the block (Eq. 4 read with Eq. 8's count 2HB(S+B))
 *   - Attn_q   = f(Q_q, K_{s + c_all + q}, ..) causal inside the question    (Eq. 5)
 *   - the sink's K/V are computed once and shared by every block       (Sec. 1, 3.1)
 *   - LSE merge of key-range partials (an implementation device for Eq. 5; it is exact
 *     algebra on the softmax of Eq. 1)
 *
 * Readings taken where the paper is silent (all listed in the design notes):
 *   causal everywhere with the diagonal included; RoPE pairs (i, i+d/2) ("rotate
 *   half"); exact fp64 cos/sin; ONE rounding of roped Q/K to bf16 (fp64 -> fp32 RNE ->
 *   bf16 RNE) because the paper's system is bf16 end to end (Sec. 4 setup); GQA maps
 *   q head h to kv head h / (Hq/Hkv); LSE is the natural log of the sum of
 *   exp(scaled scores).
 *
 * Pins (tests/test_oracle_pins.py): brute-force dense causal attention when N <= 1,
 * sink rows == full-attention rows, softmax weights sum to 1, block-permutation
 * invariance with carried positions, closed forms with K = 0 (LSE = ln #visible,
 * O = prefix mean of V), Eq. 10's pair count, RoPE closed forms (position 0 identity,
 * norm preservation, relative-position property), the bf16 rounding on hand-worked bit
 * patterns (round up, round down, ties to even both ways, the two-step case), merge ==
 * unsplit, and a literal pure-Python triple loop on tiny shapes.
 *
 * Build: gcc -O2 -ffp-contract=off -fopenmp -shared -fPIC (see oracle/build.py).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int64_t S, B, N, Q;   /* sink, block length, number of blocks, question length */
    int32_t Hq, Hkv, d;
    int32_t full_causal;  /* 0: PEVLM mask (Eq. 3-5); 1: plain causal attention (Eq. 1-2) */
    int64_t B_last;       /* length of the last context block, 1 <= B_last <= B; 0 means B.  Sec. 3.2.1
                             partitions the video uniformly and does not say what happens to a remainder:
                             here the remainder forms one shorter last block */
} oracle_shape_t;

/* number of video tokens: sink + all context blocks */
static int64_t video_len(const oracle_shape_t* sh) {
    if (sh->N <= 0) return sh->S;
    return sh->S + (sh->N - 1) * sh->B + (sh->B_last > 0 ? sh->B_last : sh->B);
}

static double bf16_to_f64(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* fp64 -> fp32 (round to nearest even, done by the cast) -> bf16 (round to nearest even) */
static uint16_t f64_to_bf16(double x) {
    float f = (float)x;
    uint32_t u;
    memcpy(&u, &f, 4);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

/* The rounding R1 as a scalar, so that it can be pinned with hand-worked bit patterns. */
uint16_t oracle_round_bf16(double x) { return f64_to_bf16(x); }

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Threads for the following calls from this host thread (a launcher may have pinned OMP_NUM_THREADS to 1). */
void oracle_set_num_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/*
 * Visible key ranges of query row t (Eq. 3-5).  Returns the number of ranges (1 or 2);
 * range r is [lo[r], hi[r]) in global token indices.
 */
int oracle_visible(const oracle_shape_t* sh, int64_t t, int64_t lo[2], int64_t hi[2]) {
    int64_t nv = video_len(sh);
    if (sh->full_causal || t < sh->S || t >= nv) {
        /* sink rows (Eq. 3) and question rows (Eq. 5): every key up to and including t */
        lo[0] = 0; hi[0] = t + 1;
        return 1;
    }
    /* row of context block b (Eq. 4): the whole sink, then its own block up to t */
    int64_t b = (t - sh->S) / sh->B;
    lo[0] = 0;                 hi[0] = sh->S;
    lo[1] = sh->S + b * sh->B; hi[1] = t + 1;
    return 2;
}

/*
 * RoPE at given positions (Sec. 3.2.2), rotate-half pairing, fp64, then one rounding to
 * bf16.  x: [n_tokens, heads, d] bf16 bits.  Position of token i is pos[i] if pos != NULL,
 * else first_pos + i.  out_bits (bf16) and/or out_f64 (before the rounding) may be NULL.
 */
void oracle_rope(const uint16_t* x, int64_t n_tokens, int32_t heads, int32_t d, double theta,
                 const int64_t* pos, int64_t first_pos, uint16_t* out_bits, double* out_f64) {
    int32_t half = d / 2;
    double* inv_freq = (double*)malloc(sizeof(double) * (size_t)half);
    for (int32_t i = 0; i < half; ++i) inv_freq[i] = pow(theta, -2.0 * (double)i / (double)d);
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < n_tokens; ++t) {
        double p = (double)(pos ? pos[t] : first_pos + t);
        for (int32_t h = 0; h < heads; ++h) {
            const uint16_t* xr = x + ((size_t)t * heads + h) * d;
            for (int32_t i = 0; i < half; ++i) {
                double ang = p * inv_freq[i];
                double c = cos(ang), s = sin(ang);
                double a = bf16_to_f64(xr[i]);
                double b = bf16_to_f64(xr[i + half]);
                double ra = a * c - b * s;
                double rb = b * c + a * s;
                size_t o = ((size_t)t * heads + h) * d;
                if (out_f64) { out_f64[o + i] = ra; out_f64[o + i + half] = rb; }
                if (out_bits) { out_bits[o + i] = f64_to_bf16(ra); out_bits[o + i + half] = f64_to_bf16(rb); }
            }
        }
    }
    free(inv_freq);
}

/*
 * Multimodal RoPE (the position embedding of the Qwen2-VL family the paper evaluates, Sec. 3.1: positions
 * carry temporal and spatial components).  Each token has three position components pos3[c][t], c = 0
 * temporal, 1 height, 2 width; rotary pair i uses component 0 for i < sec[0], component 1 for the next
 * sec[1] pairs and component 2 for the rest (sec[0] + sec[1] + sec[2] = d/2).  Everything else as
 * oracle_rope: rotate-half pairing, fp64, one rounding to bf16.  With three equal components it is
 * oracle_rope.
 */
void oracle_rope_mrope(const uint16_t* x, int64_t n_tokens, int32_t heads, int32_t d, double theta,
                       const int64_t* pos3, const int32_t* sec, uint16_t* out_bits, double* out_f64) {
    int32_t half = d / 2;
    double* inv_freq = (double*)malloc(sizeof(double) * (size_t)half);
    for (int32_t i = 0; i < half; ++i) inv_freq[i] = pow(theta, -2.0 * (double)i / (double)d);
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < n_tokens; ++t) {
        for (int32_t h = 0; h < heads; ++h) {
            const uint16_t* xr = x + ((size_t)t * heads + h) * d;
            for (int32_t i = 0; i < half; ++i) {
                int c = (i < sec[0]) ? 0 : (i < sec[0] + sec[1]) ? 1 : 2;
                double p = (double)pos3[(size_t)c * n_tokens + t];
                double ang = p * inv_freq[i];
                double co = cos(ang), si = sin(ang);
                double a = bf16_to_f64(xr[i]);
                double b = bf16_to_f64(xr[i + half]);
                double ra = a * co - b * si;
                double rb = b * co + a * si;
                size_t o = ((size_t)t * heads + h) * d;
                if (out_f64) { out_f64[o + i] = ra; out_f64[o + i + half] = rb; }
                if (out_bits) { out_bits[o + i] = f64_to_bf16(ra); out_bits[o + i + half] = f64_to_bf16(rb); }
            }
        }
    }
    free(inv_freq);
}

/*
 * Masked softmax attention (Eq. 1 under the masks of Eq. 3-5) for a list of query rows,
 * all q heads.  q: [L,Hq,d], k,v: [L,Hkv,d], bf16 bits, q and k already roped.
 * rows[n_rows]: global token indices.  o: [n_rows,Hq,d] fp64, lse: [n_rows,Hq] fp64.
 * If key_lo/key_hi >= 0 the visible set is further intersected with [key_lo, key_hi)
 * (used to produce key-range partials for the merge pin); a row with no visible key in
 * the range gets lse = -inf and o = 0.  scale <= 0 means 1/sqrt(d).
 */
void oracle_attn_rows(const oracle_shape_t* sh, const uint16_t* q, const uint16_t* k,
                      const uint16_t* v, double scale, const int64_t* rows, int64_t n_rows,
                      int64_t key_lo, int64_t key_hi, double* o, double* lse) {
    const int32_t d = sh->d, Hq = sh->Hq, Hkv = sh->Hkv;
    const int32_t G = Hq / Hkv;
    if (scale <= 0.0) scale = 1.0 / sqrt((double)d);
    const int64_t L = video_len(sh) + sh->Q;
    int64_t work = n_rows * Hq;
#pragma omp parallel
    {
        double* s = (double*)malloc(sizeof(double) * (size_t)(L > 0 ? L : 1));
        double* qf = (double*)malloc(sizeof(double) * (size_t)d);
#pragma omp for schedule(dynamic, 1)
        for (int64_t w = 0; w < work; ++w) {
            int64_t ri = w / Hq;
            int32_t h = (int32_t)(w % Hq);
            int32_t g = h / G;
            int64_t t = rows[ri];
            int64_t lo[2], hi[2];
            int nr = oracle_visible(sh, t, lo, hi);
            for (int32_t c = 0; c < d; ++c) qf[c] = bf16_to_f64(q[((size_t)t * Hq + h) * d + c]);
            /* scores of the visible keys, in key order */
            int64_t n = 0;
            double m = -INFINITY;
            for (int r = 0; r < nr; ++r) {
                int64_t a = lo[r], e = hi[r];
                if (key_lo >= 0 && a < key_lo) a = key_lo;
                if (key_hi >= 0 && e > key_hi) e = key_hi;
                for (int64_t j = a; j < e; ++j) {
                    const uint16_t* kr = k + ((size_t)j * Hkv + g) * d;
                    double acc = 0.0;
                    for (int32_t c = 0; c < d; ++c) acc += qf[c] * bf16_to_f64(kr[c]);
                    acc *= scale;
                    s[n++] = acc;
                    if (acc > m) m = acc;
                }
            }
            double* orow = o + ((size_t)ri * Hq + h) * d;
            for (int32_t c = 0; c < d; ++c) orow[c] = 0.0;
            if (n == 0) { lse[(size_t)ri * Hq + h] = -INFINITY; continue; }
            double l = 0.0;
            for (int64_t i = 0; i < n; ++i) l += exp(s[i] - m);
            double row_lse = m + log(l);
            lse[(size_t)ri * Hq + h] = row_lse;
            int64_t i = 0;
            for (int r = 0; r < nr; ++r) {
                int64_t a = lo[r], e = hi[r];
                if (key_lo >= 0 && a < key_lo) a = key_lo;
                if (key_hi >= 0 && e > key_hi) e = key_hi;
                for (int64_t j = a; j < e; ++j, ++i) {
                    double wgt = exp(s[i] - row_lse);
                    const uint16_t* vr = v + ((size_t)j * Hkv + g) * d;
                    for (int32_t c = 0; c < d; ++c) orow[c] += wgt * bf16_to_f64(vr[c]);
                }
            }
        }
        free(s);
        free(qf);
    }
}

/*
 * Softmax weights of one (row, head): w[j] for every j in [0, L), 0 where masked.
 * Used by the invariants (weights sum to 1, no weight across two context blocks).
 */
void oracle_weights_row(const oracle_shape_t* sh, const uint16_t* q, const uint16_t* k,
                        double scale, int64_t t, int32_t h, double* w) {
    const int32_t d = sh->d, Hq = sh->Hq, Hkv = sh->Hkv;
    const int32_t g = h / (Hq / Hkv);
    if (scale <= 0.0) scale = 1.0 / sqrt((double)d);
    const int64_t L = video_len(sh) + sh->Q;
    for (int64_t j = 0; j < L; ++j) w[j] = 0.0;
    int64_t lo[2], hi[2];
    int nr = oracle_visible(sh, t, lo, hi);
    double m = -INFINITY;
    for (int r = 0; r < nr; ++r)
        for (int64_t j = lo[r]; j < hi[r]; ++j) {
            double acc = 0.0;
            for (int32_t c = 0; c < d; ++c)
                acc += bf16_to_f64(q[((size_t)t * Hq + h) * d + c]) * bf16_to_f64(k[((size_t)j * Hkv + g) * d + c]);
            w[j] = acc * scale;
            if (w[j] > m) m = w[j];
        }
    double l = 0.0;
    for (int r = 0; r < nr; ++r)
        for (int64_t j = lo[r]; j < hi[r]; ++j) l += exp(w[j] - m);
    double row_lse = m + log(l);
    for (int r = 0; r < nr; ++r)
        for (int64_t j = lo[r]; j < hi[r]; ++j) w[j] = exp(w[j] - row_lse);
}

/*
 * Merge of key-range partials: given n_splits partial (o_s, lse_s) of the same rows,
 * each normalised inside its own key range, the whole-range result is
 *   lse = log sum_s exp(lse_s),  o = sum_s exp(lse_s - lse) o_s.
 * o_parts: [n_splits, n, d], lse_parts: [n_splits, n]; a split with lse = -inf (no
 * visible key) contributes nothing.
 */
void oracle_merge_lse(const double* o_parts, const double* lse_parts, int64_t n_splits,
                      int64_t n, int32_t d, double* o, double* lse) {
    for (int64_t r = 0; r < n; ++r) {
        double m = -INFINITY;
        for (int64_t s = 0; s < n_splits; ++s)
            if (lse_parts[s * n + r] > m) m = lse_parts[s * n + r];
        for (int32_t c = 0; c < d; ++c) o[r * d + c] = 0.0;
        if (m == -INFINITY) { lse[r] = -INFINITY; continue; }
        double l = 0.0;
        for (int64_t s = 0; s < n_splits; ++s) l += exp(lse_parts[s * n + r] - m);
        double tot = m + log(l);
        lse[r] = tot;
        for (int64_t s = 0; s < n_splits; ++s) {
            double ls = lse_parts[s * n + r];
            if (ls == -INFINITY) continue;
            double wgt = exp(ls - tot);
            for (int32_t c = 0; c < d; ++c) o[r * d + c] += wgt * o_parts[(s * n + r) * d + c];
        }
    }
}

/*
 * KV-cache assembly (the key/value set of Eq. 5): the cache row of global token t is
 * the video tensor's row t for t < S + N*B, else the question tensor's row t - (S+N*B).
 * row_elems = Hkv * d.
 */
void oracle_assemble_kv(const oracle_shape_t* sh, const uint16_t* video, const uint16_t* question,
                        uint16_t* cache) {
    int64_t nv = video_len(sh);
    size_t row = (size_t)sh->Hkv * sh->d;
    for (int64_t t = 0; t < nv + sh->Q; ++t) {
        const uint16_t* src = (t < nv) ? video + (size_t)t * row : question + (size_t)(t - nv) * row;
        for (size_t c = 0; c < row; ++c) cache[(size_t)t * row + c] = src[c];
    }
}

/*
 * Count of (row, key) pairs per head when the causal cut inside a row's own segment is
 * ignored (every row of a segment sees the segment's whole key set): the rectangular
 * count that the paper's operation model uses (Eq. 6-10).
 */
int64_t oracle_count_rect_pairs(const oracle_shape_t* sh) {
    int64_t nv = video_len(sh), L = nv + sh->Q, total = 0;
    for (int64_t t = 0; t < L; ++t) {
        int64_t lo[2], hi[2];
        int nr = oracle_visible(sh, t, lo, hi);
        int64_t seg_end = (t < sh->S) ? sh->S : (t < nv) ? sh->S + ((t - sh->S) / sh->B + 1) * sh->B : L;
        if (t < nv && seg_end > nv) seg_end = nv;  /* shorter last block */
        hi[nr - 1] = seg_end;
        for (int r = 0; r < nr; ++r) total += hi[r] - lo[r];
    }
    return total;
}

/* Count of visible (row, key) pairs per head, by enumeration of the mask. */
int64_t oracle_count_pairs(const oracle_shape_t* sh) {
    int64_t L = video_len(sh) + sh->Q, total = 0;
    for (int64_t t = 0; t < L; ++t) {
        int64_t lo[2], hi[2];
        int nr = oracle_visible(sh, t, lo, hi);
        for (int r = 0; r < nr; ++r) total += hi[r] - lo[r];
    }
    return total;
}
