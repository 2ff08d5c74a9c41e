/*
 * decode_attn_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, fp64 CPU statement of grouped-query single-token ("decode")
 * softmax attention over a paged bf16 KV cache.  It exists so that the CUDA
 * library can be compared with something that is obviously the definition.
 * Only the test-suite, the smoke check and the benchmark's CPU-baseline leg
 * may load it; the product never does, and it shares no source, header, table
 * or helper with the CUDA path.
 *
 * What it follows.  The paper's agent loop spends its run time in calls to a
 * central LLM inference service (Sec. 3.2, "Large-scale runs"; Sec. 4 fixes a
 * 131,072-token context, temperature 1.0 and up to 15 calls x 3 sessions per
 * operator).  The paper gives no internals for that service; its only pointer
 * to attention is the FlashAttention line of work cited under "Kernel
 * Research" (Sec. 5).  Those works reach *exactly* softmax attention by
 * re-associating it (tiling, online softmax, split-K with a log-sum-exp
 * merge), so the oracle is the textbook definition written out, two passes,
 * no tiling, no online rescaling, no splits:
 *
 *   for each sequence b with length L = seq_lens[b] (the current token's K/V
 *   are already in the cache, so the query sits at position L-1):
 *     lo = (window > 0 && window < L) ? L - window : 0
 *     for each query head h, using KV head g = h / (Hq/Hkv):
 *       s_t   = scale * sum_d q[b,h,d] * K[page(t), g, t % P, d]   t in [lo,L)
 *       m     = max_t s_t
 *       Z     = sum_t exp(s_t - m)
 *       out   = sum_t (exp(s_t - m) / Z) * V[page(t), g, t % P, :]
 *       lse   = m + log(Z)                       (natural log, scaled scores)
 *     with page(t) = block_table[b][t / P].
 *   L <= 0 gives out = 0 and lse = -inf.
 *
 * bf16 -> double conversion is exact (the 16 bits are the top half of an
 * IEEE-754 binary32).  Sums run in a fixed order (d ascending, t ascending)
 * so that results are reproducible bit for bit, whatever the thread count.
 *
 * Pins (tests/test_oracle_pins.py): one-token context, identical keys,
 * scale 0, one dominant score, huge score offsets, page permutation, GQA head
 * mapping, window identities, split/merge algebra, dense numpy brute force.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_bits_to_double(uint16_t bits)
{
    uint32_t u = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* Return codes. */
enum { ORACLE_OK = 0, ORACLE_BAD_ARG = 1, ORACLE_BAD_PAGE = 2, ORACLE_NO_MEM = 3 };

/*
 * All pointers are HOST pointers; nothing is retained.
 *   q            bf16 bits, [B, Hq, D] contiguous
 *   k_pages,
 *   v_pages      bf16 bits; element (page, g, r, d) lives at
 *                page*stride_page + g*stride_head + r*stride_tok + d  (elements)
 *   block_table  int32 [B, max_pages] contiguous; only entries with index
 *                < ceil(L/P) are read
 *   seq_lens     int32 [B]
 *   window       <= 0: full attention; else the last `window` tokens
 *   scale        multiplies q.k before the softmax
 *   out          double [B, Hq, D] contiguous
 *   lse          double [B, Hq]    contiguous (may be NULL)
 *   num_threads  <= 0: let OpenMP decide
 */
int decode_attn_oracle(const uint16_t *q, int64_t B, int64_t Hq, int64_t D,
                       const uint16_t *k_pages, const uint16_t *v_pages,
                       int64_t num_pages, int64_t Hkv, int64_t P,
                       int64_t stride_page, int64_t stride_head, int64_t stride_tok,
                       const int32_t *block_table, int64_t max_pages,
                       const int32_t *seq_lens, int32_t window, double scale,
                       double *out, double *lse, int32_t num_threads)
{
    if (!q || !k_pages || !v_pages || !block_table || !seq_lens || !out)
        return ORACLE_BAD_ARG;
    if (B < 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || P <= 0 || Hq % Hkv != 0 || num_pages < 0)
        return ORACLE_BAD_ARG;

    const int64_t G = Hq / Hkv; /* query heads per KV head; consecutive heads share one */
    int status = ORACLE_OK;

#ifdef _OPENMP
    if (num_threads > 0)
        omp_set_num_threads(num_threads);
#else
    (void)num_threads;
#endif

#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t bh = 0; bh < B * Hq; ++bh) {
        const int64_t b = bh / Hq, h = bh % Hq, g = h / G;
        double *o = out + bh * D;
        const int64_t L = seq_lens[b];

        for (int64_t d = 0; d < D; ++d)
            o[d] = 0.0;
        if (L <= 0) {
            if (lse)
                lse[bh] = -INFINITY;
            continue;
        }
        if ((L + P - 1) / P > max_pages) {
#pragma omp atomic write
            status = ORACLE_BAD_ARG;
            continue;
        }
        const int64_t lo = (window > 0 && (int64_t)window < L) ? L - window : 0;
        const int64_t n = L - lo;
        double *s = (double *)malloc((size_t)n * sizeof(double));
        if (!s) {
#pragma omp atomic write
            status = ORACLE_NO_MEM;
            continue;
        }
        const uint16_t *qv = q + bh * D;
        int bad = 0;

        /* pass 1: scores and their maximum */
        double m = -INFINITY;
        for (int64_t t = lo; t < L; ++t) {
            const int64_t page = block_table[b * max_pages + t / P];
            if (page < 0 || page >= num_pages) {
                bad = 1;
                break;
            }
            const uint16_t *kv = k_pages + page * stride_page + g * stride_head + (t % P) * stride_tok;
            double acc = 0.0;
            for (int64_t d = 0; d < D; ++d)
                acc += bf16_bits_to_double(qv[d]) * bf16_bits_to_double(kv[d]);
            s[t - lo] = scale * acc;
            if (s[t - lo] > m)
                m = s[t - lo];
        }
        if (bad) {
#pragma omp atomic write
            status = ORACLE_BAD_PAGE;
            free(s);
            continue;
        }

        /* pass 2: normaliser, then the weighted sum of V rows */
        double Z = 0.0;
        for (int64_t t = lo; t < L; ++t)
            Z += exp(s[t - lo] - m);
        for (int64_t t = lo; t < L; ++t) {
            const int64_t page = block_table[b * max_pages + t / P];
            const uint16_t *vv = v_pages + page * stride_page + g * stride_head + (t % P) * stride_tok;
            const double w = exp(s[t - lo] - m) / Z;
            for (int64_t d = 0; d < D; ++d)
                o[d] += w * bf16_bits_to_double(vv[d]);
        }
        if (lse)
            lse[bh] = m + log(Z);
        free(s);
    }
    return status;
}

/* How many threads a call with num_threads <= 0 would use. */
int decode_attn_oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * kv_append_oracle -- the step that precedes decode attention in each layer of a decoding loop:
 * the new token's key and value rows are written into the paged cache.  seq_lens already counts
 * the new token (the reading taken for decode attention), so the rows go to position L-1:
 * page block_table[b][(L-1)/P], row (L-1) % P, for every KV head.  Sequences with L <= 0 are
 * skipped.  Pure byte moves; HOST pointers; same layout conventions as decode_attn_oracle.
 *   k_new, v_new   bf16 bits [B, Hkv, D] contiguous
 * Returns ORACLE_BAD_PAGE / ORACLE_BAD_ARG if a sequence points outside the pool or its table.
 */
int kv_append_oracle(const uint16_t *k_new, const uint16_t *v_new, int64_t B, int64_t Hkv, int64_t D,
                     uint16_t *k_pages, uint16_t *v_pages, int64_t num_pages, int64_t P,
                     int64_t stride_page, int64_t stride_head, int64_t stride_tok,
                     const int32_t *block_table, int64_t max_pages, const int32_t *seq_lens)
{
    if (!k_new || !v_new || !k_pages || !v_pages || !block_table || !seq_lens)
        return ORACLE_BAD_ARG;
    for (int64_t b = 0; b < B; ++b) {
        const int64_t L = seq_lens[b];
        if (L <= 0)
            continue;
        const int64_t t = L - 1;
        if (t / P >= max_pages)
            return ORACLE_BAD_ARG;
        const int64_t page = block_table[b * max_pages + t / P];
        if (page < 0 || page >= num_pages)
            return ORACLE_BAD_PAGE;
        for (int64_t g = 0; g < Hkv; ++g) {
            const int64_t dst = page * stride_page + g * stride_head + (t % P) * stride_tok;
            const int64_t src = (b * Hkv + g) * D;
            for (int64_t d = 0; d < D; ++d) {
                k_pages[dst + d] = k_new[src + d];
                v_pages[dst + d] = v_new[src + d];
            }
        }
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------
 * The same attention over a KV cache stored in 8 bits per element.
 *
 * The paper is silent on cache precision; the reading taken is the common serving one: K and V
 * are stored as FP8 E4M3 codes (the "E4M3" interchange format of Micikevicius et al., "FP8 Formats
 * for Deep Learning", 2022, Sec. 3 / the OCP 8-bit floating point specification: 1 sign bit, 4
 * exponent bits with bias 7, 3 mantissa bits, no infinities, S.1111.111 is NaN, largest finite
 * value 448, subnormals m/8 * 2^-6), with one fp32 dequantisation factor per KV head:
 *     K[page,g,r,d] = k_scale[g] * e4m3(k_code[page,g,r,d]),   V likewise with v_scale[g].
 * Everything else is the definition at the top of this file.
 * ------------------------------------------------------------------------------------------ */

/* Value of an E4M3 code, from the format's definition. */
double e4m3_bits_to_double(uint8_t code)
{
    const int sign = code >> 7, e = (code >> 3) & 15, m = code & 7;
    double mag;
    if (e == 15 && m == 7)
        return NAN;
    if (e == 0)
        mag = ldexp((double)m / 8.0, -6);              /* subnormal: 0.mmm * 2^(1-bias) */
    else
        mag = ldexp(1.0 + (double)m / 8.0, e - 7);     /* normal:    1.mmm * 2^(e-bias) */
    return sign ? -mag : mag;
}

/*
 * Round a real number to the nearest E4M3 code: ties go to the code with an even mantissa, values
 * beyond +-448 (the largest finite magnitude) saturate to +-448, NaN gives the NaN code 0x7F.
 * Written as a search over the 127 finite non-negative codes, whose values increase with the code.
 */
uint8_t e4m3_nearest_code(double x)
{
    if (isnan(x))
        return 0x7F;
    const uint8_t sign = signbit(x) ? 0x80 : 0x00;
    const double a = fabs(x);
    int best = 0;
    double best_err = fabs(a - e4m3_bits_to_double(0));
    for (int code = 1; code <= 0x7E; ++code) {
        const double err = fabs(a - e4m3_bits_to_double((uint8_t)code));
        if (err < best_err || (err == best_err && (code & 1) == 0)) {
            best = code;
            best_err = err;
        }
    }
    return (uint8_t)(sign | best);
}

/*
 * Quantisation of a cache row: code = nearest_e4m3( x / scale ), where the quotient is taken in
 * fp32 (one correctly rounded IEEE-754 binary32 division of the bf16 value, widened exactly to
 * fp32, by the fp32 factor), the precision in which the CUDA path takes the same decision.
 *   x  bf16 bits [n];  out  uint8 [n]
 */
void e4m3_quantize_oracle(const uint16_t *x, int64_t n, float scale, uint8_t *out)
{
    for (int64_t i = 0; i < n; ++i) {
        const float xf = (float)bf16_bits_to_double(x[i]);
        volatile float y = xf / scale;   /* volatile: keep the quotient a true binary32 */
        out[i] = e4m3_nearest_code((double)y);
    }
}

/*
 * decode_attn_fp8kv_oracle -- arguments as decode_attn_oracle, except
 *   k_pages, v_pages  uint8 E4M3 codes, element (page, g, r, d) at
 *                     page*stride_page + g*stride_head + r*stride_tok + d   (elements = bytes)
 *   k_scale, v_scale  float [Hkv] dequantisation factors (NULL: all 1)
 */
int decode_attn_fp8kv_oracle(const uint16_t *q, int64_t B, int64_t Hq, int64_t D,
                             const uint8_t *k_pages, const uint8_t *v_pages,
                             int64_t num_pages, int64_t Hkv, int64_t P,
                             int64_t stride_page, int64_t stride_head, int64_t stride_tok,
                             const float *k_scale, const float *v_scale,
                             const int32_t *block_table, int64_t max_pages,
                             const int32_t *seq_lens, int32_t window, double scale,
                             double *out, double *lse, int32_t num_threads)
{
    if (!q || !k_pages || !v_pages || !block_table || !seq_lens || !out)
        return ORACLE_BAD_ARG;
    if (B < 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || P <= 0 || Hq % Hkv != 0 || num_pages < 0)
        return ORACLE_BAD_ARG;
    const int64_t G = Hq / Hkv;
    int status = ORACLE_OK;
#ifdef _OPENMP
    if (num_threads > 0)
        omp_set_num_threads(num_threads);
#else
    (void)num_threads;
#endif

#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t bh = 0; bh < B * Hq; ++bh) {
        const int64_t b = bh / Hq, h = bh % Hq, g = h / G;
        double *o = out + bh * D;
        const int64_t L = seq_lens[b];
        const double ks = k_scale ? (double)k_scale[g] : 1.0;
        const double vs = v_scale ? (double)v_scale[g] : 1.0;

        for (int64_t d = 0; d < D; ++d)
            o[d] = 0.0;
        if (L <= 0) {
            if (lse)
                lse[bh] = -INFINITY;
            continue;
        }
        if ((L + P - 1) / P > max_pages) {
#pragma omp atomic write
            status = ORACLE_BAD_ARG;
            continue;
        }
        const int64_t lo = (window > 0 && (int64_t)window < L) ? L - window : 0;
        const int64_t n = L - lo;
        double *s = (double *)malloc((size_t)n * sizeof(double));
        if (!s) {
#pragma omp atomic write
            status = ORACLE_NO_MEM;
            continue;
        }
        const uint16_t *qv = q + bh * D;
        int bad = 0;

        /* pass 1: scores s_t = scale * <q, k_scale * e4m3(k_t)> and their maximum */
        double m = -INFINITY;
        for (int64_t t = lo; t < L; ++t) {
            const int64_t page = block_table[b * max_pages + t / P];
            if (page < 0 || page >= num_pages) {
                bad = 1;
                break;
            }
            const uint8_t *kv = k_pages + page * stride_page + g * stride_head + (t % P) * stride_tok;
            double acc = 0.0;
            for (int64_t d = 0; d < D; ++d)
                acc += bf16_bits_to_double(qv[d]) * (ks * e4m3_bits_to_double(kv[d]));
            s[t - lo] = scale * acc;
            if (s[t - lo] > m)
                m = s[t - lo];
        }
        if (bad) {
#pragma omp atomic write
            status = ORACLE_BAD_PAGE;
            free(s);
            continue;
        }

        /* pass 2: normaliser, then the weighted sum of the dequantised V rows */
        double Z = 0.0;
        for (int64_t t = lo; t < L; ++t)
            Z += exp(s[t - lo] - m);
        for (int64_t t = lo; t < L; ++t) {
            const int64_t page = block_table[b * max_pages + t / P];
            const uint8_t *vv = v_pages + page * stride_page + g * stride_head + (t % P) * stride_tok;
            const double w = exp(s[t - lo] - m) / Z;
            for (int64_t d = 0; d < D; ++d)
                o[d] += w * (vs * e4m3_bits_to_double(vv[d]));
        }
        if (lse)
            lse[bh] = m + log(Z);
        free(s);
    }
    return status;
}

/*
 * kv_append_fp8_oracle -- kv_append_oracle for the 8-bit cache: the new token's bf16 K and V rows
 * are quantised per KV head (e4m3_quantize_oracle with k_scale[g], v_scale[g]; NULL: factor 1)
 * and the codes written to position L-1.
 */
int kv_append_fp8_oracle(const uint16_t *k_new, const uint16_t *v_new, int64_t B, int64_t Hkv, int64_t D,
                         uint8_t *k_pages, uint8_t *v_pages, int64_t num_pages, int64_t P,
                         int64_t stride_page, int64_t stride_head, int64_t stride_tok,
                         const float *k_scale, const float *v_scale,
                         const int32_t *block_table, int64_t max_pages, const int32_t *seq_lens)
{
    if (!k_new || !v_new || !k_pages || !v_pages || !block_table || !seq_lens)
        return ORACLE_BAD_ARG;
    for (int64_t b = 0; b < B; ++b) {
        const int64_t L = seq_lens[b];
        if (L <= 0)
            continue;
        const int64_t t = L - 1;
        if (t / P >= max_pages)
            return ORACLE_BAD_ARG;
        const int64_t page = block_table[b * max_pages + t / P];
        if (page < 0 || page >= num_pages)
            return ORACLE_BAD_PAGE;
        for (int64_t g = 0; g < Hkv; ++g) {
            const int64_t dst = page * stride_page + g * stride_head + (t % P) * stride_tok;
            const int64_t src = (b * Hkv + g) * D;
            e4m3_quantize_oracle(k_new + src, D, k_scale ? k_scale[g] : 1.0f, k_pages + dst);
            e4m3_quantize_oracle(v_new + src, D, v_scale ? v_scale[g] : 1.0f, v_pages + dst);
        }
    }
    return ORACLE_OK;
}
