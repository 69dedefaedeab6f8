/*
 * CPU oracle for mixed decode + chunked-prefill paged grouped-query attention.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the CUDA
 * library is checked against.  It shares no code, header, table or helper with
 * the CUDA path, and nothing in the product may call it: only the tests, the
 * smoke check and the benchmark's CPU-baseline leg load it.
 *
 * What it computes.  The paper's decode node builds a mixed prefill/decode batch
 * out of resident decode sequences plus locally queued prefill that reuses a
 * resident prefix (Section 5), issued in bounded units (Section 4.4); prefill
 * materialises KV and decode generates autoregressively (Section 2.1), hence the
 * causal rule.  The paper gives no attention formula (it adds no model kernels,
 * Section 5), so the arithmetic is the textbook definition of softmax attention
 * over a paged cache:
 *
 *   for sequence s, new-token row i in [0, Lq[s]), query head h (full causal attention, no sink):
 *     p = (Lc[s] - Lq[s]) + i                 absolute position of the query token
 *     g = h / (Hq / Hkv)                      KV head serving this query head
 *     k_j, v_j = cache[ block_table[s][j / B] ][ g ][ j % B ]   for j in [0, p]
 *     x_j = scale * sum_d q[d] * k_j[d]
 *     m   = max_j x_j ;  l = sum_j exp(x_j - m)
 *     O   = sum_j exp(x_j - m) * v_j / l ;  lse = m + ln l
 *
 * Everything is evaluated in fp64 from the exact bf16 input values, keys in
 * ascending order, with no blocking, fusion or reordering.
 *
 * Variant (model-specific attention; the paper evaluates GPT-OSS-120B, Section 6.1,
 * without describing its attention, so this is a reading taken from that model's
 * public description): a sliding window and per-head attention sinks.
 *   window W > 0 : the query at position p sees keys j in [max(0, p - W + 1), p]
 *                  (W = 0: every key up to p, as above)
 *   sink s_h     : a per-query-head logit (natural-log units, not multiplied by
 *                  scale) that joins the softmax denominator and carries no value:
 *                    O = sum_j exp(x_j) v_j / (exp(s_h) + sum_j exp(x_j))
 *                    lse = ln(exp(s_h) + sum_j exp(x_j))
 *                  (sinks == NULL: no sink)
 *
 * Variant (deployment precision; the paper leaves the KV precision of its runs unstated, Section 6.1): an fp8
 * KV cache.  Cache elements are e4m3 codes (1 sign, 4 exponent bits with bias 7, 3 mantissa bits, no
 * infinities, 0x7F / 0xFF = NaN, largest finite value 448) with one fp32 scale per KV head:
 *   k_j[d] = e4m3(code) * k_scale[g],  v_j[d] = e4m3(code) * v_scale[g]        (exact in fp64)
 * and the append quantises a new bf16 value x as  code = e4m3_rne_sat((float)x / scale[g]):  an IEEE fp32
 * division, then round-to-nearest-even onto the e4m3 grid with saturation at +-448 - the decision is taken
 * in fp32 on both sides, because it selects an integer code.
 *
 * Pins (tests, CPU only): brute-force dense masked attention on gathered
 * contiguous K/V, the library scaled-dot-product routine on an identity block
 * table, closed forms (Lc = 1, q = 0, constant V, dominant key) and invariants
 * (page permutation, chunking, causal mask, batch order).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* e4m3 code -> value: subnormals m/8 * 2^-6, normals (1 + m/8) * 2^(e-7), code 0x7F / 0xFF is NaN */
static double e4m3_to_f64(uint8_t c)
{
    const int e = (c >> 3) & 15, m = c & 7;
    double v;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) v = ldexp((double)m / 8.0, -6);
    else v = ldexp(1.0 + (double)m / 8.0, e - 7);
    return (c & 0x80) ? -v : v;
}

/* fp32 -> nearest e4m3 code, ties to even, saturating at +-448 (NaN -> 0x7F) */
static uint8_t f32_to_e4m3_sat(float x)
{
    if (isnan(x)) return 0x7F;
    const uint8_t sign = signbit(x) ? 0x80 : 0x00;
    const float a = fabsf(x);
    if (a >= 448.0f) return sign | 0x7E;                    /* 448 = (1 + 6/8) * 2^8, the largest finite value */
    if (a < 0.015625f) {                                    /* below 2^-6: subnormal grid of 2^-9 */
        const int q = (int)rintf(a * 512.0f);               /* exact scaling, then round to nearest even */
        return sign | (uint8_t)q;                           /* q = 8 is the code of 2^-6 itself */
    }
    int ex;
    const float f = frexpf(a, &ex);                         /* a = f * 2^ex, f in [0.5, 1) */
    int e = ex - 1;                                         /* a = (2f) * 2^e, 2f in [1, 2) */
    int q = (int)rintf((2.0f * f - 1.0f) * 8.0f);           /* exact scaling, then round to nearest even */
    if (q == 8) { q = 0; e += 1; }
    if (e + 7 > 15 || (e + 7 == 15 && q == 7)) return sign | 0x7E;
    return sign | (uint8_t)(((e + 7) << 3) | q);
}

static double bf16_to_f64(uint16_t bits)
{
    uint32_t u = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* Locate packed row r: which sequence owns it and which new-token index it is. */
static int find_row(const int32_t *query_len, int32_t num_seqs, int64_t r, int32_t *seq, int32_t *idx)
{
    int64_t at = 0;
    for (int32_t s = 0; s < num_seqs; ++s) {
        if (r < at + query_len[s]) {
            *seq = s;
            *idx = (int32_t)(r - at);
            return 0;
        }
        at += query_len[s];
    }
    return -1;
}

/*
 * rows == NULL: compute all T = sum(query_len) packed rows, outputs indexed by packed row.
 * rows != NULL: compute only rows[0..n_rows), outputs indexed by position in that list.
 * out     [n, Hq, D]  fp64
 * lse     [n, Hq]     fp64 or NULL
 * weights [n, Hq, weights_ld] fp64 or NULL: softmax weights of keys 0..p (rest zero-filled)
 * Returns 0, or a negative code on invalid arguments.
 */
int cf_oracle_mixed_attention(
    const uint16_t *q, const uint16_t *k_cache, const uint16_t *v_cache,
    int64_t k_stride_block, int64_t k_stride_head, int64_t k_stride_token,
    int64_t v_stride_block, int64_t v_stride_head, int64_t v_stride_token,
    const int32_t *block_table, int32_t max_blocks_per_seq,
    const int32_t *context_len, const int32_t *query_len, int32_t num_seqs,
    int32_t num_q_heads, int32_t num_kv_heads, int32_t head_dim, int32_t block_size,
    double scale,
    const int64_t *rows, int64_t n_rows,
    double *out, double *lse, double *weights, int64_t weights_ld,
    int32_t window, const double *sinks /* [num_q_heads] or NULL */,
    int32_t kv_fp8 /* 0: caches hold bf16; 1: e4m3 codes (uint8, strides in bytes) */,
    const double *k_scale, const double *v_scale /* [num_kv_heads] when kv_fp8 */)
{
    if (num_q_heads <= 0 || num_kv_heads <= 0 || num_q_heads % num_kv_heads != 0) return -1;
    if (head_dim <= 0 || block_size <= 0 || num_seqs < 0 || window < 0) return -1;
    if (kv_fp8 && (!k_scale || !v_scale)) return -1;
    const uint8_t *k8 = (const uint8_t *)k_cache, *v8 = (const uint8_t *)v_cache;
    int64_t T = 0;
    for (int32_t s = 0; s < num_seqs; ++s) {
        if (query_len[s] < 0 || query_len[s] > context_len[s]) return -2;
        if ((int64_t)context_len[s] > (int64_t)max_blocks_per_seq * block_size) return -3;
        T += query_len[s];
    }
    const int64_t n = rows ? n_rows : T;
    const int32_t group = num_q_heads / num_kv_heads;
    const int64_t work = n * num_q_heads;
    int bad = 0;

#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t w = 0; w < work; ++w) {
        const int64_t slot = w / num_q_heads;
        const int32_t h = (int32_t)(w % num_q_heads);
        const int64_t r = rows ? rows[slot] : slot;
        int32_t s, i;
        if (find_row(query_len, num_seqs, r, &s, &i) != 0) {
#pragma omp atomic write
            bad = 1;
            continue;
        }
        const int32_t p = context_len[s] - query_len[s] + i;
        const int32_t g = h / group;
        const uint16_t *qrow = q + (r * num_q_heads + h) * (int64_t)head_dim;
        const int32_t *bt = block_table + (int64_t)s * max_blocks_per_seq;

        /* first visible key: 0, or the left edge of the sliding window */
        const int32_t j_lo = (window > 0 && p - window + 1 > 0) ? p - window + 1 : 0;
        const double sink = sinks ? sinks[h] : -INFINITY;

        double *x = (double *)malloc(sizeof(double) * (size_t)(p + 1));
        double m = sink;
        for (int32_t j = j_lo; j <= p; ++j) {
            const int64_t koff = (int64_t)bt[j / block_size] * k_stride_block
                                 + (int64_t)g * k_stride_head + (int64_t)(j % block_size) * k_stride_token;
            double dot = 0.0;
            if (kv_fp8)
                for (int32_t d = 0; d < head_dim; ++d) dot += bf16_to_f64(qrow[d]) * (e4m3_to_f64(k8[koff + d]) * k_scale[g]);
            else
                for (int32_t d = 0; d < head_dim; ++d) dot += bf16_to_f64(qrow[d]) * bf16_to_f64(k_cache[koff + d]);
            x[j] = scale * dot;
            if (x[j] > m) m = x[j];
        }
        double l = 0.0;
        for (int32_t j = j_lo; j <= p; ++j) {
            x[j] = exp(x[j] - m);
            l += x[j];
        }
        if (sinks) l += exp(sink - m);        /* the sink adds to the denominator only */
        double *o = out + (slot * num_q_heads + h) * (int64_t)head_dim;
        for (int32_t d = 0; d < head_dim; ++d) o[d] = 0.0;
        for (int32_t j = j_lo; j <= p; ++j) {
            const int64_t voff = (int64_t)bt[j / block_size] * v_stride_block
                                 + (int64_t)g * v_stride_head + (int64_t)(j % block_size) * v_stride_token;
            if (kv_fp8)
                for (int32_t d = 0; d < head_dim; ++d) o[d] += x[j] * (e4m3_to_f64(v8[voff + d]) * v_scale[g]);
            else
                for (int32_t d = 0; d < head_dim; ++d) o[d] += x[j] * bf16_to_f64(v_cache[voff + d]);
        }
        for (int32_t d = 0; d < head_dim; ++d) o[d] /= l;
        if (lse) lse[slot * num_q_heads + h] = m + log(l);
        if (weights) {
            double *wr = weights + (slot * num_q_heads + h) * weights_ld;
            for (int64_t j = 0; j < weights_ld; ++j) wr[j] = (j >= j_lo && j <= p) ? x[j] / l : 0.0;
        }
        free(x);
    }
    return bad ? -4 : 0;
}

/*
 * Scatter this iteration's new K/V rows into the paged cache: token i of sequence s
 * goes to position P + i, i.e. page block_table[s][(P+i)/B], slot (P+i)%B
 * (prefill "materializes" the KV cache, Section 2.1).  Pure byte copy.
 */
int cf_oracle_kv_append(
    uint16_t *k_cache, uint16_t *v_cache,
    int64_t k_stride_block, int64_t k_stride_head, int64_t k_stride_token,
    int64_t v_stride_block, int64_t v_stride_head, int64_t v_stride_token,
    const uint16_t *k_new, const uint16_t *v_new,
    const int32_t *block_table, int32_t max_blocks_per_seq,
    const int32_t *context_len, const int32_t *query_len, int32_t num_seqs,
    int32_t num_kv_heads, int32_t head_dim, int32_t block_size)
{
    int64_t row = 0;
    for (int32_t s = 0; s < num_seqs; ++s) {
        if (query_len[s] < 0 || query_len[s] > context_len[s]) return -2;
        if ((int64_t)context_len[s] > (int64_t)max_blocks_per_seq * block_size) return -3;
        const int32_t prefix = context_len[s] - query_len[s];
        const int32_t *bt = block_table + (int64_t)s * max_blocks_per_seq;
        for (int32_t i = 0; i < query_len[s]; ++i, ++row) {
            const int32_t pos = prefix + i;
            const int64_t blk = bt[pos / block_size];
            const int64_t slot = pos % block_size;
            for (int32_t g = 0; g < num_kv_heads; ++g) {
                const int64_t src = (row * num_kv_heads + g) * (int64_t)head_dim;
                memcpy(k_cache + blk * k_stride_block + g * k_stride_head + slot * k_stride_token,
                       k_new + src, sizeof(uint16_t) * (size_t)head_dim);
                memcpy(v_cache + blk * v_stride_block + g * v_stride_head + slot * v_stride_token,
                       v_new + src, sizeof(uint16_t) * (size_t)head_dim);
            }
        }
    }
    return 0;
}

/*
 * The same scatter into an fp8 cache: every new bf16 value x of KV head g is stored as
 * e4m3_rne_sat((float)x / scale[g]) (see the header).  Caches are uint8, strides in bytes.
 */
int cf_oracle_kv_append_fp8(
    uint8_t *k_cache, uint8_t *v_cache,
    int64_t k_stride_block, int64_t k_stride_head, int64_t k_stride_token,
    int64_t v_stride_block, int64_t v_stride_head, int64_t v_stride_token,
    const uint16_t *k_new, const uint16_t *v_new,
    const int32_t *block_table, int32_t max_blocks_per_seq,
    const int32_t *context_len, const int32_t *query_len, int32_t num_seqs,
    int32_t num_kv_heads, int32_t head_dim, int32_t block_size,
    const float *k_scale, const float *v_scale)
{
    int64_t row = 0;
    for (int32_t s = 0; s < num_seqs; ++s) {
        if (query_len[s] < 0 || query_len[s] > context_len[s]) return -2;
        if ((int64_t)context_len[s] > (int64_t)max_blocks_per_seq * block_size) return -3;
        const int32_t prefix = context_len[s] - query_len[s];
        const int32_t *bt = block_table + (int64_t)s * max_blocks_per_seq;
        for (int32_t i = 0; i < query_len[s]; ++i, ++row) {
            const int32_t pos = prefix + i;
            const int64_t blk = bt[pos / block_size];
            const int64_t slot = pos % block_size;
            for (int32_t g = 0; g < num_kv_heads; ++g) {
                const int64_t src = (row * num_kv_heads + g) * (int64_t)head_dim;
                uint8_t *kd = k_cache + blk * k_stride_block + g * k_stride_head + slot * k_stride_token;
                uint8_t *vd = v_cache + blk * v_stride_block + g * v_stride_head + slot * v_stride_token;
                for (int32_t d = 0; d < head_dim; ++d) {
                    const float kx = (float)bf16_to_f64(k_new[src + d]), vx = (float)bf16_to_f64(v_new[src + d]);
                    kd[d] = f32_to_e4m3_sat(kx / k_scale[g]);
                    vd[d] = f32_to_e4m3_sat(vx / v_scale[g]);
                }
            }
        }
    }
    return 0;
}

/* the two conversions on their own, for the tests that pin them */
void cf_oracle_e4m3_decode(const uint8_t *codes, int64_t n, double *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = e4m3_to_f64(codes[i]);
}
void cf_oracle_e4m3_encode(const float *x, int64_t n, uint8_t *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = f32_to_e4m3_sat(x[i]);
}

int cf_oracle_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp master
        n = omp_get_num_threads();
    }
#endif
    return n;
}
