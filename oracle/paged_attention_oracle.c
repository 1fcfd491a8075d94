/*
 * CPU oracle for decode-step attention over a paged KV cache.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the CUDA
 * path is judged against; the product never links, imports or calls it, and
 * it shares no code, header, table or constant with the CUDA sources.
 *
 * What it computes (Section 3.1 and Algorithm 1 step 2 of the paper: one
 * query row per sequence attends over that sequence's resident KV through the
 * page mappings; the row's own K/V was written before attention, so all
 * seq_len cached tokens are attended and there is no causal mask).  The
 * paper does not restate the attention formula; it is the textbook scaled
 * dot-product softmax attention with grouped-query heads:
 *
 *   g      = h / (Hq / Hkv)                      consecutive query heads share a KV head
 *   page   = block_table[b][t / P],  slot = t % P           (Invariant 2: page mappings)
 *   s_t    = scale * sum_d q[b][h][d] * K[page][slot][g][d]
 *   m      = max_t s_t,  p_t = exp(s_t - m),  l = sum_t p_t
 *   out[d] = (sum_t p_t * V[page][slot][g][d]) / l,   lse = m + log(l)
 *
 * Two passes, ascending t, fp64 throughout (bf16 -> fp64 and fp16 -> fp64 are exact).  A row
 * with seq_len 0, or a row whose RUN mask byte is 0 (a Project-Only row of
 * Algorithm 1 step 2), reads no KV and emits zeros, lse = -inf.
 *
 * Also here: the own-layer KV write that precedes attention (Invariant 1),
 * a byte copy pinned in tests/test_oracle_pins.py by reading the rows back.
 *
 * Parity status: the paper prints no attention values, so the numerics are
 * "unpinned by the paper"; the functions below are pinned instead by
 * brute-force dense attention, closed forms, invariants and a library
 * cross-check in tests/test_oracle_pins.py.  The zero output of masked rows
 * and the per-token byte count are the paper-pinned facts.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_bits_to_f64(uint16_t bits)
{
    uint32_t u = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* IEEE binary16: 1 sign, 5 exponent (bias 15), 10 fraction bits; exact in fp64. */
static double fp16_bits_to_f64(uint16_t bits)
{
    const int sign = bits >> 15, e = (bits >> 10) & 31, m = bits & 1023;
    double v;
    if (e == 0)
        v = ldexp((double)m, -24);                      /* subnormal: m / 1024 * 2^-14 */
    else if (e == 31)
        v = m ? NAN : INFINITY;
    else
        v = ldexp(1.0 + (double)m / 1024.0, e - 15);
    return sign ? -v : v;
}

typedef struct {
    int32_t batch, num_q_heads, num_kv_heads, head_dim, page_size, max_pages_per_seq;
    int64_t k_stride_page, k_stride_token, k_stride_head;   /* elements */
    int64_t v_stride_page, v_stride_token, v_stride_head;
    int32_t in_fp16;   /* q, K and V are fp16 bit patterns (the paper serves Llama in fp16 and Qwen in
                          bf16, Section 4.1); 0: bf16 */
    int32_t pad;
} oracle_shape_t;

static double in_bits_to_f64(const oracle_shape_t *s, uint16_t bits)
{
    return s->in_fp16 ? fp16_bits_to_f64(bits) : bf16_bits_to_f64(bits);
}

int oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* The input decoding by itself: n 16-bit patterns to fp64 (pinned against a
 * library's view of the same bits in tests/test_oracle_pins.py). */
int oracle_decode_bits(int in_fp16, const uint16_t *bits, int64_t n, double *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = in_fp16 ? fp16_bits_to_f64(bits[i]) : bf16_bits_to_f64(bits[i]);
    return 0;
}

/* Address of row (token t, kv head g) of sequence b in a pool, in elements. */
static int64_t row_offset(const oracle_shape_t *s, const int32_t *block_table, int b, int t, int g,
                          int64_t stride_page, int64_t stride_token, int64_t stride_head)
{
    int64_t page = block_table[(int64_t)b * s->max_pages_per_seq + t / s->page_size];
    int slot = t % s->page_size;
    return page * stride_page + slot * stride_token + g * stride_head;
}

/* Attention of one (sequence, query head) over tokens [t_begin, t_end).
 * Writes the normalised output (o, length D), the maximum logit m and the
 * sum of exponentials l.  An empty range gives o = 0, m = -inf, l = 0.
 * probs_or_null, if given, receives p_t / l for every token of the range. */
static void attend_range(const oracle_shape_t *s, const uint16_t *q, const uint16_t *k_pool,
                         const uint16_t *v_pool, const int32_t *block_table, double scale, int b, int h,
                         int t_begin, int t_end, double *o, double *m_out, double *l_out,
                         double *probs_or_null)
{
    const int D = s->head_dim;
    const int g = h / (s->num_q_heads / s->num_kv_heads);
    const int n = t_end - t_begin;
    for (int d = 0; d < D; ++d) o[d] = 0.0;
    if (n <= 0) {
        *m_out = -INFINITY;
        *l_out = 0.0;
        return;
    }
    double *logit = (double *)malloc(sizeof(double) * (size_t)n);
    const uint16_t *qrow = q + ((int64_t)b * s->num_q_heads + h) * D;
    double m = -INFINITY;
    for (int t = t_begin; t < t_end; ++t) {
        const uint16_t *krow = k_pool + row_offset(s, block_table, b, t, g, s->k_stride_page,
                                                   s->k_stride_token, s->k_stride_head);
        double dot = 0.0;
        for (int d = 0; d < D; ++d) dot += in_bits_to_f64(s, qrow[d]) * in_bits_to_f64(s, krow[d]);
        logit[t - t_begin] = scale * dot;
        if (logit[t - t_begin] > m) m = logit[t - t_begin];
    }
    double l = 0.0;
    for (int t = t_begin; t < t_end; ++t) {
        const uint16_t *vrow = v_pool + row_offset(s, block_table, b, t, g, s->v_stride_page,
                                                   s->v_stride_token, s->v_stride_head);
        double p = exp(logit[t - t_begin] - m);
        l += p;
        for (int d = 0; d < D; ++d) o[d] += p * in_bits_to_f64(s, vrow[d]);
        if (probs_or_null) probs_or_null[t - t_begin] = p;
    }
    for (int d = 0; d < D; ++d) o[d] /= l;
    if (probs_or_null)
        for (int i = 0; i < n; ++i) probs_or_null[i] /= l;
    *m_out = m;
    *l_out = l;
    free(logit);
}

/* Whole-batch decode attention.  out [B,Hq,D] and lse [B,Hq] are fp64.
 * run_mask_or_null [B]: byte 0 marks a row that reads nothing and emits zero.
 * num_threads <= 0 uses every core OpenMP offers.  Returns 0. */
int oracle_paged_decode_attention(const oracle_shape_t *s, const uint16_t *q, const uint16_t *k_pool,
                                  const uint16_t *v_pool, const int32_t *block_table,
                                  const int32_t *seq_lens, const uint8_t *run_mask_or_null,
                                  double scale, double *out, double *lse, int num_threads)
{
    const int B = s->batch, Hq = s->num_q_heads, D = s->head_dim;
#ifdef _OPENMP
    if (num_threads <= 0) num_threads = omp_get_max_threads();
#else
    (void)num_threads;
#endif
#pragma omp parallel for collapse(2) schedule(dynamic, 1) num_threads(num_threads)
    for (int b = 0; b < B; ++b) {
        for (int h = 0; h < Hq; ++h) {
            double *o = out + ((int64_t)b * Hq + h) * D;
            int L = seq_lens[b];
            if (run_mask_or_null && run_mask_or_null[b] == 0) L = 0;
            double m, l;
            attend_range(s, q, k_pool, v_pool, block_table, scale, b, h, 0, L, o, &m, &l, NULL);
            if (lse) lse[(int64_t)b * Hq + h] = (L > 0) ? m + log(l) : -INFINITY;
        }
    }
    return 0;
}

/* Attention of one (b, h) restricted to tokens [t_begin, t_end): the quantity
 * one split-KV partition contributes (normalised o, its m and l). */
int oracle_partial_attention(const oracle_shape_t *s, const uint16_t *q, const uint16_t *k_pool,
                             const uint16_t *v_pool, const int32_t *block_table, double scale, int b,
                             int h, int t_begin, int t_end, double *o, double *m, double *l)
{
    attend_range(s, q, k_pool, v_pool, block_table, scale, b, h, t_begin, t_end, o, m, l, NULL);
    return 0;
}

/* Softmax probabilities of one (b, h) over its whole sequence: probs [L]. */
int oracle_attention_probs(const oracle_shape_t *s, const uint16_t *q, const uint16_t *k_pool,
                           const uint16_t *v_pool, const int32_t *block_table, const int32_t *seq_lens,
                           double scale, int b, int h, double *probs)
{
    double m, l;
    double *o = (double *)malloc(sizeof(double) * (size_t)s->head_dim);
    attend_range(s, q, k_pool, v_pool, block_table, scale, b, h, 0, seq_lens[b], o, &m, &l, probs);
    free(o);
    return 0;
}

/* Log-sum-exp merge of n partial results of one (b, h), in ascending order:
 *   M = max_i m_i;  w_i = exp(m_i - M) * l_i;  out = sum_i w_i o_i / sum_i w_i;
 *   lse = M + log(sum_i w_i).
 * o_parts [n][D] are normalised partial outputs.  Partitions with l = 0
 * (m = -inf) weigh exactly 0; if every partition is empty the result is
 * zeros with lse = -inf. */
int oracle_merge_partials(int n, int D, const double *o_parts, const double *m_parts,
                          const double *l_parts, double *out, double *lse)
{
    double M = -INFINITY;
    for (int i = 0; i < n; ++i)
        if (l_parts[i] > 0.0 && m_parts[i] > M) M = m_parts[i];
    for (int d = 0; d < D; ++d) out[d] = 0.0;
    if (M == -INFINITY) {
        if (lse) *lse = -INFINITY;
        return 0;
    }
    double wsum = 0.0;
    for (int i = 0; i < n; ++i) {
        if (!(l_parts[i] > 0.0)) continue;
        double w = exp(m_parts[i] - M) * l_parts[i];
        wsum += w;
        for (int d = 0; d < D; ++d) out[d] += w * o_parts[(int64_t)i * D + d];
    }
    for (int d = 0; d < D; ++d) out[d] /= wsum;
    if (lse) *lse = M + log(wsum);
    return 0;
}

/* Logical gather of one sequence: rows [L][Hkv][D] of K and of V, copied bit
 * for bit from the pools through the block table. */
int oracle_gather_kv(const oracle_shape_t *s, const uint16_t *k_pool, const uint16_t *v_pool,
                     const int32_t *block_table, const int32_t *seq_lens, int b, uint16_t *k_out,
                     uint16_t *v_out)
{
    const int D = s->head_dim, H = s->num_kv_heads;
    for (int t = 0; t < seq_lens[b]; ++t)
        for (int g = 0; g < H; ++g) {
            int64_t ko = row_offset(s, block_table, b, t, g, s->k_stride_page, s->k_stride_token,
                                    s->k_stride_head);
            int64_t vo = row_offset(s, block_table, b, t, g, s->v_stride_page, s->v_stride_token,
                                    s->v_stride_head);
            memcpy(k_out + ((int64_t)t * H + g) * D, k_pool + ko, sizeof(uint16_t) * (size_t)D);
            memcpy(v_out + ((int64_t)t * H + g) * D, v_pool + vo, sizeof(uint16_t) * (size_t)D);
        }
    return 0;
}

/* Own-layer KV write (Invariant 1; Algorithm 1 step 2, first sentence): every
 * valid row - RUN or Project-Only alike - stores the K and V rows its layer
 * projected for the current token at logical position seq_len - 1 of its
 * sequence, i.e. page block_table[b][(L-1) / P], slot (L-1) % P, before
 * attention runs.  new_k / new_v are [B][Hkv][D] bf16 bit patterns; rows with
 * seq_len 0 write nothing.  Pools are modified in place; nothing else moves. */
int oracle_append_kv(const oracle_shape_t *s, const uint16_t *new_k, const uint16_t *new_v,
                     const int32_t *block_table, const int32_t *seq_lens, uint16_t *k_pool,
                     uint16_t *v_pool)
{
    const int D = s->head_dim, H = s->num_kv_heads;
    for (int b = 0; b < s->batch; ++b) {
        if (seq_lens[b] <= 0) continue;
        const int t = seq_lens[b] - 1;
        for (int g = 0; g < H; ++g) {
            int64_t ko = row_offset(s, block_table, b, t, g, s->k_stride_page, s->k_stride_token,
                                    s->k_stride_head);
            int64_t vo = row_offset(s, block_table, b, t, g, s->v_stride_page, s->v_stride_token,
                                    s->v_stride_head);
            memcpy(k_pool + ko, new_k + ((int64_t)b * H + g) * D, sizeof(uint16_t) * (size_t)D);
            memcpy(v_pool + vo, new_v + ((int64_t)b * H + g) * D, sizeof(uint16_t) * (size_t)D);
        }
    }
    return 0;
}
