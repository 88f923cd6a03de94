/*
 * CPU oracle for cache-aware causal prefill attention (TEST INFRASTRUCTURE ONLY).
 *
 * Plain, slow, fp64.  Used by the tests, by the smoke check and by the benchmark's
 * CPU-baseline leg; never by the product path, and it shares no code with the CUDA
 * library.  One function: causal softmax attention of selected (query row, head)
 * pairs over keys fetched through a page table, written as the definition reads.
 *
 * Definition followed (paper Section 2.1, the causal self-attention formula, and
 * Section 2.2, prefix caching): with P cached tokens and R new tokens, new token r
 * sits at absolute position i = P + r and attends to keys j = 0..i (mask M_ij = 0
 * for j <= i, -inf otherwise, diagonal included).  For query head h with KV head
 * g = h / (Hq / Hkv):
 *
 *     S_j  = scale * sum_d q[r,h,d] * k[j,g,d]
 *     m    = max_j S_j
 *     l    = sum_j exp(S_j - m)
 *     O    = (sum_j exp(S_j - m) * v[j,g,:]) / l
 *     LSE  = m + ln l            (natural log of the scaled scores)
 *
 * A key subset can be given as a list of half-open absolute ranges; keys outside
 * the ranges (or above the diagonal) are not attended.  An empty visible set gives
 * O = 0 and LSE = -inf.  Inputs are bf16 bit patterns and are widened exactly.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static inline double bf16_to_f64(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* Element offset of logical token t, KV head g, in a paged cache. */
static inline int64_t paged_offset(const int32_t *page_table, int64_t t, int32_t page_size,
                                   int64_t stride_page, int64_t stride_tok, int64_t stride_head, int32_t g)
{
    return (int64_t)page_table[t / page_size] * stride_page + (t % page_size) * stride_tok + (int64_t)g * stride_head;
}

/* 1 if absolute key position j belongs to the attended subset (all keys when no ranges are given). */
static inline int key_attended(int64_t j, const int64_t *key_ranges, int32_t n_ranges)
{
    if (n_ranges == 0 || key_ranges == NULL) return 1;
    for (int32_t t = 0; t < n_ranges; ++t)
        if (j >= key_ranges[2 * t] && j < key_ranges[2 * t + 1]) return 1;
    return 0;
}

/*
 * q            [R, Hq, D] bf16 bits, new tokens in original order
 * k, v         paged caches, bf16 bits, addressed with the three strides (elements; dim stride 1)
 * page_table   logical page -> physical page of this request, ceil((P+R)/page_size) entries
 * rows, heads  n (query row, head) pairs to evaluate
 * key_ranges   n_ranges half-open [begin,end) absolute key ranges; NULL/0 means all keys
 * out          [n, D] fp64,  lse [n] fp64
 * Returns 0, or -1 on a bad argument.
 */
int oracle_attn_pairs(const uint16_t *q, int64_t R, int32_t Hq, int32_t Hkv, int32_t D,
                      const uint16_t *k, const uint16_t *v, int32_t page_size,
                      int64_t stride_page, int64_t stride_tok, int64_t stride_head,
                      const int32_t *page_table, int64_t P, double scale,
                      const int64_t *rows, const int32_t *heads, int64_t n,
                      const int64_t *key_ranges, int32_t n_ranges,
                      double *out, double *lse, int32_t n_threads)
{
    if (Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || D <= 0 || page_size <= 0 || R < 0 || P < 0) return -1;
    const int32_t G = Hq / Hkv;
    int bad = 0;
    if (n_threads <= 0) n_threads = 1;

#pragma omp parallel num_threads(n_threads)
    {
        double *S = (double *)malloc(sizeof(double) * (size_t)(P + R + 1));
        double *qd = (double *)malloc(sizeof(double) * (size_t)D);
        double *acc = (double *)malloc(sizeof(double) * (size_t)D);
#pragma omp for schedule(dynamic, 1)
        for (int64_t idx = 0; idx < n; ++idx) {
            const int64_t r = rows[idx];
            const int32_t h = heads[idx];
            if (r < 0 || r >= R || h < 0 || h >= Hq) {
#pragma omp atomic write
                bad = 1;
                continue;
            }
            const int32_t g = h / G;
            const int64_t i = P + r;                    /* absolute position: sees keys 0..i */
            for (int32_t d = 0; d < D; ++d) qd[d] = bf16_to_f64(q[(r * Hq + h) * (int64_t)D + d]);

            /* pass 1: scaled scores of the attended keys and their maximum */
            double m = -INFINITY;
            for (int64_t j = 0; j <= i; ++j) {
                if (!key_attended(j, key_ranges, n_ranges)) continue;
                const uint16_t *kr = k + paged_offset(page_table, j, page_size, stride_page, stride_tok, stride_head, g);
                double s = 0.0;
                for (int32_t d = 0; d < D; ++d) s += qd[d] * bf16_to_f64(kr[d]);
                s *= scale;
                S[j] = s;
                if (s > m) m = s;
            }
            for (int32_t d = 0; d < D; ++d) acc[d] = 0.0;
            double l = 0.0;
            if (m > -INFINITY) {                        /* pass 2: softmax weights and weighted values */
                for (int64_t j = 0; j <= i; ++j) {
                    if (!key_attended(j, key_ranges, n_ranges)) continue;
                    const double p = exp(S[j] - m);
                    l += p;
                    const uint16_t *vr = v + paged_offset(page_table, j, page_size, stride_page, stride_tok, stride_head, g);
                    for (int32_t d = 0; d < D; ++d) acc[d] += p * bf16_to_f64(vr[d]);
                }
            }
            if (l > 0.0) {
                for (int32_t d = 0; d < D; ++d) out[idx * (int64_t)D + d] = acc[d] / l;
                lse[idx] = m + log(l);
            } else {
                for (int32_t d = 0; d < D; ++d) out[idx * (int64_t)D + d] = 0.0;
                lse[idx] = -INFINITY;
            }
        }
        free(S); free(qd); free(acc);
    }
    return bad ? -1 : 0;
}
