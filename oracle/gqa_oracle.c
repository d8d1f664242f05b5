/*
 * gqa_oracle.c -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, host-only evaluation of grouped-query attention for one decode step over a paged
 * key-value cache, written out from its definition.  It exists only so that tests and the benchmark's
 * CPU-baseline leg have something independent to compare the CUDA path against; it shares no code,
 * header, table or helper with the CUDA sources.
 *
 * What it follows (paper, Sec. 4.6 "Kernel Analysis: GQA Paged Decode", and the kernel's row of Table 2):
 * every batch item contributes ONE new query token; the kernel attends over the keys and values already
 * stored in the paged cache; several query heads share one key-value head.  The paper gives no formula:
 * it is standard scaled-dot-product attention,
 *     s_t = sm_scale * sum_d q[b,h,d] * k[t,g,d]           for the L_b cached tokens t of batch item b,
 *     p_t = exp(s_t - max_t s_t) / sum_t exp(s_t - max_t s_t),
 *     o[b,h,d] = sum_t p_t * v[t,g,d],                     g = h / (Hq / Hkv) the head's key-value head,
 *     lse[b,h] = max_t s_t + log(sum_t exp(s_t - max_t s_t))   (natural logarithm),
 * with the cache addressed through pages: token t of item b lives in page kv_indices[kv_indptr[b] + t / P]
 * at slot t % P; L_b = (pages of b - 1) * P + kv_last_page_len[b], and 0 for an item without pages.
 * Cache layout: [num_pages, P, Hkv, D], bf16.  An item with no cached token has o = 0 and lse = -inf.
 *
 * Arithmetic type: every floating-point operation is done in REAL (float or double, set by the build);
 * bf16 inputs are widened exactly.  No blocking, no online rescaling, no reordering: the sums run over t
 * (and d) in index order.  OpenMP only distributes independent (item, head) pairs over threads.
 *
 * Pins (tests/test_oracle_gqa.py): hand-derived closed forms (one token; equal scores give the mean of
 * the values; two tokens with a known score gap), torch's scaled_dot_product_attention on the gathered
 * dense keys and values, invariance under a permutation of the physical pages, invariance of o under a
 * shift of all scores, the query-group structure (heads of one group with equal queries agree), and a
 * NumPy float64 evaluation written with matrix products.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#ifndef REAL
#define REAL double
#endif

#define ORACLE_OK 0
#define ORACLE_ERR_ARG (-1)
#define ORACLE_ERR_NOMEM (-3)

static inline REAL real_exp(REAL v) { return sizeof(REAL) == sizeof(float) ? (REAL)expf((float)v) : (REAL)exp((double)v); }
static inline REAL real_log(REAL v) { return sizeof(REAL) == sizeof(float) ? (REAL)logf((float)v) : (REAL)log((double)v); }

/* bfloat16 is the upper half of an IEEE binary32: widening is exact. */
static inline REAL bf16_to_real(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (REAL)f;
}

int gqa_oracle_real_bytes(void) { return (int)sizeof(REAL); }

int gqa_oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Number of cached tokens of batch item b (Sec. 4.6: "the keys and values already stored in the paged KV cache"). */
static long long kv_length(const int32_t *indptr, const int32_t *last_page_len, int b, int page_size) {
    const long long pages = (long long)indptr[b + 1] - indptr[b];
    if (pages <= 0) return 0;
    return (pages - 1) * page_size + last_page_len[b];
}

/*
 * q [B,Hq,D] bf16 bits; k_cache, v_cache [num_pages,P,Hkv,D] bf16 bits; kv_indptr [B+1]; kv_indices [kv_indptr[B]];
 * kv_last_page_len [B]; out [B,Hq,D] REAL; lse [B,Hq] REAL or NULL.
 */
int gqa_oracle_paged_decode(const uint16_t *q, const uint16_t *k_cache, const uint16_t *v_cache, const int32_t *kv_indptr,
                            const int32_t *kv_indices, const int32_t *kv_last_page_len, int B, int Hq, int Hkv, int D,
                            int page_size, int num_pages, double sm_scale, REAL *out, REAL *lse) {
    if (B < 0 || Hq < 1 || Hkv < 1 || D < 1 || page_size < 1 || num_pages < 0 || Hq % Hkv != 0) return ORACLE_ERR_ARG;
    const int group = Hq / Hkv;
    for (int b = 0; b < B; ++b) {
        const long long L = kv_length(kv_indptr, kv_last_page_len, b, page_size);
        if (L < 0 || kv_last_page_len[b] < 0 || kv_last_page_len[b] > page_size) return ORACLE_ERR_ARG;
        for (int i = kv_indptr[b]; i < kv_indptr[b + 1]; ++i)
            if (kv_indices[i] < 0 || kv_indices[i] >= num_pages) return ORACLE_ERR_ARG;
    }
    int failed = 0;
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        for (int h = 0; h < Hq; ++h) {
            const long long L = kv_length(kv_indptr, kv_last_page_len, b, page_size);
            const int g = h / group;
            REAL *o = out + ((size_t)b * Hq + h) * D;
            for (int d = 0; d < D; ++d) o[d] = (REAL)0;
            if (L == 0) {
                if (lse) lse[(size_t)b * Hq + h] = (REAL)-INFINITY;
                continue;
            }
            REAL *s = (REAL *)malloc((size_t)L * sizeof(REAL));
            if (!s) {
                failed = 1;
                continue;
            }
            const uint16_t *qv = q + ((size_t)b * Hq + h) * D;
            /* scores, in token order */
            for (long long t = 0; t < L; ++t) {
                const size_t page = (size_t)kv_indices[kv_indptr[b] + t / page_size];
                const uint16_t *kv = k_cache + ((page * page_size + (size_t)(t % page_size)) * Hkv + g) * D;
                REAL dot = (REAL)0;
                for (int d = 0; d < D; ++d) dot += bf16_to_real(qv[d]) * bf16_to_real(kv[d]);
                s[t] = (REAL)sm_scale * dot;
            }
            /* softmax over the tokens */
            REAL m = s[0];
            for (long long t = 1; t < L; ++t)
                if (s[t] > m) m = s[t];
            REAL sum = (REAL)0;
            for (long long t = 0; t < L; ++t) {
                s[t] = real_exp(s[t] - m);
                sum += s[t];
            }
            /* weighted sum of the values, in token order */
            for (long long t = 0; t < L; ++t) {
                const size_t page = (size_t)kv_indices[kv_indptr[b] + t / page_size];
                const uint16_t *vv = v_cache + ((page * page_size + (size_t)(t % page_size)) * Hkv + g) * D;
                const REAL p = s[t] / sum;
                for (int d = 0; d < D; ++d) o[d] += p * bf16_to_real(vv[d]);
            }
            if (lse) lse[(size_t)b * Hq + h] = m + real_log(sum);
            free(s);
        }
    }
    return failed ? ORACLE_ERR_NOMEM : ORACLE_OK;
}
