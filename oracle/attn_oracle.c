/*
 * CPU oracle for mixed-batch paged-KV attention.  TEST INFRASTRUCTURE ONLY:
 * the library's product path never links, imports or calls this file.
 *
 * What it computes is the plain definition (paper section 2.1, "LLM Inference
 * Workflow"): self-attention Softmax(Q K^T / sqrt(d)) V using the K and V of
 * all previous tokens.  For request r, new token i in [0, q_len[r]), q head h,
 * with kv head g = h / (Hq / Hkv) and L = prior[r] + i + 1 visible keys:
 *
 *     s_j  = (sum_t Q[r,i,h,t] * K[r,j,g,t]) / sqrt(d)        j = 0 .. L-1
 *     out  = sum_j softmax_j(s) * V[r,j,g,:]
 *     lse  = log sum_j exp(s_j)
 *
 * A decode row is q_len = 1; a prefill chunk (section 2.4, chunked prefill;
 * section 4.7, dynamic chunking) is q_len > 1 whose rows see the prior context
 * plus the chunk's own earlier tokens and themselves.
 *
 * Readings where the paper is silent: a token attends itself (inclusive causal
 * mask); consecutive q heads share a kv head; all arithmetic is fp64 on the
 * bf16 inputs widened exactly; softmax is evaluated by max subtraction.
 *
 * K and V are read from the oracle's own paged layout, which differs from the
 * GPU library's on purpose:
 *     k_pool, v_pool : uint16 [num_pages][page_size][Hkv][d]   (bf16 bits)
 * token j of request r lives in page block_table[r*max_pages + j/page_size],
 * slot j % page_size.
 *
 * No blocking, fusion or reordering: one pass for scores, one for the max,
 * one for the weights, one for the weighted sum.  OpenMP over (row, head).
 *
 * Pins (tests/test_oracle_pins.py): brute force with an explicit mask matrix
 * in extended precision, constant V, single key, one-hot key, zero Q (prefix
 * mean), chunk split == unchunked, decode row == last prefill row, key
 * permutation invariance, GQA mapping, torch CPU fp64 causal SDPA, page
 * permutation with NaN-poisoned spare pages, split + log-sum-exp merge; the FP8
 * variant equals the bf16 one on data that E4M3 holds exactly.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static inline double bf16_to_f64(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Attention for a list of output rows.  Row k is (request row_req[k], new
 * token row_tok[k]); q is the packed [T, Hq, d] bf16 tensor of the whole batch
 * (requests in order, tokens in order).  out: [n_rows, Hq, d], lse: [n_rows, Hq].
 * Returns 0, or a negative code for bad arguments / out-of-range page ids.
 */
int oracle_attn_rows(const uint16_t *q, const uint16_t *k_pool, const uint16_t *v_pool,
                     int64_t num_pages, const int32_t *block_table, int32_t max_pages,
                     const int32_t *prior, const int32_t *q_len, int32_t n,
                     int32_t Hq, int32_t Hkv, int32_t d, int32_t page_size,
                     const int32_t *row_req, const int32_t *row_tok, int64_t n_rows,
                     double *out, double *lse) {
    if (Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || d <= 0 || page_size <= 0) return -1;
    const int G = Hq / Hkv;
    int64_t *q_start = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n + 1));
    if (!q_start) return -2;
    q_start[0] = 0;
    for (int r = 0; r < n; ++r) {
        if (q_len[r] < 1 || prior[r] < 0) { free(q_start); return -3; }
        if ((int64_t)prior[r] + q_len[r] > (int64_t)max_pages * page_size) { free(q_start); return -4; }
        q_start[r + 1] = q_start[r] + q_len[r];
    }
    for (int64_t k = 0; k < n_rows; ++k) {
        int r = row_req[k];
        if (r < 0 || r >= n || row_tok[k] < 0 || row_tok[k] >= q_len[r]) { free(q_start); return -5; }
    }
    int bad = 0;
    const double scale = 1.0 / sqrt((double)d);
    const int64_t n_work = n_rows * Hq;
#pragma omp parallel
    {
        double *s = NULL;
        int64_t cap = 0;
#pragma omp for schedule(dynamic, 1)
        for (int64_t w = 0; w < n_work; ++w) {
            const int64_t k = w / Hq;
            const int h = (int)(w % Hq);
            const int g = h / G;
            const int r = row_req[k];
            const int i = row_tok[k];
            const int64_t L = (int64_t)prior[r] + i + 1;
            if (L > cap) {
                free(s);
                s = (double *)malloc(sizeof(double) * (size_t)L);
                cap = L;
            }
            const uint16_t *qv = q + ((q_start[r] + i) * Hq + h) * (int64_t)d;
            const int32_t *bt = block_table + (int64_t)r * max_pages;
            /* scores */
            for (int64_t j = 0; j < L; ++j) {
                const int64_t page = bt[j / page_size];
                if (page < 0 || page >= num_pages) {
#pragma omp atomic write
                    bad = 1;
                    s[j] = 0.0;
                    continue;
                }
                const uint16_t *kv = k_pool + ((page * page_size + j % page_size) * Hkv + g) * (int64_t)d;
                double acc = 0.0;
                for (int t = 0; t < d; ++t) acc += bf16_to_f64(qv[t]) * bf16_to_f64(kv[t]);
                s[j] = acc * scale;
            }
            /* softmax by max subtraction */
            double m = s[0];
            for (int64_t j = 1; j < L; ++j) if (s[j] > m) m = s[j];
            double denom = 0.0;
            for (int64_t j = 0; j < L; ++j) { s[j] = exp(s[j] - m); denom += s[j]; }
            /* weighted sum of V */
            double *o = out + (k * Hq + h) * (int64_t)d;
            for (int t = 0; t < d; ++t) o[t] = 0.0;
            for (int64_t j = 0; j < L; ++j) {
                const int64_t page = bt[j / page_size];
                if (page < 0 || page >= num_pages) continue;
                const uint16_t *vv = v_pool + ((page * page_size + j % page_size) * Hkv + g) * (int64_t)d;
                const double p = s[j] / denom;
                for (int t = 0; t < d; ++t) o[t] += p * bf16_to_f64(vv[t]);
            }
            lse[k * Hq + h] = m + log(denom);
        }
        free(s);
    }
    free(q_start);
    return bad ? -6 : 0;
}

/*
 * The same attention over an FP8 (E4M3) KV cache: k_codes / v_codes hold one code per element,
 * uint8 [num_pages][page_size][Hkv][d]; k_scale / v_scale one fp32 scale per (token, kv head),
 * float [num_pages][page_size][Hkv]; an element's value is e4m3[code] * scale, evaluated in fp64
 * (exact).  e4m3 is the 256-entry table of code values (built by the caller from the format's
 * definition: bias 7, 3 mantissa bits, subnormals m * 2^-9).  Q stays bf16.  The quantisation
 * format is this repository's reading (the paper states no precision); the arithmetic below is
 * the plain definition again.
 */
int oracle_attn_rows_fp8(const uint16_t *q, const uint8_t *k_codes, const uint8_t *v_codes,
                         const float *k_scale, const float *v_scale, const double *e4m3,
                         int64_t num_pages, const int32_t *block_table, int32_t max_pages,
                         const int32_t *prior, const int32_t *q_len, int32_t n,
                         int32_t Hq, int32_t Hkv, int32_t d, int32_t page_size,
                         const int32_t *row_req, const int32_t *row_tok, int64_t n_rows,
                         double *out, double *lse) {
    if (Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || d <= 0 || page_size <= 0) return -1;
    const int G = Hq / Hkv;
    int64_t *q_start = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n + 1));
    if (!q_start) return -2;
    q_start[0] = 0;
    for (int r = 0; r < n; ++r) {
        if (q_len[r] < 1 || prior[r] < 0) { free(q_start); return -3; }
        if ((int64_t)prior[r] + q_len[r] > (int64_t)max_pages * page_size) { free(q_start); return -4; }
        q_start[r + 1] = q_start[r] + q_len[r];
    }
    for (int64_t k = 0; k < n_rows; ++k) {
        int r = row_req[k];
        if (r < 0 || r >= n || row_tok[k] < 0 || row_tok[k] >= q_len[r]) { free(q_start); return -5; }
    }
    int bad = 0;
    const double scale = 1.0 / sqrt((double)d);
    const int64_t n_work = n_rows * Hq;
#pragma omp parallel
    {
        double *s = NULL;
        int64_t cap = 0;
#pragma omp for schedule(dynamic, 1)
        for (int64_t w = 0; w < n_work; ++w) {
            const int64_t k = w / Hq;
            const int h = (int)(w % Hq);
            const int g = h / G;
            const int r = row_req[k];
            const int i = row_tok[k];
            const int64_t L = (int64_t)prior[r] + i + 1;
            if (L > cap) {
                free(s);
                s = (double *)malloc(sizeof(double) * (size_t)L);
                cap = L;
            }
            const uint16_t *qv = q + ((q_start[r] + i) * Hq + h) * (int64_t)d;
            const int32_t *bt = block_table + (int64_t)r * max_pages;
            /* scores */
            for (int64_t j = 0; j < L; ++j) {
                const int64_t page = bt[j / page_size];
                if (page < 0 || page >= num_pages) {
#pragma omp atomic write
                    bad = 1;
                    s[j] = 0.0;
                    continue;
                }
                const int64_t slot = (page * page_size + j % page_size) * Hkv + g;
                const uint8_t *kc = k_codes + slot * (int64_t)d;
                const double ks = (double)k_scale[slot];
                double acc = 0.0;
                for (int t = 0; t < d; ++t) acc += bf16_to_f64(qv[t]) * (e4m3[kc[t]] * ks);
                s[j] = acc * scale;
            }
            /* softmax by max subtraction */
            double m = s[0];
            for (int64_t j = 1; j < L; ++j) if (s[j] > m) m = s[j];
            double denom = 0.0;
            for (int64_t j = 0; j < L; ++j) { s[j] = exp(s[j] - m); denom += s[j]; }
            /* weighted sum of V */
            double *o = out + (k * Hq + h) * (int64_t)d;
            for (int t = 0; t < d; ++t) o[t] = 0.0;
            for (int64_t j = 0; j < L; ++j) {
                const int64_t page = bt[j / page_size];
                if (page < 0 || page >= num_pages) continue;
                const int64_t slot = (page * page_size + j % page_size) * Hkv + g;
                const uint8_t *vc = v_codes + slot * (int64_t)d;
                const double vs = (double)v_scale[slot];
                const double p = s[j] / denom;
                for (int t = 0; t < d; ++t) o[t] += p * (e4m3[vc[t]] * vs);
            }
            lse[k * Hq + h] = m + log(denom);
        }
        free(s);
    }
    free(q_start);
    return bad ? -6 : 0;
}

/* Every row of every request, in packed order: out [T, Hq, d], lse [T, Hq]. */
int oracle_attn_paged(const uint16_t *q, const uint16_t *k_pool, const uint16_t *v_pool,
                      int64_t num_pages, const int32_t *block_table, int32_t max_pages,
                      const int32_t *prior, const int32_t *q_len, int32_t n,
                      int32_t Hq, int32_t Hkv, int32_t d, int32_t page_size,
                      double *out, double *lse) {
    int64_t T = 0;
    for (int r = 0; r < n; ++r) {
        if (q_len[r] < 1) return -3;
        T += q_len[r];
    }
    int32_t *rr = (int32_t *)malloc(sizeof(int32_t) * (size_t)(T > 0 ? T : 1));
    int32_t *rt = (int32_t *)malloc(sizeof(int32_t) * (size_t)(T > 0 ? T : 1));
    if (!rr || !rt) { free(rr); free(rt); return -2; }
    int64_t k = 0;
    for (int r = 0; r < n; ++r)
        for (int i = 0; i < q_len[r]; ++i) { rr[k] = r; rt[k] = i; ++k; }
    int rc = oracle_attn_rows(q, k_pool, v_pool, num_pages, block_table, max_pages, prior, q_len, n,
                              Hq, Hkv, d, page_size, rr, rt, T, out, lse);
    free(rr);
    free(rt);
    return rc;
}

/*
 * Gather logical tokens [0, len) of one sequence from the oracle's paged pool
 * into contiguous [len, Hkv, d] (bit copy).
 */
int oracle_kv_gather(const uint16_t *pool, int64_t num_pages, const int32_t *block_table_row,
                     int32_t len, int32_t Hkv, int32_t d, int32_t page_size, uint16_t *dst) {
    const int64_t row = (int64_t)Hkv * d;
    for (int32_t j = 0; j < len; ++j) {
        const int64_t page = block_table_row[j / page_size];
        if (page < 0 || page >= num_pages) return -6;
        memcpy(dst + j * row, pool + (page * page_size + j % page_size) * row, sizeof(uint16_t) * (size_t)row);
    }
    return 0;
}

/*
 * Combine attention results computed over disjoint key subsets of the same
 * query.  Partial s has normalised output o_s[d] and log-sum-exp lse_s.  With
 * M = max_s lse_s:
 *     out = sum_s exp(lse_s - M) o_s / sum_s exp(lse_s - M)
 *     lse = M + log sum_s exp(lse_s - M)
 * This is the identity softmax-over-a-union = convex mix of the softmaxes over
 * the parts, weighted by the parts' exponential mass.  o: [n_seg, d].
 */
int oracle_lse_merge(const double *o, const double *lse_in, int32_t n_seg, int32_t d,
                     double *out, double *lse_out) {
    if (n_seg < 1) return -1;
    double M = lse_in[0];
    for (int s = 1; s < n_seg; ++s) if (lse_in[s] > M) M = lse_in[s];
    double denom = 0.0;
    for (int s = 0; s < n_seg; ++s) denom += exp(lse_in[s] - M);
    for (int t = 0; t < d; ++t) out[t] = 0.0;
    for (int s = 0; s < n_seg; ++s) {
        const double w = exp(lse_in[s] - M) / denom;
        for (int t = 0; t < d; ++t) out[t] += w * o[(int64_t)s * d + t];
    }
    *lse_out = M + log(denom);
    return 0;
}
