/*
 * polyserve_sched.h -- host-side consumers of the profiled latency table.
 *
 * The scheduler of the paper keeps, per serving instance, a profiled map from
 * (token batch size, KV-cache size) to iteration time (section 4.5) and asks
 * it two kinds of question:
 *   - may this decode request join that instance without pushing an iteration
 *     past the TPOT?  (section 4.5, "Profile-Based Batch Formation")
 *   - how should a prompt be cut into prefill chunks, and can the chunk size
 *     chosen now be kept until the prompt is done?  (section 4.7, "dynamic
 *     chunking" and "continuous chunked prefill prediction")
 * These entry points answer them from a table built out of the rows that
 * ps_profile_grid emits.  The table follows the paper's model of an iteration
 * (section 3.4): a term that depends on the token batch size, decode attention
 * as a function of the KV-cache size, and prefill attention as a function of
 * the prefill work; section 4.5 drops the third term for prompts below 10 K
 * tokens, here it is kept as an optional coefficient because the profiled
 * step is attention alone, where a large chunk is not negligible.
 *
 * All of this is plain host code: no device is touched, no stream is taken,
 * and the calls may come from any thread (a table is immutable once built).  They live in the same shared library as the
 * attention entry points and report errors the same way (ps_status,
 * ps_last_error).
 *
 * Notation.  A running decode request r holds kv_len[r] >= 1 tokens in the
 * cache, the token it is generating in the coming iteration included, and
 * still has remaining[r] >= 1 tokens to generate, that one included (for a
 * request whose length is unknown the caller passes the average decode length,
 * as section 4.5 does).  Iterations are numbered t = 0, 1, ... from the coming
 * one.  Request r takes part in iterations 0 .. remaining[r] - 1 and holds
 * kv_len[r] + t tokens in iteration t.
 */
#ifndef POLYSERVE_SCHED_H_
#define POLYSERVE_SCHED_H_

#include "polyserve_attn.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ps_table ps_table; /* (token batch, KV tokens, prefill work) -> microseconds */

/* Prefill-attention work of one chunk of c tokens on `prior` earlier tokens, in
 * the unit of ps_grid_row.prefill_flops: 4 d Hq (c prior + c (c + 1) / 2). */
#define PS_PREFILL_FLOPS(head_dim, n_q_heads, c, prior) \
    (4.0 * (double)(head_dim) * (double)(n_q_heads) * ((double)(c) * (double)(prior) + 0.5 * (double)(c) * ((double)(c) + 1.0)))

/* ------------------------------------------------------------------------ */
/* Latency table (section 4.5).                                               */
/* ------------------------------------------------------------------------ */

/*
 * Build a table from n_rows sweep rows (host array, e.g. the output of
 * ps_profile_grid).  Rows with the same token_batch form one line of the
 * table: the ordinary least-squares fit
 *     latency_us = intercept + slope_kv * kv_tokens + slope_pf * prefill_flops
 * over the line's rows (section 3.4: decode attention time is a function of
 * the total number of KV tokens, prefill attention of the prefill work; the
 * intercept carries whatever depends on the batch size alone).  With
 * centred sums Sxx, Spp, Sxp of the two regressors: if Spp = 0 (no chunk, or
 * the same work in every row) the line is fitted on kv_tokens alone with
 * slope_pf = 0; if Sxx = 0 on prefill_flops alone; if both vanish the line is
 * the mean latency; if the two are collinear (Sxx Spp - Sxp^2 <= 1e-9 Sxx
 * Spp) on kv_tokens alone.  Lines are kept sorted by token_batch.
 * Errors: PS_ERR_INVALID (null pointers, n_rows < 1, a row with
 * token_batch < 1, kv_tokens < 0 or a latency that is not finite),
 * PS_ERR_OOM.
 */
ps_status ps_table_build(const ps_grid_row *rows, int64_t n_rows, ps_table **out);

/*
 * The same sweep fitted in the overlap form.  This library runs the decode
 * rows and the prefill chunk of a mixed batch side by side on disjoint SMs, so
 * a mixed batch takes about as long as the slower of its two parts, not their
 * sum (section 3.4 adds the terms for engines that run them one after the
 * other).  A line of an overlap table predicts
 *     latency_us = base + max(decode_intercept + slope_kv * kv_tokens,
 *                             prefill_intercept + slope_pf * prefill_flops),
 * with the prefill term left out when prefill_flops = 0 and the decode term
 * when kv_tokens = 0; base is 0 after this call and takes what
 * ps_table_add_batch_term adds.  The four parameters are fitted once over all
 * rows (every line of the table, one per distinct token_batch, carries the
 * same four) by alternating least squares:
 *   1. the sum form a + s kv + q pf over all rows (rules of ps_table_build)
 *      gives the start: decode_intercept = prefill_intercept = a, s, q (a
 *      negative slope is taken as 0);
 *   2. a row belongs to the decode side if its prefill_flops = 0, to the
 *      prefill side if its kv_tokens = 0, else to the side whose term (at the
 *      start: s kv against q pf; later the whole term with its intercept) is
 *      the larger, ties to the decode side;
 *   3. decode side first, then prefill side: least-squares line of latency
 *      over that side's own regressor on that side's rows; a side with fewer
 *      than two rows, or whose regressor does not vary, keeps its parameters;
 *   4. rows are assigned again (step 2); repeat 3-4 until no row moves, at
 *      most 64 times.
 * ps_table_get_lines returns base and the two slopes of such a table,
 * ps_table_get_overlap whether a table is in this form and the two intercepts
 * (outputs may be NULL; capacity in lines; for a sum-form table only
 * *is_overlap_out = 0 is written).  ps_table_scale multiplies all five
 * coefficients; prediction, admission and chunk prediction use whichever form
 * the table has.  Errors as for ps_table_build.
 */
ps_status ps_table_build_overlap(const ps_grid_row *rows, int64_t n_rows, ps_table **out);
ps_status ps_table_get_overlap(const ps_table *table, int32_t *is_overlap_out, double *decode_intercept_us_out,
                               double *prefill_intercept_us_out, int32_t capacity);

/*
 * Build a table from explicit lines: line i predicts intercept_us[i] +
 * slope_us_per_token[i] * kv_tokens + slope_us_per_flop[i] * prefill_flops at
 * batch size token_batch[i] (slope_us_per_flop == NULL: all zero).  The lines
 * may come in any order; two lines with the same token_batch are an error.
 */
ps_status ps_table_from_lines(const int32_t *token_batch, const double *intercept_us,
                              const double *slope_us_per_token, const double *slope_us_per_flop, int32_t n_lines,
                              ps_table **out);

ps_status ps_table_free(ps_table *table);

/*
 * Add a term that depends on the token batch size alone to every line of the
 * table -- the GEMM(B) of the paper's iteration model (section 3.4: T_iter =
 * GEMM(B) + decode attention + prefill attention), measured by the caller for
 * its model's linear layers.  The term is given at n >= 1 sample batch sizes
 * (any order, distinct) and interpolated linearly between them; outside the
 * samples the nearest one is used.  ps_table_scale multiplies every
 * coefficient by factor > 0 (n identical layers: n times one layer).  Both
 * change the table in place: call them before sharing it between threads.
 * Errors: PS_ERR_INVALID (null pointers, n < 1, a batch size < 1 or repeated,
 * a value that is not finite, factor <= 0).
 */
ps_status ps_table_add_batch_term(ps_table *table, const int32_t *token_batch, const double *term_us, int32_t n);
ps_status ps_table_scale(ps_table *table, double factor);

/* Number of lines; and a copy of them, sorted by token_batch (any output may
 * be NULL; capacity in lines). */
ps_status ps_table_size(const ps_table *table, int32_t *n_lines_out);
ps_status ps_table_get_lines(const ps_table *table, int32_t *token_batch_out, double *intercept_us_out,
                             double *slope_us_per_token_out, double *slope_us_per_flop_out, int32_t capacity);

/*
 * Predicted iteration time in microseconds for a batch of token_batch tokens
 * (decode rows count one token each, a prefill chunk its length) whose rows
 * hold kv_tokens tokens of K/V in total (the chunk's row included) and whose
 * chunks amount to prefill_flops of attention work (PS_PREFILL_FLOPS summed
 * over the chunks; 0 for a decode-only batch).  Between two lines the two
 * lines' values are interpolated linearly in token_batch; below the first
 * line and above the last one the nearest line is used as it is (no
 * extrapolation in the batch size).  Errors: PS_ERR_INVALID (null pointers,
 * token_batch < 1, kv_tokens < 0, prefill_flops < 0 or not finite).
 */
ps_status ps_table_predict(const ps_table *table, int32_t token_batch, int64_t kv_tokens, double prefill_flops,
                           double *latency_us_out);

/* ------------------------------------------------------------------------ */
/* Decode admission (section 4.5).                                            */
/* ------------------------------------------------------------------------ */

/*
 * Simulate the future iterations of a set of decode requests (host arrays of
 * n >= 0 entries) and return the largest total KV-cache size any iteration
 * sees, peak = max over t of the sum, over requests with remaining > t, of
 * kv_len + t, and the first iteration at which it occurs.  n == 0 gives
 * peak 0 at iteration 0.  Errors: PS_ERR_INVALID (kv_len < 1, remaining < 1).
 */
ps_status ps_peak_kv(const int32_t *kv_len, const int32_t *remaining, int32_t n, int64_t *peak_kv_out,
                     int32_t *peak_iter_out);

/*
 * Admission test for one new decode request (new_kv_len tokens cached once
 * its first decode iteration runs, new_remaining tokens to generate) on an
 * instance running n_running requests: the peak KV-cache size of the running
 * set plus the new request is looked up in the table at the current token
 * batch size (n_running + 1 + extra_tokens; extra_tokens >= 0 counts prefill
 * tokens batched alongside, extra_kv_tokens >= 0 the K/V their rows hold and
 * extra_prefill_flops >= 0 their attention work), and the request is admitted
 * when the predicted iteration time is below tpot_us.  Outputs (each may be
 * NULL): *admit_out 1 or 0, the predicted time, and the decode requests' peak
 * KV size (extra_kv_tokens not included).
 */
ps_status ps_admit(const ps_table *table, const int32_t *kv_len, const int32_t *remaining, int32_t n_running,
                   int32_t new_kv_len, int32_t new_remaining, int32_t extra_tokens, int64_t extra_kv_tokens,
                   double extra_prefill_flops, double tpot_us, int32_t *admit_out, double *predicted_us_out,
                   int64_t *peak_kv_out);

/* ------------------------------------------------------------------------ */
/* Prefill chunking (section 4.7).                                            */
/* ------------------------------------------------------------------------ */

/*
 * Chunk lengths for the coming iteration of a prefill instance with a token
 * budget (section 4.7, PD-disaggregation).  remaining[i] >= 1 is the number of
 * prompt tokens request i still has to prefill; requests are served first come
 * first served in array order; `used` tokens of the budget are already taken.
 * With dynamic == 0 (plain chunked prefill) each request gets
 * min(remaining, budget left) until the budget is spent.  With dynamic != 0,
 * a request whose remaining length is below twice the budget is finished at
 * once -- its whole remainder becomes the chunk even where that exceeds the
 * budget left -- and no further request is admitted behind it in this
 * iteration; longer requests get min(remaining, budget left) as before.
 * chunk_out[i] receives request i's chunk (0 = not scheduled now).
 * Errors: PS_ERR_INVALID (budget < 1, used < 0, remaining < 1).
 */
ps_status ps_chunk_next(const int32_t *remaining, int32_t n, int32_t budget, int32_t used, int32_t dynamic,
                        int32_t *chunk_out);

/*
 * The whole chunk sequence of one prompt of prompt_len tokens that is alone
 * in its instance except that first_free <= budget tokens of the first
 * iteration's budget are still free (the rest taken by earlier requests):
 * ps_chunk_next applied iteration after iteration.  chunks_out (capacity
 * entries) receives the lengths, *n_chunks_out their number (also when the
 * capacity is too small, which returns PS_ERR_INVALID after filling what
 * fits).  The paper's example: a 2050-token prompt under a budget of 1024
 * takes 1024 + 1024 + 2 statically, 1 + 1024 + 1024 + 1 when the first
 * iteration has one token left, and 1024 + 1026 dynamically.
 */
ps_status ps_chunk_schedule(int32_t prompt_len, int32_t budget, int32_t first_free, int32_t dynamic,
                            int32_t *chunks_out, int32_t capacity, int32_t *n_chunks_out);

/*
 * Continuous chunked-prefill prediction for co-located serving (section 4.7):
 * a prompt of prompt_len tokens is to be prefilled in chunks beside the
 * n_running decode requests of an instance without any iteration exceeding
 * tpot_us.  The chunk size predicted at scheduling time is the largest c in
 * [1, min(prompt_len, max_chunk)] for which the table predicts at most tpot_us
 * for iteration 0 (token batch = decode requests alive + c, KV tokens = their
 * KV + c, prefill work = flops_per_pair c (c + 1) / 2 with flops_per_pair =
 * 4 head_dim n_q_heads); 0 if there is none.  The prefill
 * then takes ceil(prompt_len / c) iterations; in iteration k the decode
 * requests still alive have grown by k tokens each, the prompt's row holds
 * min((k + 1) c, prompt_len) tokens and its chunk of c_k tokens works on k c
 * prior tokens.
 * *maintained_out is 1 when every one of those iterations is still predicted
 * at or below tpot_us with that same chunk size (the paper admits the request
 * only then), *completion_us_out the sum of the predicted iteration times (the
 * completion-time estimate to compare with the TTFT), *n_iters_out the number
 * of iterations.  With *chunk_out == 0 the other outputs are 0.
 * Errors: PS_ERR_INVALID (prompt_len < 1, max_chunk < 1, flops_per_pair < 0,
 * bad request arrays).
 */
ps_status ps_chunk_predict(const ps_table *table, const int32_t *kv_len, const int32_t *remaining, int32_t n_running,
                           int32_t prompt_len, int32_t max_chunk, double flops_per_pair, double tpot_us,
                           int32_t *chunk_out, int32_t *n_iters_out, double *completion_us_out,
                           int32_t *maintained_out);

#ifdef __cplusplus
}
#endif
#endif /* POLYSERVE_SCHED_H_ */
