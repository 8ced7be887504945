// Host-side consumers of the profiled latency table: the table itself, the
// decode admission test (paper section 4.5) and the prefill chunk sizers
// (section 4.7).  Plain host code; nothing here touches the device.
#include <algorithm>
#include <cmath>
#include <new>
#include <numeric>
#include <vector>

#include "common.cuh"
#include "../../include/polyserve_sched.h"

struct ps_table {
    std::vector<int32_t> batch;   // sorted, distinct
    std::vector<double> intercept;
    std::vector<double> slope;     // microseconds per KV token
    std::vector<double> slope_pf;  // microseconds per flop of prefill attention
    // Overlap form (decode and prefill attention side by side): a line is intercept + max(dec_icpt + slope kv,
    // pf_icpt + slope_pf pf); `intercept` then holds only what depends on the batch size alone.
    bool overlap = false;
    std::vector<double> dec_icpt, pf_icpt;
};

namespace ps {
namespace {

double line_at(const ps_table& t, size_t i, int64_t kv, double pf) {
    if (!t.overlap) return t.intercept[i] + t.slope[i] * (double)kv + t.slope_pf[i] * pf;
    const double dec = t.dec_icpt[i] + t.slope[i] * (double)kv, pre = t.pf_icpt[i] + t.slope_pf[i] * pf;
    // a batch without a chunk runs no prefill kernel, one without KV tokens no decode kernel
    const double attn = pf == 0.0 ? dec : kv == 0 ? pre : std::max(dec, pre);
    return t.intercept[i] + attn;
}

// Least squares of y = a + s x + q p over the rows listed in idx (centred sums; a regressor that does not vary, or
// the second of two collinear ones, is left out).
struct Plane { double a, s, q; };
Plane fit_plane(const ps_grid_row* rows, const int64_t* idx, int64_t n_idx) {
    const double n = (double)n_idx;
    double sum_x = 0.0, sum_p = 0.0, sum_y = 0.0;
    for (int64_t k = 0; k < n_idx; ++k) {
        const ps_grid_row& r = rows[idx[k]];
        sum_x += (double)r.kv_tokens, sum_p += r.prefill_flops, sum_y += (double)r.latency_us;
    }
    const double mx = sum_x / n, mp = sum_p / n, my = sum_y / n;
    double sxx = 0.0, spp = 0.0, sxp = 0.0, sxy = 0.0, spy = 0.0;
    for (int64_t k = 0; k < n_idx; ++k) {
        const ps_grid_row& r = rows[idx[k]];
        const double dx = (double)r.kv_tokens - mx, dp = r.prefill_flops - mp, dy = (double)r.latency_us - my;
        sxx += dx * dx, spp += dp * dp, sxp += dx * dp, sxy += dx * dy, spy += dp * dy;
    }
    const double det = sxx * spp - sxp * sxp;
    Plane f{0.0, 0.0, 0.0};
    if (sxx > 0.0 && spp > 0.0 && det > 1e-9 * sxx * spp) {
        f.s = (sxy * spp - spy * sxp) / det;
        f.q = (spy * sxx - sxy * sxp) / det;
    } else if (sxx > 0.0) {
        f.s = sxy / sxx;
    } else if (spp > 0.0) {
        f.q = spy / spp;
    }
    f.a = my - f.s * mx - f.q * mp;
    return f;
}

ps_status check_rows(const char* who, const ps_grid_row* rows, int64_t n_rows) {
    for (int64_t i = 0; i < n_rows; ++i)
        if (rows[i].token_batch < 1 || rows[i].kv_tokens < 0 || !std::isfinite(rows[i].latency_us) || !std::isfinite(rows[i].prefill_flops) ||
            rows[i].prefill_flops < 0.0)
            return fail(PS_ERR_INVALID, "%s: row %lld has token_batch %d, kv_tokens %lld, latency %g", who, (long long)i,
                        rows[i].token_batch, (long long)rows[i].kv_tokens, (double)rows[i].latency_us);
    return PS_OK;
}

double predict(const ps_table& t, int32_t token_batch, int64_t kv, double pf) {
    const size_t n = t.batch.size();
    if (token_batch <= t.batch.front()) return line_at(t, 0, kv, pf);
    if (token_batch >= t.batch.back()) return line_at(t, n - 1, kv, pf);
    // lines lo, hi with batch[lo] <= token_batch < batch[hi]
    const size_t hi = (size_t)(std::upper_bound(t.batch.begin(), t.batch.end(), token_batch) - t.batch.begin());
    const size_t lo = hi - 1;
    const double w = (double)(token_batch - t.batch[lo]) / (double)(t.batch[hi] - t.batch[lo]);
    const double a = line_at(t, lo, kv, pf), b = line_at(t, hi, kv, pf);
    return a + (b - a) * w;
}

ps_status check_requests(const int32_t* kv_len, const int32_t* remaining, int32_t n) {
    if (n < 0 || (n > 0 && (!kv_len || !remaining))) return fail(PS_ERR_INVALID, "request arrays: n = %d with a null pointer", n);
    for (int32_t i = 0; i < n; ++i)
        if (kv_len[i] < 1 || remaining[i] < 1)
            return fail(PS_ERR_INVALID, "request %d: kv_len = %d, remaining = %d (both must be >= 1)", i, kv_len[i], remaining[i]);
    return PS_OK;
}

// The decode requests of an instance ordered by the iteration at which they leave, with running sums, so
// that the requests alive in iteration t (remaining > t) and their total length are a suffix.
struct Future {
    std::vector<int32_t> rem;      // ascending
    std::vector<int64_t> len_suf;  // len_suf[i] = sum of kv_len over sorted positions >= i (n + 1 entries)
    Future(const int32_t* kv_len, const int32_t* remaining, int32_t n) : rem(n), len_suf(n + 1, 0) {
        std::vector<int32_t> order(n);
        std::iota(order.begin(), order.end(), 0);
        std::sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return remaining[a] < remaining[b]; });
        for (int32_t i = 0; i < n; ++i) rem[i] = remaining[order[i]];
        for (int32_t i = n - 1; i >= 0; --i) len_suf[i] = len_suf[i + 1] + kv_len[order[i]];
    }
    // first sorted position alive in iteration t; `from` is a position known not to be past it
    size_t first_alive(int64_t t, size_t from = 0) const {
        while (from < rem.size() && rem[from] <= t) ++from;
        return from;
    }
    int64_t kv(size_t pos, int64_t t) const { return len_suf[pos] + (int64_t)(rem.size() - pos) * t; }
    // Between two departures the total grows by one token per request and iteration, so the largest
    // value before each departure is in the last iteration of the requests that leave.
    void peak(int64_t* peak_out, int32_t* iter_out) const {
        int64_t best = 0;
        int32_t when = 0;
        for (size_t i = 0; i < rem.size(); ++i) {
            if (i > 0 && rem[i] == rem[i - 1]) continue;
            const int64_t t = (int64_t)rem[i] - 1;
            const int64_t v = kv(i, t);
            if (v > best) best = v, when = (int32_t)t;
        }
        *peak_out = best;
        *iter_out = when;
    }
};

// attention work of a chunk of c tokens on `prior` earlier ones
double prefill_work(double flops_per_pair, int64_t c, int64_t prior) {
    return flops_per_pair * ((double)c * (double)prior + 0.5 * (double)c * ((double)c + 1.0));
}

}  // namespace
}  // namespace ps

using ps::fail;

extern "C" {

ps_status ps_table_from_lines(const int32_t* token_batch, const double* intercept_us, const double* slope_us_per_token,
                              const double* slope_us_per_flop, int32_t n_lines, ps_table** out) {
    ps::clear_error();
    if (!token_batch || !intercept_us || !slope_us_per_token || !out || n_lines < 1)
        return fail(PS_ERR_INVALID, "ps_table_from_lines: null pointer or n_lines < 1");
    std::vector<int32_t> order(n_lines);
    std::iota(order.begin(), order.end(), 0);
    std::sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return token_batch[a] < token_batch[b]; });
    ps_table* t = new (std::nothrow) ps_table;
    if (!t) return fail(PS_ERR_OOM, "ps_table_from_lines: out of host memory");
    for (int32_t k = 0; k < n_lines; ++k) {
        const int32_t i = order[k];
        const double pf_slope = slope_us_per_flop ? slope_us_per_flop[i] : 0.0;
        if (token_batch[i] < 1 || !std::isfinite(intercept_us[i]) || !std::isfinite(slope_us_per_token[i]) || !std::isfinite(pf_slope) ||
            (k > 0 && token_batch[i] == token_batch[order[k - 1]])) {
            delete t;
            return fail(PS_ERR_INVALID, "ps_table_from_lines: line %d (token_batch %d) is not usable or is a duplicate", i, token_batch[i]);
        }
        t->batch.push_back(token_batch[i]);
        t->intercept.push_back(intercept_us[i]);
        t->slope.push_back(slope_us_per_token[i]);
        t->slope_pf.push_back(pf_slope);
    }
    *out = t;
    return PS_OK;
}

ps_status ps_table_build(const ps_grid_row* rows, int64_t n_rows, ps_table** out) {
    ps::clear_error();
    if (!rows || !out || n_rows < 1) return fail(PS_ERR_INVALID, "ps_table_build: null pointer or n_rows < 1");
    if (ps_status st = ps::check_rows("ps_table_build", rows, n_rows)) return st;
    // rows of one batch size together, in their input order
    std::vector<int64_t> order(n_rows);
    std::iota(order.begin(), order.end(), (int64_t)0);
    std::stable_sort(order.begin(), order.end(), [&](int64_t a, int64_t b) { return rows[a].token_batch < rows[b].token_batch; });
    std::vector<int32_t> batch;
    std::vector<double> icpt, slope, slope_pf;
    for (int64_t g0 = 0; g0 < n_rows;) {
        int64_t g1 = g0;
        while (g1 < n_rows && rows[order[g1]].token_batch == rows[order[g0]].token_batch) ++g1;
        const ps::Plane f = ps::fit_plane(rows, order.data() + g0, g1 - g0);
        batch.push_back(rows[order[g0]].token_batch);
        slope.push_back(f.s);
        slope_pf.push_back(f.q);
        icpt.push_back(f.a);
        g0 = g1;
    }
    return ps_table_from_lines(batch.data(), icpt.data(), slope.data(), slope_pf.data(), (int32_t)batch.size(), out);
}

ps_status ps_table_build_overlap(const ps_grid_row* rows, int64_t n_rows, ps_table** out) {
    ps::clear_error();
    if (!rows || !out || n_rows < 1) return fail(PS_ERR_INVALID, "ps_table_build_overlap: null pointer or n_rows < 1");
    if (ps_status st = ps::check_rows("ps_table_build_overlap", rows, n_rows)) return st;
    std::vector<int64_t> all(n_rows);
    std::iota(all.begin(), all.end(), (int64_t)0);
    // start from the sum form over all rows: each row goes to the side whose term is the larger one there
    const ps::Plane sum = ps::fit_plane(rows, all.data(), n_rows);
    // (a slope below zero at the start would let that term fall with the work; it is taken as zero until fitted)
    double a_d = sum.a, s = std::max(sum.s, 0.0), a_p = sum.a, q = std::max(sum.q, 0.0);
    std::vector<char> on_decode(n_rows);
    auto side = [&](int64_t i, double dec, double pre) -> char {
        if (rows[i].prefill_flops == 0.0) return 1;
        if (rows[i].kv_tokens == 0) return 0;
        return dec >= pre ? 1 : 0;
    };
    for (int64_t i = 0; i < n_rows; ++i) on_decode[i] = side(i, s * (double)rows[i].kv_tokens, q * rows[i].prefill_flops);
    std::vector<int64_t> idx;
    for (int pass = 0; pass < 64; ++pass) {
        // one regressor per side: the other one's column is hidden from the fit
        for (int which = 1; which >= 0; --which) {
            idx.clear();
            for (int64_t i = 0; i < n_rows; ++i)
                if (on_decode[i] == which) idx.push_back(i);
            if (idx.size() < 2) continue;  // keeps the parameters it has
            const double n = (double)idx.size();
            double sum_x = 0.0, sum_y = 0.0;
            for (int64_t i : idx) sum_x += which ? (double)rows[i].kv_tokens : rows[i].prefill_flops, sum_y += (double)rows[i].latency_us;
            const double mx = sum_x / n, my = sum_y / n;
            double sxx = 0.0, sxy = 0.0;
            for (int64_t i : idx) {
                const double dx = (which ? (double)rows[i].kv_tokens : rows[i].prefill_flops) - mx;
                sxx += dx * dx, sxy += dx * ((double)rows[i].latency_us - my);
            }
            if (!(sxx > 0.0)) continue;
            const double slope = sxy / sxx;
            if (which) s = slope, a_d = my - slope * mx;
            else q = slope, a_p = my - slope * mx;
        }
        bool changed = false;
        for (int64_t i = 0; i < n_rows; ++i) {
            const char now = side(i, a_d + s * (double)rows[i].kv_tokens, a_p + q * rows[i].prefill_flops);
            changed = changed || now != on_decode[i];
            on_decode[i] = now;
        }
        if (!changed) break;
    }
    std::vector<int32_t> batch(n_rows);
    for (int64_t i = 0; i < n_rows; ++i) batch[i] = rows[i].token_batch;
    std::sort(batch.begin(), batch.end());
    batch.erase(std::unique(batch.begin(), batch.end()), batch.end());
    ps_table* t = new (std::nothrow) ps_table;
    if (!t) return fail(PS_ERR_OOM, "ps_table_build_overlap: out of host memory");
    const size_t n_lines = batch.size();
    t->batch = batch;
    t->overlap = true;
    t->intercept.assign(n_lines, 0.0);
    t->dec_icpt.assign(n_lines, a_d);
    t->slope.assign(n_lines, s);
    t->pf_icpt.assign(n_lines, a_p);
    t->slope_pf.assign(n_lines, q);
    *out = t;
    return PS_OK;
}

ps_status ps_table_get_overlap(const ps_table* table, int32_t* is_overlap_out, double* decode_intercept_us_out,
                               double* prefill_intercept_us_out, int32_t capacity) {
    ps::clear_error();
    if (!table || !is_overlap_out) return fail(PS_ERR_INVALID, "ps_table_get_overlap: null pointer");
    *is_overlap_out = table->overlap ? 1 : 0;
    if (!table->overlap || (!decode_intercept_us_out && !prefill_intercept_us_out)) return PS_OK;
    if (capacity < (int32_t)table->batch.size()) return fail(PS_ERR_INVALID, "ps_table_get_overlap: capacity %d < %zu lines", capacity, table->batch.size());
    for (size_t i = 0; i < table->batch.size(); ++i) {
        if (decode_intercept_us_out) decode_intercept_us_out[i] = table->dec_icpt[i];
        if (prefill_intercept_us_out) prefill_intercept_us_out[i] = table->pf_icpt[i];
    }
    return PS_OK;
}

ps_status ps_table_free(ps_table* table) {
    delete table;
    return PS_OK;
}

ps_status ps_table_add_batch_term(ps_table* table, const int32_t* token_batch, const double* term_us, int32_t n) {
    ps::clear_error();
    if (!table || !token_batch || !term_us || n < 1) return fail(PS_ERR_INVALID, "ps_table_add_batch_term: null pointer or n < 1");
    std::vector<int32_t> order(n);
    std::iota(order.begin(), order.end(), 0);
    std::sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return token_batch[a] < token_batch[b]; });
    for (int32_t k = 0; k < n; ++k) {
        const int32_t i = order[k];
        if (token_batch[i] < 1 || !std::isfinite(term_us[i]) || (k > 0 && token_batch[i] == token_batch[order[k - 1]]))
            return fail(PS_ERR_INVALID, "ps_table_add_batch_term: sample %d (token_batch %d) is not usable or is a duplicate", i, token_batch[i]);
    }
    for (size_t l = 0; l < table->batch.size(); ++l) {
        const int32_t b = table->batch[l];
        double term;
        if (b <= token_batch[order.front()]) {
            term = term_us[order.front()];
        } else if (b >= token_batch[order.back()]) {
            term = term_us[order.back()];
        } else {
            int32_t k = 0;
            while (token_batch[order[k + 1]] <= b) ++k;  // samples k, k + 1 with batch[k] <= b < batch[k + 1]
            const int32_t lo = order[k], hi = order[k + 1];
            term = term_us[lo] + (term_us[hi] - term_us[lo]) * ((double)(b - token_batch[lo]) / (double)(token_batch[hi] - token_batch[lo]));
        }
        table->intercept[l] += term;
    }
    return PS_OK;
}

ps_status ps_table_scale(ps_table* table, double factor) {
    ps::clear_error();
    if (!table || !(factor > 0.0) || !std::isfinite(factor)) return fail(PS_ERR_INVALID, "ps_table_scale: null table or factor %g", factor);
    for (size_t l = 0; l < table->batch.size(); ++l) {
        table->intercept[l] *= factor;
        table->slope[l] *= factor;
        table->slope_pf[l] *= factor;
        if (table->overlap) table->dec_icpt[l] *= factor, table->pf_icpt[l] *= factor;
    }
    return PS_OK;
}

ps_status ps_table_size(const ps_table* table, int32_t* n_lines_out) {
    ps::clear_error();
    if (!table || !n_lines_out) return fail(PS_ERR_INVALID, "ps_table_size: null pointer");
    *n_lines_out = (int32_t)table->batch.size();
    return PS_OK;
}

ps_status ps_table_get_lines(const ps_table* table, int32_t* token_batch_out, double* intercept_us_out,
                             double* slope_us_per_token_out, double* slope_us_per_flop_out, int32_t capacity) {
    ps::clear_error();
    if (!table) return fail(PS_ERR_INVALID, "ps_table_get_lines: null table");
    if (capacity < (int32_t)table->batch.size()) return fail(PS_ERR_INVALID, "ps_table_get_lines: capacity %d < %zu lines", capacity, table->batch.size());
    for (size_t i = 0; i < table->batch.size(); ++i) {
        if (token_batch_out) token_batch_out[i] = table->batch[i];
        if (intercept_us_out) intercept_us_out[i] = table->intercept[i];
        if (slope_us_per_token_out) slope_us_per_token_out[i] = table->slope[i];
        if (slope_us_per_flop_out) slope_us_per_flop_out[i] = table->slope_pf[i];
    }
    return PS_OK;
}

ps_status ps_table_predict(const ps_table* table, int32_t token_batch, int64_t kv_tokens, double prefill_flops, double* latency_us_out) {
    ps::clear_error();
    if (!table || !latency_us_out) return fail(PS_ERR_INVALID, "ps_table_predict: null pointer");
    if (token_batch < 1 || kv_tokens < 0 || !(prefill_flops >= 0.0) || !std::isfinite(prefill_flops))
        return fail(PS_ERR_INVALID, "ps_table_predict: token_batch %d, kv_tokens %lld, prefill_flops %g", token_batch, (long long)kv_tokens, prefill_flops);
    *latency_us_out = ps::predict(*table, token_batch, kv_tokens, prefill_flops);
    return PS_OK;
}

ps_status ps_peak_kv(const int32_t* kv_len, const int32_t* remaining, int32_t n, int64_t* peak_kv_out, int32_t* peak_iter_out) {
    ps::clear_error();
    if (!peak_kv_out || !peak_iter_out) return fail(PS_ERR_INVALID, "ps_peak_kv: null output");
    if (ps_status st = ps::check_requests(kv_len, remaining, n)) return st;
    ps::Future(kv_len, remaining, n).peak(peak_kv_out, peak_iter_out);
    return PS_OK;
}

ps_status ps_admit(const ps_table* table, const int32_t* kv_len, const int32_t* remaining, int32_t n_running, int32_t new_kv_len,
                   int32_t new_remaining, int32_t extra_tokens, int64_t extra_kv_tokens, double extra_prefill_flops, double tpot_us,
                   int32_t* admit_out, double* predicted_us_out, int64_t* peak_kv_out) {
    ps::clear_error();
    if (!table) return fail(PS_ERR_INVALID, "ps_admit: null table");
    if (extra_tokens < 0 || extra_kv_tokens < 0 || !(extra_prefill_flops >= 0.0) || !std::isfinite(extra_prefill_flops))
        return fail(PS_ERR_INVALID, "ps_admit: extra_tokens %d, extra_kv_tokens %lld, extra_prefill_flops %g", extra_tokens,
                    (long long)extra_kv_tokens, extra_prefill_flops);
    if (ps_status st = ps::check_requests(kv_len, remaining, n_running)) return st;
    if (ps_status st = ps::check_requests(&new_kv_len, &new_remaining, 1)) return st;
    std::vector<int32_t> len(kv_len, kv_len + n_running), rem(remaining, remaining + n_running);
    len.push_back(new_kv_len);
    rem.push_back(new_remaining);
    int64_t peak = 0;
    int32_t when = 0;
    ps::Future(len.data(), rem.data(), n_running + 1).peak(&peak, &when);
    const double pred = ps::predict(*table, n_running + 1 + extra_tokens, peak + extra_kv_tokens, extra_prefill_flops);
    if (admit_out) *admit_out = pred < tpot_us ? 1 : 0;
    if (predicted_us_out) *predicted_us_out = pred;
    if (peak_kv_out) *peak_kv_out = peak;
    return PS_OK;
}

ps_status ps_chunk_next(const int32_t* remaining, int32_t n, int32_t budget, int32_t used, int32_t dynamic, int32_t* chunk_out) {
    ps::clear_error();
    if (n < 0 || (n > 0 && (!remaining || !chunk_out))) return fail(PS_ERR_INVALID, "ps_chunk_next: n = %d with a null pointer", n);
    if (budget < 1 || used < 0) return fail(PS_ERR_INVALID, "ps_chunk_next: budget %d, used %d", budget, used);
    for (int32_t i = 0; i < n; ++i)
        if (remaining[i] < 1) return fail(PS_ERR_INVALID, "ps_chunk_next: remaining[%d] = %d", i, remaining[i]);
    int64_t left = (int64_t)budget - used;
    int32_t i = 0;
    for (; i < n && left > 0; ++i) {
        if (dynamic && remaining[i] < 2 * (int64_t)budget) {
            chunk_out[i] = remaining[i];  // finished at once; the iteration is closed behind it
            ++i;
            break;
        }
        chunk_out[i] = (int32_t)std::min<int64_t>(remaining[i], left);
        left -= chunk_out[i];
    }
    for (; i < n; ++i) chunk_out[i] = 0;
    return PS_OK;
}

ps_status ps_chunk_schedule(int32_t prompt_len, int32_t budget, int32_t first_free, int32_t dynamic, int32_t* chunks_out,
                            int32_t capacity, int32_t* n_chunks_out) {
    ps::clear_error();
    if (!n_chunks_out || (capacity > 0 && !chunks_out) || capacity < 0) return fail(PS_ERR_INVALID, "ps_chunk_schedule: null pointer");
    if (prompt_len < 1 || budget < 1 || first_free < 0 || first_free > budget)
        return fail(PS_ERR_INVALID, "ps_chunk_schedule: prompt_len %d, budget %d, first_free %d", prompt_len, budget, first_free);
    int32_t n = 0, rem = prompt_len, used = budget - first_free;
    while (rem > 0) {
        int32_t c = 0;
        ps_status st = ps_chunk_next(&rem, 1, budget, used, dynamic, &c);
        if (st) return st;
        if (c > 0) {
            if (n < capacity) chunks_out[n] = c;
            ++n;
            rem -= c;
        }
        used = 0;
    }
    *n_chunks_out = n;
    if (n > capacity) return fail(PS_ERR_INVALID, "ps_chunk_schedule: %d chunks do not fit a capacity of %d", n, capacity);
    return PS_OK;
}

ps_status ps_chunk_predict(const ps_table* table, const int32_t* kv_len, const int32_t* remaining, int32_t n_running,
                           int32_t prompt_len, int32_t max_chunk, double flops_per_pair, double tpot_us, int32_t* chunk_out,
                           int32_t* n_iters_out, double* completion_us_out, int32_t* maintained_out) {
    ps::clear_error();
    if (!table || !chunk_out || !n_iters_out || !completion_us_out || !maintained_out) return fail(PS_ERR_INVALID, "ps_chunk_predict: null pointer");
    if (prompt_len < 1 || max_chunk < 1 || !(flops_per_pair >= 0.0) || !std::isfinite(flops_per_pair))
        return fail(PS_ERR_INVALID, "ps_chunk_predict: prompt_len %d, max_chunk %d, flops_per_pair %g", prompt_len, max_chunk, flops_per_pair);
    if (ps_status st = ps::check_requests(kv_len, remaining, n_running)) return st;
    const ps::Future fut(kv_len, remaining, n_running);
    const int64_t kv0 = fut.kv(0, 0);
    int32_t chunk = 0;
    for (int32_t c = std::min(prompt_len, max_chunk); c >= 1; --c)
        if (ps::predict(*table, n_running + c, kv0 + c, ps::prefill_work(flops_per_pair, c, 0)) <= tpot_us) {
            chunk = c;
            break;
        }
    *chunk_out = chunk;
    *n_iters_out = 0;
    *completion_us_out = 0.0;
    *maintained_out = 0;
    if (chunk == 0) return PS_OK;
    const int32_t iters = (int32_t)(((int64_t)prompt_len + chunk - 1) / chunk);
    double total = 0.0;
    bool kept = true;
    size_t pos = 0;
    for (int32_t k = 0; k < iters; ++k) {
        pos = fut.first_alive(k, pos);
        const int64_t alive = (int64_t)n_running - (int64_t)pos;
        const int64_t done = std::min<int64_t>((int64_t)(k + 1) * chunk, prompt_len);
        const int64_t c_k = std::min<int64_t>(chunk, (int64_t)prompt_len - (int64_t)k * chunk);
        const double pred = ps::predict(*table, (int32_t)(alive + c_k), fut.kv(pos, k) + done, ps::prefill_work(flops_per_pair, c_k, (int64_t)k * chunk));
        total += pred;
        kept = kept && pred <= tpot_us;
    }
    *n_iters_out = iters;
    *completion_us_out = total;
    *maintained_out = kept ? 1 : 0;
    return PS_OK;
}

}  // extern "C"
