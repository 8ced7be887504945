"""CPU oracle for the scheduler-side consumers of the latency table (test infrastructure).

Plain, slow Python written from the paper's text; only the tests and the
bench scripts' baseline legs may import it, the library and its binding never
do.  Every function simulates or enumerates directly -- no sweeps, no sorting
tricks, no closed forms -- so that it can be checked against the paper by eye.

Notation (paper section 4.5): a running decode request holds ``kv_len`` tokens
in the cache (the token of the coming iteration included) and still has
``remaining`` tokens to generate (that one included).  Iterations are numbered
t = 0, 1, ... from the coming one; the request takes part in iterations
0 .. remaining - 1 and holds ``kv_len + t`` tokens in iteration t.

parity pins: tests/test_sched_oracle_pins.py (the paper's chunk-schedule
example, closed forms, numpy's least-squares routine, brute force by explicit
matrices).
"""
from __future__ import annotations


# ---------------------------------------------------------------------------
# latency table (section 4.5: a profiled map of (batch size, KV cache size) to execution time)
# ---------------------------------------------------------------------------
def table_build(rows):
    """rows: iterable of (token_batch, kv_tokens, prefill_flops, latency_us).  Returns the table as a list of
    lines (token_batch, intercept_us, slope_us_per_token, slope_us_per_flop) sorted by token_batch: per batch
    size the ordinary least-squares fit latency = intercept + slope_kv kv_tokens + slope_pf prefill_flops
    (section 3.4: an iteration is a batch-size term plus decode attention, a function of the KV-cache size, plus
    prefill attention, a function of the prefill work).  Normal equations on centred sums; a regressor that does
    not vary within the line, or the second of two collinear ones, is left out (slope 0)."""
    groups = {}
    for b, kv, pf, lat in rows:
        groups.setdefault(int(b), []).append((float(kv), float(pf), float(lat)))
    lines = []
    for b in sorted(groups):
        pts = groups[b]
        n = len(pts)
        mx = sum(x for x, _, _ in pts) / n
        mp = sum(q for _, q, _ in pts) / n
        my = sum(y for _, _, y in pts) / n
        sxx = sum((x - mx) * (x - mx) for x, _, _ in pts)
        spp = sum((q - mp) * (q - mp) for _, q, _ in pts)
        sxp = sum((x - mx) * (q - mp) for x, q, _ in pts)
        sxy = sum((x - mx) * (y - my) for x, _, y in pts)
        spy = sum((q - mp) * (y - my) for _, q, y in pts)
        det = sxx * spp - sxp * sxp
        if sxx > 0.0 and spp > 0.0 and det > 1e-9 * sxx * spp:
            s_kv = (sxy * spp - spy * sxp) / det
            s_pf = (spy * sxx - sxy * sxp) / det
        elif sxx > 0.0:
            s_kv, s_pf = sxy / sxx, 0.0
        elif spp > 0.0:
            s_kv, s_pf = 0.0, spy / spp
        else:
            s_kv, s_pf = 0.0, 0.0
        lines.append((b, my - s_kv * mx - s_pf * mp, s_kv, s_pf))
    return lines


def table_predict(lines, token_batch, kv_tokens, prefill_flops=0.0):
    """Predicted iteration time: the line of that batch size evaluated at (kv_tokens, prefill_flops); between two
    lines their two values interpolated linearly in the batch size; outside the lines the nearest line as it is."""
    lines = sorted(lines)

    def at(ln):
        if len(ln) == 4:  # sum form
            return ln[1] + ln[2] * float(kv_tokens) + ln[3] * float(prefill_flops)
        _, base, a_d, s, a_p, q = ln  # overlap form, see table_build_overlap
        dec, pre = a_d + s * float(kv_tokens), a_p + q * float(prefill_flops)
        if prefill_flops == 0:
            return base + dec
        if kv_tokens == 0:
            return base + pre
        return base + max(dec, pre)

    if token_batch <= lines[0][0]:
        return at(lines[0])
    if token_batch >= lines[-1][0]:
        return at(lines[-1])
    for lo, hi in zip(lines[:-1], lines[1:]):
        if lo[0] <= token_batch < hi[0]:
            w = (token_batch - lo[0]) / float(hi[0] - lo[0])
            return at(lo) + (at(hi) - at(lo)) * w
    raise AssertionError("unreachable")


def table_build_overlap(rows):
    """The sweep fitted for an engine that runs the decode rows and the prefill chunk of a batch side by side: a
    mixed batch then takes about as long as the slower part, latency = base + max(a_d + s kv_tokens, a_p + q
    prefill_flops), the prefill term absent without a chunk and the decode term without KV tokens (section 3.4 adds
    the terms, for parts that run one after the other).  One set of four parameters for the whole sweep, found by
    alternating least squares: start from the sum form fitted over all rows (a_d = a_p = its intercept, a negative
    slope taken as 0); give each
    row to the side whose term is larger (rows without prefill work to the decode side, rows without KV tokens to
    the prefill side, ties to the decode side; at the start the terms are compared without intercepts); fit each
    side's line on its own rows and its own regressor (a side with fewer than two rows or a constant regressor
    keeps what it has), decode side first; assign again; stop when no row moves or after 64 rounds.  Returns one
    line (token_batch, base = 0, a_d, s, a_p, q) per distinct batch size, all with the same four parameters."""
    rows = [(int(b), float(kv), float(pf), float(lat)) for b, kv, pf, lat in rows]
    (_, a, s, q), = table_build([(1, kv, pf, lat) for _, kv, pf, lat in rows])
    a_d = a_p = a
    s, q = max(s, 0.0), max(q, 0.0)

    def side(kv, pf, dec, pre):
        if pf == 0.0:
            return "decode"
        if kv == 0.0:
            return "prefill"
        return "decode" if dec >= pre else "prefill"

    sides = [side(kv, pf, s * kv, q * pf) for _, kv, pf, _ in rows]
    for _ in range(64):
        for which in ("decode", "prefill"):
            pts = [((kv if which == "decode" else pf), lat) for (_, kv, pf, lat), z in zip(rows, sides) if z == which]
            if len(pts) < 2:
                continue
            mx = sum(x for x, _ in pts) / len(pts)
            my = sum(y for _, y in pts) / len(pts)
            sxx = sum((x - mx) * (x - mx) for x, _ in pts)
            sxy = sum((x - mx) * (y - my) for x, y in pts)
            if not sxx > 0.0:
                continue
            if which == "decode":
                s = sxy / sxx
                a_d = my - s * mx
            else:
                q = sxy / sxx
                a_p = my - q * mx
        again = [side(kv, pf, a_d + s * kv, a_p + q * pf) for _, kv, pf, _ in rows]
        if again == sides:
            break
        sides = again
    return [(b, 0.0, a_d, s, a_p, q) for b in sorted({b for b, _, _, _ in rows})]


def table_add_batch_term(lines, samples):
    """The table with a term that depends on the token batch size alone added to every line (section 3.4: the
    GEMMs and collectives of an iteration depend on the batch size only).  samples: (token_batch, microseconds)
    pairs; between two samples the term is interpolated linearly, outside them the nearest sample is used."""
    samples = sorted(samples)

    def term(b):
        if b <= samples[0][0]:
            return samples[0][1]
        if b >= samples[-1][0]:
            return samples[-1][1]
        for lo, hi in zip(samples[:-1], samples[1:]):
            if lo[0] <= b < hi[0]:
                return lo[1] + (hi[1] - lo[1]) * ((b - lo[0]) / float(hi[0] - lo[0]))
        raise AssertionError("unreachable")

    return [(ln[0], ln[1] + term(ln[0])) + tuple(ln[2:]) for ln in lines]


def table_scale(lines, factor):
    """Every coefficient times factor (a model of n identical layers is n times one layer)."""
    return [(ln[0],) + tuple(c * factor for c in ln[1:]) for ln in lines]


# ---------------------------------------------------------------------------
# decode admission (section 4.5: simulate future iterations, take the largest KV-cache size)
# ---------------------------------------------------------------------------
def kv_at(kv_len, remaining, t):
    """Total KV tokens and number of requests in iteration t."""
    alive = [L + t for L, R in zip(kv_len, remaining) if R > t]
    return sum(alive), len(alive)


def peak_kv(kv_len, remaining):
    """(largest total KV-cache size over the future iterations, first iteration where it occurs)."""
    peak, when = 0, 0
    horizon = max(remaining) if len(remaining) else 0
    for t in range(horizon):  # admission look-ahead (section 4.5): step iteration by iteration until every request is done
        kv, _ = kv_at(kv_len, remaining, t)
        if kv > peak:
            peak, when = kv, t
    return peak, when


def admit(lines, kv_len, remaining, new_kv_len, new_remaining, extra_tokens, extra_kv_tokens, extra_prefill_flops, tpot_us):
    """(admitted?, predicted iteration time, peak KV of the decode requests) for one new decode request: the table
    at the current token batch size and the largest future KV-cache size must stay below the TPOT.  Prefill
    tokens batched alongside add their tokens, the K/V of their rows and their attention work to the lookup."""
    peak, _ = peak_kv(list(kv_len) + [new_kv_len], list(remaining) + [new_remaining])
    batch = len(kv_len) + 1 + extra_tokens
    pred = table_predict(lines, batch, peak + extra_kv_tokens, extra_prefill_flops)
    return pred < tpot_us, pred, peak


# ---------------------------------------------------------------------------
# prefill chunking (section 4.7)
# ---------------------------------------------------------------------------
def chunk_next(remaining, budget, used, dynamic):
    """Chunk length per request for the coming iteration, first come first served.  Dynamic chunking: a request
    with fewer than two budgets of prompt left is finished at once and nobody is admitted behind it."""
    left = budget - used
    out = [0] * len(remaining)
    for i, rem in enumerate(remaining):
        if left <= 0:
            break
        if dynamic and rem < 2 * budget:
            out[i] = rem
            break
        out[i] = min(rem, left)
        left -= out[i]
    return out


def chunk_schedule(prompt_len, budget, first_free, dynamic):
    """All chunks of one prompt; the first iteration has only first_free tokens of its budget left."""
    chunks, rem, used = [], prompt_len, budget - first_free
    while rem > 0:
        c = chunk_next([rem], budget, used, dynamic)[0]
        if c > 0:
            chunks.append(c)
            rem -= c
        used = 0
    return chunks


def prefill_work(flops_per_pair, c, prior):
    """Attention work of a chunk of c tokens on `prior` earlier ones: token i sees prior + i + 1 keys."""
    return flops_per_pair * (float(c) * float(prior) + 0.5 * float(c) * (float(c) + 1.0))


def chunk_predict(lines, kv_len, remaining, prompt_len, max_chunk, flops_per_pair, tpot_us):
    """Continuous chunked-prefill prediction.  Returns (chunk, iterations, completion_us, maintained)."""
    kv0, n0 = kv_at(kv_len, remaining, 0)
    chunk = 0
    for c in range(min(prompt_len, max_chunk), 0, -1):
        if table_predict(lines, n0 + c, kv0 + c, prefill_work(flops_per_pair, c, 0)) <= tpot_us:
            chunk = c
            break
    if chunk == 0:
        return 0, 0, 0.0, False
    iters = -(-prompt_len // chunk)  # ceil
    completion, maintained = 0.0, True
    for k in range(iters):
        kv, n = kv_at(kv_len, remaining, k)
        c_k = min(chunk, prompt_len - k * chunk)
        pred = table_predict(lines, n + c_k, kv + min((k + 1) * chunk, prompt_len), prefill_work(flops_per_pair, c_k, k * chunk))
        completion += pred
        maintained = maintained and pred <= tpot_us
    return chunk, iters, completion, maintained
