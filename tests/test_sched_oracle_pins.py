"""Pins of the scheduler-side oracle (oracle/sched_oracle.py) against things other than itself: the paper's
worked chunk-schedule example (section 4.7), closed forms, numpy's least-squares routine and explicit-matrix
brute force."""
import os

import numpy as np
import pytest

from oracle import sched_oracle as so

HERE = os.path.dirname(os.path.abspath(__file__))


def read_example():
    out = {}
    for line in open(os.path.join(HERE, "golden", "dynamic_chunking_example.txt")):
        line = line.strip()
        if line and not line.startswith("#"):
            name, *vals = line.split()
            out[name] = [int(v) for v in vals]
    return out


# ---------------------------------------------------------------------------
# chunk schedules: the paper's example, section 4.7
# ---------------------------------------------------------------------------
def test_chunk_schedules_of_the_papers_example():
    ex = read_example()
    budget, prompt = ex["budget"][0], ex["prompt"][0]
    assert so.chunk_schedule(prompt, budget, budget, dynamic=False) == ex["static"]
    assert so.chunk_schedule(prompt, budget, 1, dynamic=False) == ex["static_worst"]
    assert so.chunk_schedule(prompt, budget, budget, dynamic=True) == ex["dynamic"]
    # "allows almost every request to reduce one iteration": the worst case drops from four iterations to three
    worst_dynamic = so.chunk_schedule(prompt, budget, 1, dynamic=True)
    assert worst_dynamic == [1, 1024, 1025] and len(worst_dynamic) == len(ex["static_worst"]) - 1


def test_chunk_schedule_invariants():
    rng = np.random.default_rng(5)
    for _ in range(300):
        budget = int(rng.integers(1, 600))
        prompt = int(rng.integers(1, 6 * budget + 2))
        free = int(rng.integers(1, budget + 1))
        st = so.chunk_schedule(prompt, budget, free, False)
        dy = so.chunk_schedule(prompt, budget, free, True)
        assert sum(st) == prompt and sum(dy) == prompt
        assert st[0] <= free and all(c <= budget for c in st)
        # static chunking is ceil((prompt - first) / budget) + 1 iterations
        first = min(prompt, free)
        assert len(st) == 1 + -(-(prompt - first) // budget)
        assert all(c < 2 * budget for c in dy) and len(dy) <= len(st)
        # only the last dynamic chunk may exceed what was free in its iteration
        assert all(c <= budget for c in dy[:-1])


def test_chunk_next_is_first_come_first_served():
    # plain chunked prefill fills the budget in order
    assert so.chunk_next([300, 500, 900], 1024, 0, False) == [300, 500, 224]
    assert so.chunk_next([300, 500, 900], 1024, 1000, False) == [24, 0, 0]
    assert so.chunk_next([300], 1024, 1024, False) == [0]
    # dynamic: the first request with fewer than two budgets left is finished at once and closes the iteration
    assert so.chunk_next([5000, 1500, 10], 1024, 0, True) == [1024, 0, 0]
    assert so.chunk_next([2047, 10], 1024, 0, True) == [2047, 0]
    assert so.chunk_next([2048, 10], 1024, 0, True) == [1024, 0]
    assert so.chunk_next([3000, 10], 1024, 1000, True) == [24, 0]
    assert so.chunk_next([10, 3000], 1024, 1000, True) == [10, 0]


# ---------------------------------------------------------------------------
# peak KV of the simulated future iterations, section 4.5
# ---------------------------------------------------------------------------
def test_peak_kv_closed_forms():
    # one request: it grows by one token per iteration until its last one
    assert so.peak_kv([100], [7]) == (106, 6)
    # equal remaining lengths: everybody is there until the end
    assert so.peak_kv([10, 20, 30], [5, 5, 5]) == (60 + 3 * 4, 4)
    # a long context that leaves at once dominates: the peak is now
    assert so.peak_kv([10, 1000], [3, 1]) == (1010, 0)
    # worked by hand: t0 = 5+6+7 = 18, t1 = 6+7 = 13 (third left), t2 = 7 (second left)
    assert so.peak_kv([5, 6, 7], [3, 2, 1]) == (18, 0)
    assert so.peak_kv([5, 6, 7], [4, 4, 1]) == (18, 0)   # t0 18, t1 13, t2 15, t3 17
    assert so.peak_kv([5, 6, 7], [5, 5, 1]) == (19, 4)   # ... t4 = 9 + 10 = 19
    assert so.peak_kv([10, 3], [4, 1]) == (13, 0)        # t0 13, t1 11, t2 12, t3 13: a tie reports the first
    assert so.peak_kv([], []) == (0, 0)


def test_peak_kv_against_explicit_matrix():
    rng = np.random.default_rng(11)
    for _ in range(200):
        n = int(rng.integers(1, 40))
        kv = rng.integers(1, 5000, n)
        rem = rng.integers(1, 300, n)
        t = np.arange(rem.max())[:, None]                       # iterations x requests
        total = ((kv[None, :] + t) * (rem[None, :] > t)).sum(axis=1)
        assert so.peak_kv(kv.tolist(), rem.tolist()) == (int(total.max()), int(total.argmax()))


def test_peak_kv_monotone_in_the_request_set():
    rng = np.random.default_rng(12)
    for _ in range(100):
        n = int(rng.integers(1, 20))
        kv, rem = rng.integers(1, 3000, n).tolist(), rng.integers(1, 200, n).tolist()
        base, _ = so.peak_kv(kv, rem)
        more, _ = so.peak_kv(kv + [int(rng.integers(1, 3000))], rem + [int(rng.integers(1, 200))])
        assert more > base  # the newcomer is present at iteration 0 at least... and at the old peak or earlier
        assert more >= so.kv_at(kv, rem, 0)[0]


# ---------------------------------------------------------------------------
# table: least-squares lines and the lookup
# ---------------------------------------------------------------------------
def test_table_fit_recovers_exact_lines_and_matches_numpy():
    rng = np.random.default_rng(3)
    rows = []
    truth = {72: (15.0, 2.5e-4, 0.0), 320: (40.0, 3.0e-4, 0.0), 2304: (310.0, 1.0e-4, 0.0)}
    for b, (a, s, _) in truth.items():
        for kv in rng.integers(1000, 2_000_000, 27):
            rows.append((b, int(kv), 0.0, a + s * float(kv)))   # no chunk: the prefill regressor does not vary
    lines = so.table_build(rows)
    assert [ln[0] for ln in lines] == sorted(truth)
    for b, a, s, q in lines:
        assert abs(a - truth[b][0]) < 1e-6 and abs(s - truth[b][1]) < 1e-12 and q == 0.0
    # noisy data: the same coefficients as numpy's least squares
    noisy = [(b, kv, pf, lat * (1.0 + 0.05 * rng.standard_normal())) for b, kv, pf, lat in rows]
    for b, a, s, q in so.table_build(noisy):
        x = np.array([kv for bb, kv, _, _ in noisy if bb == b], dtype=np.float64)
        y = np.array([lat for bb, _, _, lat in noisy if bb == b], dtype=np.float64)
        coef, *_ = np.linalg.lstsq(np.stack([np.ones_like(x), x], axis=1), y, rcond=None)
        assert abs(a - coef[0]) < 1e-6 * max(1.0, abs(coef[0])) and abs(s - coef[1]) < 1e-9 * abs(coef[1])
    # a line whose rows share one KV size: slope 0 and their mean
    flat = so.table_build([(8, 500, 0.0, 10.0), (8, 500, 0.0, 14.0)])
    assert flat == [(8, 12.0, 0.0, 0.0)]


def test_table_fit_with_the_prefill_term():
    rng = np.random.default_rng(4)
    # exact planes are recovered
    rows, truth = [], {1032: (42.0, 6.0e-4, 1.1e-9), 2056: (60.0, 6.5e-4, 0.9e-9)}
    for b, (a, s, q) in truth.items():
        for _ in range(27):
            kv, pf = int(rng.integers(10_000, 300_000)), float(rng.uniform(1e9, 4e11))
            rows.append((b, kv, pf, a + s * kv + q * pf))
    for b, a, s, q in so.table_build(rows):
        assert abs(a - truth[b][0]) < 1e-6 and abs(s - truth[b][1]) < 1e-12 and abs(q - truth[b][2]) < 1e-18
    # noisy: numpy's least squares on [1, kv, pf] (columns scaled for its conditioning), and residual orthogonal to the regressors
    noisy = [(b, kv, pf, lat * (1.0 + 0.05 * rng.standard_normal())) for b, kv, pf, lat in rows]
    for b, a, s, q in so.table_build(noisy):
        x = np.array([kv for bb, kv, _, _ in noisy if bb == b], dtype=np.float64)
        w = np.array([pf for bb, _, pf, _ in noisy if bb == b], dtype=np.float64)
        y = np.array([lat for bb, _, _, lat in noisy if bb == b], dtype=np.float64)
        coef, *_ = np.linalg.lstsq(np.stack([np.ones_like(x), x / 1e5, w / 1e11], axis=1), y, rcond=None)
        assert abs(a - coef[0]) < 1e-6 * max(1.0, abs(coef[0]))
        assert abs(s - coef[1] / 1e5) < 1e-8 * abs(coef[1] / 1e5) and abs(q - coef[2] / 1e11) < 1e-8 * abs(coef[2] / 1e11)
        res = y - (a + s * x + q * w)
        assert abs(res.sum()) < 1e-6 * np.abs(y).sum() and abs((res * (x - x.mean())).sum()) < 1e-6 * np.abs(y * x).sum()
        assert abs((res * (w - w.mean())).sum()) < 1e-6 * np.abs(y * w).sum()
    # collinear regressors: the prefill term is left out, the KV line is fitted alone
    col = so.table_build([(520, kv, 3.0e5 * kv, 20.0 + 7e-4 * kv) for kv in (1000, 2000, 5000, 9000)])
    assert col[0][3] == 0.0 and abs(col[0][2] - 7e-4) < 1e-12 and abs(col[0][1] - 20.0) < 1e-9
    # only the prefill work varies
    pf_only = so.table_build([(520, 4000, pf, 30.0 + 1e-9 * pf) for pf in (1e9, 5e9, 2e10)])
    assert pf_only[0][2] == 0.0 and abs(pf_only[0][3] - 1e-9) < 1e-18 and abs(pf_only[0][1] - 30.0) < 1e-9


def test_table_lookup_interpolates_in_batch_and_clamps():
    lines = [(100, 10.0, 1e-3, 0.0), (300, 50.0, 2e-3, 1e-9)]
    assert so.table_predict(lines, 100, 1000) == pytest.approx(11.0)
    assert so.table_predict(lines, 300, 1000) == pytest.approx(52.0)
    assert so.table_predict(lines, 200, 1000) == pytest.approx(0.5 * (11.0 + 52.0))   # midpoint
    assert so.table_predict(lines, 150, 0) == pytest.approx(10.0 + 0.25 * 40.0)
    assert so.table_predict(lines, 5, 1000) == pytest.approx(11.0)                   # below: first line
    assert so.table_predict(lines, 9000, 1000) == pytest.approx(52.0)                # above: last line
    assert so.table_predict(list(reversed(lines)), 200, 1000) == pytest.approx(31.5)  # order of the lines is free
    # the prefill work enters through each line's own coefficient
    assert so.table_predict(lines, 300, 1000, 4e9) == pytest.approx(56.0)
    assert so.table_predict(lines, 100, 1000, 4e9) == pytest.approx(11.0)
    assert so.table_predict(lines, 200, 1000, 4e9) == pytest.approx(0.5 * (11.0 + 56.0))


def test_batch_term_and_scaling():
    lines = [(100, 10.0, 1e-3, 1e-9), (200, 20.0, 2e-3, 2e-9), (900, 50.0, 3e-3, 0.0)]
    # GEMM(B) sampled at 64, 128 and 512 tokens: 100 -> 30 + 36/64 * 20 = 41.25, 200 -> 50 + 72/384 * 100, 900 -> clamped
    got = so.table_add_batch_term(lines, [(512, 150.0), (64, 30.0), (128, 50.0)])
    assert [ln[0] for ln in got] == [100, 200, 900]
    assert got[0][1] == pytest.approx(10.0 + 41.25) and got[1][1] == pytest.approx(20.0 + 50.0 + 72.0 / 384.0 * 100.0)
    assert got[2][1] == pytest.approx(50.0 + 150.0)
    assert [ln[2:] for ln in got] == [ln[2:] for ln in lines]          # the slopes are untouched
    assert so.table_add_batch_term(lines, [(300, 7.0)])[0][1] == pytest.approx(17.0)  # one sample: a constant
    # a sum of per-layer terms over 32 layers is 32 times every coefficient, hence 32 times every prediction
    x32 = so.table_scale(lines, 32.0)
    for b, kv, pf in [(100, 5000, 0.0), (150, 123456, 3e9), (5000, 10, 1e12)]:
        assert so.table_predict(x32, b, kv, pf) == pytest.approx(32.0 * so.table_predict(lines, b, kv, pf))


def test_admission_uses_the_peak_and_the_current_batch_size():
    # table(b, kv) = 2 b + 0.01 kv
    lines = [(1, 2.0, 0.01, 1e-9), (1001, 2002.0, 0.01, 1e-9)]
    kv, rem = [100, 200], [10, 3]
    # with the newcomer (50 tokens, 5 to go): t0 = 350, t1 = 353, t2 = 356, t3 = 103+53 = 156, t4 = 158 -> peak 356
    ok, pred, peak = so.admit(lines, kv, rem, 50, 5, 0, 0, 0.0, 10.0)
    assert peak == 356 and pred == pytest.approx(2 * 3 + 3.56) and ok
    assert not so.admit(lines, kv, rem, 50, 5, 0, 0, 0.0, 9.56)[0]          # strictly below the TPOT is required
    assert so.admit(lines, kv, rem, 50, 5, 0, 0, 0.0, 9.5601)[0]
    # prefill tokens batched alongside: their tokens, the K/V of their rows and their attention work join the lookup
    ok, pred, peak = so.admit(lines, kv, rem, 50, 5, 100, 0, 0.0, 1e9)
    assert peak == 356 and pred == pytest.approx(2 * 103 + 3.56)
    ok, pred, peak = so.admit(lines, kv, rem, 50, 5, 100, 1100, 3e9, 1e9)
    assert peak == 356 and pred == pytest.approx(2 * 103 + 0.01 * (356 + 1100) + 3.0)


def test_chunk_prediction_closed_form():
    # table(b, kv) = alpha b + beta kv, no decode requests: chunk c costs (alpha + beta) c in iteration 0
    alpha, beta = 0.1, 0.002
    lines = [(1, alpha, beta, 0.0), (100001, alpha * 100001, beta, 0.0)]
    tpot = 50.0
    c, iters, total, kept = so.chunk_predict(lines, [], [], 3000, 2048, 16384.0, tpot)
    assert c == int(tpot / (alpha + beta))                       # 490
    assert iters == -(-3000 // c)
    # iteration k costs alpha c_k + beta min((k + 1) c, P); it grows with k, so the chunk size is not kept
    want = sum(alpha * min(c, 3000 - k * c) + beta * min((k + 1) * c, 3000) for k in range(iters))
    assert total == pytest.approx(want) and not kept
    # with beta = 0 the cost does not grow: the chunk is kept
    lines0 = [(1, alpha, 0.0, 0.0), (100001, alpha * 100001, 0.0, 0.0)]
    c, iters, total, kept = so.chunk_predict(lines0, [], [], 3000, 2048, 16384.0, tpot)
    assert c == 500 and iters == 6 and kept and total == pytest.approx(alpha * 3000)
    # decode requests take their share: alpha (n + c) + beta (KV + c) <= tpot
    kv, rem = [1000] * 20, [1000] * 20
    c, *_ = so.chunk_predict(lines, kv, rem, 3000, 2048, 16384.0, tpot)
    assert c == int((tpot - alpha * 20 - beta * 20000) / (alpha + beta) + 1e-9)
    # no chunk fits
    assert so.chunk_predict(lines, [10 ** 6], [5], 100, 2048, 16384.0, tpot) == (0, 0, 0.0, False)
    # the cap and the prompt length bound the chunk
    assert so.chunk_predict(lines0, [], [], 3000, 128, 16384.0, tpot)[0] == 128
    assert so.chunk_predict(lines0, [], [], 77, 2048, 16384.0, tpot)[:2] == (77, 1)
    # a table with a prefill term only: iteration 0 costs g phi c (c + 1) / 2, so c is the root of a quadratic;
    # later chunks work on k c prior tokens and cost more, so the size is not kept past the first
    g, phi = 1e-9, 16384.0
    lines_pf = [(1, 0.0, 0.0, g), (100001, 0.0, 0.0, g)]
    c, iters, total, kept = so.chunk_predict(lines_pf, [], [], 5000, 4096, phi, tpot)
    root = int((-1.0 + (1.0 + 8.0 * tpot / (g * phi)) ** 0.5) / 2.0)
    assert c == root and iters == -(-5000 // c) and not kept
    want = sum(g * phi * (min(c, 5000 - k * c) * k * c + 0.5 * min(c, 5000 - k * c) * (min(c, 5000 - k * c) + 1)) for k in range(iters))
    assert total == pytest.approx(want)
    assert so.prefill_work(4.0 * 128 * 32, 1536, 3885) == 4 * 128 * 32 * (1536 * 3885 + 1536 * 1537 // 2)


# ---------------------------------------------------------------------------
# overlap form: base + max(decode term, prefill term)
# ---------------------------------------------------------------------------
def overlap_rows(rng, a_d, s, a_p, q, n=400, noise=0.0):
    rows = []
    for i in range(n):
        kv = float(rng.integers(2_000, 2_000_000))
        pf = float(rng.uniform(1e9, 1.2e12))
        if i % 10 == 0:
            pf = 0.0  # decode-only batches
        if i % 10 == 1:
            kv = 0.0  # a chunk alone
        dec, pre = a_d + s * kv, a_p + q * pf
        lat = dec if pf == 0.0 else pre if kv == 0.0 else max(dec, pre)
        rows.append((int(rng.choice([72, 320, 1032])), kv, pf, lat * (1.0 + noise * rng.standard_normal())))
    return rows


def test_overlap_fit_recovers_an_exact_max_of_two_lines():
    rng = np.random.default_rng(11)
    a_d, s, a_p, q = 26.0, 6.1e-4, 34.0, 9.9e-10
    lines = so.table_build_overlap(overlap_rows(rng, a_d, s, a_p, q))
    assert [ln[0] for ln in lines] == [72, 320, 1032]
    for ln in lines:
        assert ln[1] == 0.0
        np.testing.assert_allclose(ln[2:], (a_d, s, a_p, q), rtol=1e-9)
    # with 3 % noise on the latencies the parameters come back within a few per cent, the slopes within one
    noisy = so.table_build_overlap(overlap_rows(np.random.default_rng(12), a_d, s, a_p, q, n=3000, noise=0.03))[0]
    np.testing.assert_allclose(noisy[3], s, rtol=0.02)
    np.testing.assert_allclose(noisy[5], q, rtol=0.02)


def test_overlap_fit_without_chunks_is_the_plain_regression_line():
    """No row carries prefill work: every row is on the decode side and the fit is numpy's straight line."""
    rng = np.random.default_rng(13)
    kv = rng.integers(1_000, 3_000_000, 60).astype(np.float64)
    lat = 20.0 + 6e-4 * kv + rng.normal(0.0, 3.0, 60)
    (ln,) = so.table_build_overlap([(256, x, 0.0, y) for x, y in zip(kv, lat)])
    slope, icpt = np.polyfit(kv, lat, 1)
    np.testing.assert_allclose((ln[2], ln[3]), (icpt, slope), rtol=1e-8)
    # and the other way round: chunks alone
    pf = rng.uniform(1e9, 1e12, 60)
    lat = 30.0 + 1e-9 * pf + rng.normal(0.0, 3.0, 60)
    (ln,) = so.table_build_overlap([(256, 0.0, x, y) for x, y in zip(pf, lat)])
    slope, icpt = np.polyfit(pf, lat, 1)
    np.testing.assert_allclose((ln[4], ln[5]), (icpt, slope), rtol=1e-8)


def test_overlap_lookup_by_hand():
    lines = [(64, 5.0, 10.0, 1e-3, 20.0, 1e-9), (128, 9.0, 10.0, 1e-3, 20.0, 1e-9)]
    # decode side larger: 5 + max(10 + 100, 20 + 50); prefill side larger; a batch without a chunk; a chunk alone
    assert so.table_predict(lines, 64, 100_000, 5e10) == pytest.approx(115.0, rel=1e-12)
    assert so.table_predict(lines, 64, 10_000, 5e10) == pytest.approx(75.0, rel=1e-12)
    assert so.table_predict(lines, 64, 1_000, 0.0) == pytest.approx(16.0, rel=1e-12)  # not max(11, 20)
    assert so.table_predict(lines, 64, 0, 1e9) == pytest.approx(26.0, rel=1e-12)  # not max(10, 21)
    assert so.table_predict(lines, 96, 100_000, 5e10) == pytest.approx(117.0, rel=1e-12)  # half way between the bases
    # never above the sum of the two terms, never below either; the batch term and the scaling act on it as on a sum table
    rng = np.random.default_rng(14)
    for _ in range(200):
        kv, pf = int(rng.integers(1, 10**6)), float(rng.uniform(1.0, 1e12))
        t = so.table_predict(lines, 64, kv, pf)
        dec, pre = 10.0 + 1e-3 * kv, 20.0 + 1e-9 * pf
        assert max(dec, pre) + 5.0 == pytest.approx(t, rel=1e-12) and t <= 5.0 + dec + pre
    more = so.table_scale(so.table_add_batch_term(lines, [(64, 100.0), (128, 300.0)]), 32.0)
    assert so.table_predict(more, 64, 100_000, 5e10) == pytest.approx(32.0 * 215.0, rel=1e-12)
    assert so.table_predict(more, 128, 100_000, 5e10) == pytest.approx(32.0 * 419.0, rel=1e-12)
