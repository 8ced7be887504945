"""Scheduler-side entry points (include/polyserve_sched.h) through the C ABI against oracle/sched_oracle.py.

Host code on both sides, so these run without a GPU.  Integers must agree exactly; predicted times to 1e-12
relative (both sides work in fp64 on the same formula; only the summation order of the fit may differ)."""
import os
import re

import numpy as np
import pytest

import paper_2507_17769_b200 as ps
from paper_2507_17769_b200 import binding as B
from paper_2507_17769_b200 import sched_binding as S
from oracle import sched_oracle as so

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
REL = 1e-12


def test_library_exports_every_symbol_of_the_sched_header():
    header = open(os.path.join(ROOT, "include", "polyserve_sched.h")).read()
    declared = set(re.findall(r"\b(ps_[a-z_]+)\s*\(", header)) - {"ps_profile_grid"}  # named in prose only
    assert declared == set(S.EXPORTS)
    lib = B.load()
    for name in declared:
        assert getattr(lib, name) is not None


def grid_rows(rng, batches, per_line=27):
    rows, plain = [], []
    for b in batches:
        a, s, q = float(rng.uniform(10, 400)), float(rng.uniform(5e-5, 5e-4)), float(rng.uniform(5e-10, 2e-9))
        with_chunk = b != batches[0]  # the first line is decode-only: its prefill work is 0 in every row
        for _ in range(per_line):
            kv = int(rng.integers(1000, 3_000_000))
            pf = float(rng.uniform(1e9, 5e11)) if with_chunk else 0.0
            lat = np.float32((a + s * kv + q * pf) * (1.0 + 0.03 * rng.standard_normal()))
            r = ps.ps_grid_row()
            r.token_batch, r.kv_tokens, r.prefill_flops, r.latency_us = b, kv, pf, float(lat)
            rows.append(r)
            plain.append((b, kv, pf, float(lat)))
    order = rng.permutation(len(rows))  # rows of one line need not be adjacent
    return [rows[i] for i in order], [plain[i] for i in order]


def close(a, b):
    return abs(a - b) <= REL * max(1.0, abs(a), abs(b))


def test_table_build_and_predict_match_the_oracle():
    rng = np.random.default_rng(21)
    rows, plain = grid_rows(rng, [72, 96, 192, 320, 1032, 2304])
    t = S.ps_table_build(rows)
    try:
        want = so.table_build(plain)
        b, a, s, q = S.ps_table_get_lines(t)
        assert b.tolist() == [ln[0] for ln in want]
        for i, ln in enumerate(want):
            assert abs(a[i] - ln[1]) <= 1e-9 * max(1.0, abs(ln[1])) and abs(s[i] - ln[2]) <= 1e-9 * abs(ln[2])
            assert abs(q[i] - ln[3]) <= 1e-9 * abs(ln[3]) and (q[i] != 0.0) == (i > 0)
        lines = list(zip(b.tolist(), a.tolist(), s.tolist(), q.tolist()))  # the lookup is compared on the library's own lines
        for _ in range(2000):
            tb, kv, pf = int(rng.integers(1, 4000)), int(rng.integers(0, 5_000_000)), float(rng.uniform(0, 6e11))
            assert close(S.ps_table_predict(t, tb, kv, pf), so.table_predict(lines, tb, kv, pf))
        for tb in (1, 72, 73, 95, 96, 2303, 2304, 2305, 10 ** 6):  # at, next to and beyond the lines
            assert close(S.ps_table_predict(t, tb, 12345, 1e10), so.table_predict(lines, tb, 12345, 1e10))
    finally:
        S.ps_table_free(t)
    # degenerate lines: collinear regressors, only the prefill work varying, nothing varying
    cases = [[(520, kv, 3.0e5 * kv, 20.0 + 7e-4 * kv) for kv in (1000, 2000, 5000, 9000)],
             [(520, 4000, pf, 30.0 + 1e-9 * pf) for pf in (1e9, 5e9, 2e10)],
             [(8, 500, 0.0, 10.0), (8, 500, 0.0, 14.0)]]
    for plain in cases:
        rows = []
        for b, kv, pf, lat in plain:
            r = ps.ps_grid_row()
            r.token_batch, r.kv_tokens, r.prefill_flops, r.latency_us = b, kv, pf, lat
            rows.append(r)
        t = S.ps_table_build(rows)
        try:
            got = [x.tolist()[0] for x in S.ps_table_get_lines(t)]
            want = so.table_build([(b, kv, pf, float(np.float32(lat))) for b, kv, pf, lat in plain])[0]
            assert got[0] == want[0] and all(abs(g - w) <= 1e-9 * max(1e-12, abs(w)) for g, w in zip(got[1:], want[1:]))
            assert [g == 0.0 for g in got[2:]] == [w == 0.0 for w in want[2:]]
        finally:
            S.ps_table_free(t)


def test_batch_term_and_scale_match_the_oracle():
    rng = np.random.default_rng(26)
    lines = [(72, 14.0, 2.2e-4, 0.0), (96, 16.0, 2.4e-4, 6e-10), (320, 30.0, 2.5e-4, 1.0e-9), (2304, 60.0, 2.7e-4, 1.0e-9)]
    for samples in ([(64, 30.0), (128, 50.0), (512, 150.0), (4096, 900.0)], [(300, 7.0)], [(2304, 1.0), (72, 2.0)]):
        t = S.ps_table_from_lines(*zip(*lines))
        try:
            perm = rng.permutation(len(samples))
            S.ps_table_add_batch_term(t, [samples[i][0] for i in perm], [samples[i][1] for i in perm])
            S.ps_table_scale(t, 32.0)
            want = so.table_scale(so.table_add_batch_term(lines, samples), 32.0)
            got = list(zip(*[x.tolist() for x in S.ps_table_get_lines(t)]))
            assert len(got) == len(want)
            for g, w in zip(got, want):
                assert g[0] == w[0] and all(close(a, b) for a, b in zip(g[1:], w[1:]))
            with pytest.raises(ps.PsError):
                S.ps_table_add_batch_term(t, [8, 8], [1.0, 2.0])
            with pytest.raises(ps.PsError):
                S.ps_table_scale(t, 0.0)
        finally:
            S.ps_table_free(t)


def overlap_grid_rows(rng, n, with_pure=True):
    """Sweep-like rows of an engine that overlaps the two parts: latency ~ max(decode term, prefill term), 4 % noise."""
    rows, plain = [], []
    for i in range(n):
        b = int(rng.choice([72, 96, 320, 1032, 2304]))
        kv = int(rng.integers(2_000, 3_000_000))
        pf = float(rng.uniform(1e9, 1.5e12))
        if with_pure and i % 9 == 0:
            pf = 0.0
        if with_pure and i % 9 == 1:
            kv = 0
        dec, pre = 26.0 + 6.1e-4 * kv, 34.0 + 9.9e-10 * pf
        lat = dec if pf == 0.0 else pre if kv == 0 else max(dec, pre)
        lat = float(np.float32(lat * (1.0 + 0.04 * rng.standard_normal())))
        r = ps.ps_grid_row()
        r.token_batch, r.kv_tokens, r.prefill_flops, r.latency_us = b, kv, pf, lat
        rows.append(r)
        plain.append((b, kv, pf, lat))
    return rows, plain


def test_overlap_table_matches_the_oracle():
    rng = np.random.default_rng(31)
    for n, with_pure in ((648, True), (300, False), (40, True), (3, False)):
        rows, plain = overlap_grid_rows(rng, n, with_pure)
        t = S.ps_table_build_overlap(rows)
        try:
            want = so.table_build_overlap(plain)
            b, base, s, q = S.ps_table_get_lines(t)
            a_d, a_p = S.ps_table_get_overlap(t)
            assert b.tolist() == [ln[0] for ln in want]
            for i, ln in enumerate(want):
                got = (base[i], a_d[i], s[i], a_p[i], q[i])
                assert got[0] == 0.0 and all(abs(g - w) <= 1e-9 * max(1e-12, abs(w)) for g, w in zip(got, ln[1:]))
            lines = list(zip(b.tolist(), base.tolist(), a_d.tolist(), s.tolist(), a_p.tolist(), q.tolist()))
            for _ in range(1000):
                tb, kv, pf = int(rng.integers(1, 4000)), int(rng.integers(0, 5_000_000)), float(rng.uniform(0, 2e12))
                if rng.random() < 0.1:
                    pf = 0.0
                if rng.random() < 0.1:
                    kv = 0
                assert close(S.ps_table_predict(t, tb, kv, pf), so.table_predict(lines, tb, kv, pf))
            # the batch term, the scaling and the admission test act on this form as on a sum table
            S.ps_table_add_batch_term(t, [64, 512, 4096], [30.0, 150.0, 900.0])
            S.ps_table_scale(t, 32.0)
            more = so.table_scale(so.table_add_batch_term(lines, [(64, 30.0), (512, 150.0), (4096, 900.0)]), 32.0)
            for tb, kv, pf in ((72, 100_000, 0.0), (500, 762_000, 1.2e11), (3000, 0, 4e11), (1, 5, 1.0)):
                assert close(S.ps_table_predict(t, tb, kv, pf), so.table_predict(more, tb, kv, pf))
            kv_len, rem = rng.integers(1, 9000, 64).astype(np.int32), rng.integers(1, 500, 64).astype(np.int32)
            for tpot in (2e4, 6e4, 2e5):
                got = S.ps_admit(t, kv_len, rem, 700, 300, 512, 4000, 8e10, tpot)
                ok, pred, peak = so.admit(more, kv_len.tolist(), rem.tolist(), 700, 300, 512, 4000, 8e10, tpot)
                assert bool(got[0]) == ok and close(got[1], pred) and got[2] == peak
        finally:
            S.ps_table_free(t)
    # a sweep whose chunks never matter: the prefill side stays empty and keeps the start's values, slope not below 0
    plain = [(96 + 32 * (i % 3), int(kv), float(pf), float(np.float32(30.0 + 6e-4 * kv - 2e-9 * pf + rng.normal(0, 0.5))))
             for i, (kv, pf) in enumerate(zip(rng.integers(50_000, 900_000, 60), rng.uniform(1e8, 4e9, 60)))]
    rows = []
    for b, kv, pf, lat in plain:
        r = ps.ps_grid_row()
        r.token_batch, r.kv_tokens, r.prefill_flops, r.latency_us = b, kv, pf, lat
        rows.append(r)
    t = S.ps_table_build_overlap(rows)
    want = so.table_build_overlap(plain)
    _, _, s, q = S.ps_table_get_lines(t)
    a_d, a_p = S.ps_table_get_overlap(t)
    assert q[0] == 0.0 and want[0][5] == 0.0 and s[0] > 0
    assert all(abs(g - w) <= 1e-9 * max(1e-12, abs(w)) for g, w in zip((a_d[0], s[0], a_p[0]), (want[0][2], want[0][3], want[0][4])))
    S.ps_table_free(t)
    t = S.ps_table_from_lines([5], [1.0], [0.1])
    assert S.ps_table_get_overlap(t) is None
    S.ps_table_free(t)
    r = ps.ps_grid_row()
    r.token_batch, r.kv_tokens, r.latency_us = 8, -1, 1.0
    with pytest.raises(ps.PsError):
        S.ps_table_build_overlap([r])


def test_table_rejects_bad_input():
    with pytest.raises(ps.PsError):
        S.ps_table_from_lines([10, 10], [1.0, 2.0], [0.1, 0.1])  # duplicate batch size
    with pytest.raises(ps.PsError):
        S.ps_table_from_lines([0], [1.0], [0.1])
    with pytest.raises(ps.PsError):
        S.ps_table_from_lines([5], [float("nan")], [0.1])
    r = ps.ps_grid_row()
    r.token_batch, r.kv_tokens, r.latency_us = 8, -1, 1.0
    with pytest.raises(ps.PsError):
        S.ps_table_build([r])
    t = S.ps_table_from_lines([5], [1.0], [0.1])
    with pytest.raises(ps.PsError):
        S.ps_table_predict(t, 0, 10)
    with pytest.raises(ps.PsError):
        S.ps_table_predict(t, 1, -10)
    with pytest.raises(ps.PsError):
        S.ps_table_predict(t, 1, 10, -1.0)
    S.ps_table_free(t)


def random_requests(rng, n, max_len=40000, max_rem=2000):
    return rng.integers(1, max_len, n).astype(np.int32), rng.integers(1, max_rem, n).astype(np.int32)


def test_peak_kv_matches_the_simulation():
    rng = np.random.default_rng(22)
    for n in [1, 2, 3, 7, 64, 256]:
        for _ in range(20):
            kv, rem = random_requests(rng, n, max_rem=400)
            assert S.ps_peak_kv(kv, rem) == so.peak_kv(kv.tolist(), rem.tolist())
    # ties and equal remaining lengths
    assert S.ps_peak_kv([10, 3], [4, 1]) == (13, 0)
    assert S.ps_peak_kv([5, 5, 5], [9, 9, 9]) == so.peak_kv([5, 5, 5], [9, 9, 9])
    assert S.ps_peak_kv([], []) == (0, 0)
    with pytest.raises(ps.PsError):
        S.ps_peak_kv([5, 0], [3, 3])
    with pytest.raises(ps.PsError):
        S.ps_peak_kv([5, 5], [3, 0])


def test_admission_matches_the_oracle():
    rng = np.random.default_rng(23)
    lines = [(8, 14.0, 2.2e-4, 0.0), (64, 16.0, 2.4e-4, 0.0), (256, 30.0, 2.5e-4, 1.0e-9), (512, 55.0, 2.6e-4, 1.2e-9),
             (2304, 80.0, 2.6e-4, 1.1e-9)]
    t = S.ps_table_from_lines(*zip(*lines))
    try:
        flips = 0
        for _ in range(300):
            n = int(rng.integers(0, 300))
            kv, rem = random_requests(rng, n, max_len=9000, max_rem=600)
            new_kv, new_rem, extra = int(rng.integers(1, 9000)), int(rng.integers(1, 600)), int(rng.integers(0, 3) * 512)
            extra_kv = extra + int(rng.integers(0, 8192)) if extra else 0
            extra_pf = 4.0 * 128 * 32 * (extra * (extra_kv - extra) + extra * (extra + 1) / 2)
            tpot = float(rng.uniform(20.0, 500.0))
            got = S.ps_admit(t, kv, rem, new_kv, new_rem, extra, extra_kv, extra_pf, tpot)
            want = so.admit(lines, kv.tolist(), rem.tolist(), new_kv, new_rem, extra, extra_kv, extra_pf, tpot)
            assert got[0] == want[0] and close(got[1], want[1]) and got[2] == want[2]
            flips += got[0]
        assert 20 < flips < 280  # both answers occur
    finally:
        S.ps_table_free(t)


def test_chunk_next_and_schedule_match_the_oracle_and_the_papers_example():
    assert S.ps_chunk_schedule(2050, 1024, 1024, False).tolist() == [1024, 1024, 2]
    assert S.ps_chunk_schedule(2050, 1024, 1, False).tolist() == [1, 1024, 1024, 1]
    assert S.ps_chunk_schedule(2050, 1024, 1024, True).tolist() == [1024, 1026]
    rng = np.random.default_rng(24)
    for _ in range(500):
        budget = int(rng.integers(1, 3000))
        n = int(rng.integers(0, 12))
        rem = rng.integers(1, 5 * budget + 2, n).astype(np.int32)
        used = int(rng.integers(0, budget + 3))
        for dyn in (False, True):
            assert S.ps_chunk_next(rem, budget, used, dyn).tolist() == so.chunk_next(rem.tolist(), budget, used, dyn)
        prompt, free = int(rng.integers(1, 9 * budget + 2)), int(rng.integers(0, budget + 1))
        for dyn in (False, True):
            assert S.ps_chunk_schedule(prompt, budget, free, dyn).tolist() == so.chunk_schedule(prompt, budget, free, dyn)
    with pytest.raises(ps.PsError):
        S.ps_chunk_next([5], 0, 0, True)
    with pytest.raises(ps.PsError):
        S.ps_chunk_next([0], 8, 0, True)
    with pytest.raises(ps.PsError):
        S.ps_chunk_schedule(100, 8, 9, False)
    with pytest.raises(ps.PsError):
        S.ps_chunk_schedule(100, 8, 8, False, capacity=3)  # 13 chunks do not fit


def test_chunk_prediction_matches_the_oracle():
    rng = np.random.default_rng(25)
    lines = [(8, 14.0, 2.2e-4, 0.0), (64, 16.0, 2.4e-4, 6e-10), (256, 30.0, 2.5e-4, 1.0e-9), (512, 35.0, 2.6e-4, 1.2e-9),
             (1024, 40.0, 2.6e-4, 1.1e-9), (2304, 60.0, 2.7e-4, 1.0e-9)]
    t = S.ps_table_from_lines(*zip(*lines))
    try:
        seen = set()
        for _ in range(300):
            n = int(rng.integers(0, 200))
            kv, rem = random_requests(rng, n, max_len=6000, max_rem=40)
            prompt, cap = int(rng.integers(1, 20000)), int(rng.choice([64, 512, 2048, 100000]))
            tpot = float(rng.uniform(15.0, 900.0))
            got = S.ps_chunk_predict(t, kv, rem, prompt, cap, 4.0 * 128 * 32, tpot)
            want = so.chunk_predict(lines, kv.tolist(), rem.tolist(), prompt, cap, 4.0 * 128 * 32, tpot)
            assert got[0] == want[0] and got[1] == want[1] and close(got[2], want[2]) and got[3] == want[3]
            seen.add((got[0] > 0, got[3]))
        assert seen == {(False, False), (True, False), (True, True)}
    finally:
        S.ps_table_free(t)
