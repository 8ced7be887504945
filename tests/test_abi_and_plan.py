"""CPU-side checks of the C-ABI library: it loads, exports what the header
declares, validates arguments, and the host partitioner covers every
(query row, visible key) exactly once.  No kernel is launched here."""
import os
import re

import numpy as np
import pytest

import paper_2507_17769_b200 as ps
from paper_2507_17769_b200 import binding as B
from workloads import gen

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def opts(num_sms=148, dec=0, pre=0):
    return ps.ps_plan_opts(dec, pre, num_sms)


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "polyserve_attn.h")).read()
    declared = set(re.findall(r"\b(ps_[a-z_0-9]+)\s*\(", header))
    assert declared == set(B.EXPORTS)
    lib = B.load()
    for name in declared:
        assert getattr(lib, name) is not None
    assert "sm_100a" in ps.ps_version()


def test_kv_bytes_and_shape_validation():
    s = ps.make_shape(32, 8, 128)
    assert ps.ps_kv_bytes(s, 10) == 10 * 8 * 2 * 16 * 128 * 2
    assert ps.ps_kv_bytes(ps.make_shape(4, 2, 64), 3) == 3 * 2 * 2 * 16 * 64 * 2
    for bad, code in [((32, 8, 96, 16), B.PS_ERR_UNSUPPORTED), ((32, 8, 128, 32), B.PS_ERR_UNSUPPORTED),
                      ((32, 5, 128, 16), B.PS_ERR_INVALID), ((48, 1, 128, 16), B.PS_ERR_UNSUPPORTED)]:
        with pytest.raises(ps.PsError) as e:
            ps.ps_kv_bytes(ps.make_shape(*bad), 4)
        assert e.value.status == code
    with pytest.raises(ps.PsError):
        ps.ps_kv_bytes(s, 0)


def test_plan_rejects_bad_lengths():
    s = ps.make_shape(32, 8, 128)
    for prior, q_len, max_pages in [([5], [0], 4), ([-1], [1], 4), ([100], [1], 4), ([0], [65], 4)]:
        with pytest.raises(ps.PsError) as e:
            ps.ps_attn_plan(s, prior, q_len, max_pages, opts())
        assert e.value.status == B.PS_ERR_INVALID
    with pytest.raises(ps.PsError):
        ps.ps_attn_plan(s, [5], [1], 4, opts(dec=24))  # not a multiple of the page size


def coverage_check(batch, plan):
    """Every (request, kv head, q token, key <= causal limit) is covered by exactly one item."""
    s = batch.shape
    G = s.group
    dec, pre = ps.ps_plan_get_items(plan)
    q_start = batch.q_start
    # decode: per (req, new token, kv head) the pieces tile [0, keys the token sees) in order; a decode request has
    # one new token, a chunk of a few tokens may run as that many rows
    seen = {}
    for it in dec:
        r, g, k0, k1, qt, nt, slot, fp = it.tolist()
        i = qt - q_start[r]
        assert nt == 1 and 0 <= i < batch.q_len[r] and fp == batch.prior[r] + i
        assert k0 % 16 == 0 and k0 < k1 <= batch.prior[r] + i + 1
        seen.setdefault((r, i, g), []).append((k0, k1, slot))
    as_decode = {r for r, _, _ in seen}
    for r in range(batch.n):
        if batch.q_len[r] == 1:
            assert r in as_decode
        if r not in as_decode:
            continue
        for i in range(int(batch.q_len[r])):
            for g in range(s.n_kv_heads):
                segs = sorted(seen[(r, i, g)])
                assert segs[0][0] == 0 and segs[-1][1] == batch.prior[r] + i + 1
                for a, b in zip(segs[:-1], segs[1:]):
                    assert a[1] == b[0]
                slots = [x[2] for x in segs]
                if len(segs) == 1:
                    assert slots == [-1]
                else:
                    assert all(x >= 0 for x in slots) and [x - slots[0] for x in slots] == [k * G for k in range(len(slots))]
    # prefill: per (req, kv head, tile) the segments tile [0, first_pos + n_tok)
    tiles = {}
    for it in pre:
        r, g, k0, k1, qt, nt, slot, fp = it.tolist()
        assert batch.q_len[r] > 1 and r not in as_decode and k0 % 128 == 0 and k0 < k1
        tok0 = qt - q_start[r]
        assert fp == batch.prior[r] + tok0 and 1 <= nt <= 256 // G and tok0 % (256 // G) == 0
        assert k1 <= fp + nt
        tiles.setdefault((r, g, tok0, nt), []).append((k0, k1, slot))
    for r in range(batch.n):
        c = int(batch.q_len[r])
        if r in as_decode:
            continue
        tt = 256 // G
        for g in range(s.n_kv_heads):
            covered = 0
            for tok0 in range(0, c, tt):
                nt = min(tt, c - tok0)
                segs = sorted(tiles[(r, g, tok0, nt)])
                assert segs[0][0] == 0 and segs[-1][1] == batch.prior[r] + tok0 + nt
                for a, b in zip(segs[:-1], segs[1:]):
                    assert a[1] == b[0]
                if len(segs) == 1:
                    assert segs[0][2] == -1
                else:
                    base = segs[0][2]
                    assert [x[2] - base for x in segs] == [i * nt * G for i in range(len(segs))]
                covered += nt
            assert covered == c
    # partial slots of different groups never overlap
    info = ps.ps_plan_get_info(plan)
    used = np.zeros(info.n_partial_slots, dtype=np.int32)
    for _, segs in seen.items():
        for k0, k1, slot in segs:
            if slot >= 0:
                used[slot : slot + G] += 1
    for (r, g, tok0, nt), segs in tiles.items():
        for k0, k1, slot in segs:
            if slot >= 0:
                used[slot : slot + nt * G] += 1
    assert np.all(used == 1)
    return info


@pytest.mark.parametrize("make,kw", [
    (gen.config0, {}), (gen.config0, {"dec": 16, "pre": 128}), (gen.config1, {}), (gen.config2, {}),
    (lambda: gen.config3_cell(64, 8, 8192, 3001), {}), (lambda: gen.config3_cell(2048, 256, 512, 3002), {}),
    (gen.config4, {}),
])
def test_partition_covers_every_row_and_key_once(make, kw):
    batch = make()
    sh = ps.make_shape(batch.shape.n_q_heads, batch.shape.n_kv_heads, batch.shape.head_dim)
    plan, ws = ps.ps_attn_plan(sh, batch.prior, batch.q_len, batch.max_pages, opts(**kw))
    try:
        info = coverage_check(batch, plan)
        assert info.total_q_tokens == batch.total_q
        assert ws >= 256 + info.n_partial_slots * (batch.shape.head_dim + 1) * 4
    finally:
        ps.ps_plan_free(plan)


def test_chunks_of_a_few_tokens_run_as_decode_rows():
    """Up to 8 new tokens on a context short enough to re-read: one decode row per token, no prefill item.  Longer
    chunks, long contexts and plans with forced prefill segments keep the prefill kernel."""
    shape = gen.SHAPE_8B
    b = gen.make_batch(shape, 5, [2048, 0, 100, 511, 7, 300, 60000], [2, 8, 1, 5, 9, 1, 4])
    plan, _ = ps.ps_attn_plan(ps.make_shape(32, 8, 128), b.prior, b.q_len, b.max_pages, opts(), None)
    try:
        info = coverage_check(b, plan)
        dec, pre = ps.ps_plan_get_items(plan)
        assert set(pre[:, 0].tolist()) == {4, 6}  # the 9-token chunk, and 4 tokens on 60 000 (a 1 GB re-read)
        assert set(dec[:, 0].tolist()) == {0, 1, 2, 3, 5}
        rows = {(r, qt) for r, qt in zip(dec[:, 0].tolist(), dec[:, 4].tolist())}
        assert len(rows) == 2 + 8 + 1 + 5 + 1
        assert info.n_prefill_items == len(pre) > 0
    finally:
        ps.ps_plan_free(plan)
    plan, _ = ps.ps_attn_plan(ps.make_shape(32, 8, 128), b.prior, b.q_len, b.max_pages, opts(pre=128), None)
    try:
        coverage_check(b, plan)
        dec, pre = ps.ps_plan_get_items(plan)
        assert set(dec[:, 0].tolist()) == {2, 5} and set(pre[:, 0].tolist()) == {0, 1, 3, 4, 6}
    finally:
        ps.ps_plan_free(plan)
    # a batch of tiny chunks only launches the decode kernel alone
    b = gen.make_batch(shape, 6, [2048, 10], [2, 3])
    plan, _ = ps.ps_attn_plan(ps.make_shape(32, 8, 128), b.prior, b.q_len, b.max_pages, opts(), None)
    try:
        info = coverage_check(b, plan)
        assert info.n_prefill_items == 0 and info.n_launches == 1 and info.decode_sms == info.prefill_sms == 148
    finally:
        ps.ps_plan_free(plan)


    # beside many decode rows the chunk's prefill kernel is hidden: it stays a prefill item
    b = gen.make_batch(shape, 7, [1500] + [2047] * 128, [4] + [1] * 128)
    plan, _ = ps.ps_attn_plan(ps.make_shape(32, 8, 128), b.prior, b.q_len, b.max_pages, opts(), None)
    try:
        coverage_check(b, plan)
        _, pre = ps.ps_plan_get_items(plan)
        assert set(pre[:, 0].tolist()) == {0}
    finally:
        ps.ps_plan_free(plan)


def test_partition_ignores_page_ids_and_replans_in_place():
    b = gen.config2()
    sh = ps.make_shape(32, 8, 128)
    plan, ws1 = ps.ps_attn_plan(sh, b.prior, b.q_len, b.max_pages, opts())
    d1, p1 = ps.ps_plan_get_items(plan)
    plan2, ws2 = ps.ps_attn_plan(sh, b.prior, b.q_len, b.max_pages + 7, opts())
    d2, p2 = ps.ps_plan_get_items(plan2)
    assert np.array_equal(d1, d2) and np.array_equal(p1, p2) and ws1 == ws2
    # rebuild the first handle for another batch, then back: same items again
    c = gen.config1()
    same, _ = ps.ps_attn_plan(sh, c.prior, c.q_len, c.max_pages, opts(), plan)
    assert same == plan and ps.ps_plan_get_info(plan).n_prefill_items == 0
    ps.ps_attn_plan(sh, b.prior, b.q_len, b.max_pages, opts(), plan)
    d3, p3 = ps.ps_plan_get_items(plan)
    assert np.array_equal(d1, d3) and np.array_equal(p1, p3)
    ps.ps_plan_free(plan)
    ps.ps_plan_free(plan2)


def test_decode_units_are_balanced():
    b = gen.config1()
    sh = ps.make_shape(32, 8, 128)
    plan, _ = ps.ps_attn_plan(sh, b.prior, b.q_len, b.max_pages, opts())
    info = ps.ps_plan_get_info(plan)
    total_pages = int(((b.kv_len + 15) // 16).sum()) * 8
    per_unit = info.decode_segment_tokens // 16
    assert per_unit == max(8, -(-total_pages // (148 * 12)))  # one unit per resident warp (12 warps per SM)
    # partial rows stay a small fraction of the KV stream
    assert info.n_partial_slots * 128 * 4 < 0.1 * b.decode_bytes()
    ps.ps_plan_free(plan)


def test_mixed_batches_split_the_sms_and_single_class_batches_do_not():
    sh = ps.make_shape(32, 8, 128)
    for make, mixed in [(gen.config1, False), (gen.config2, True), (lambda: gen.make_batch(gen.SHAPE_8B, 5, [700], [300]), False),
                        (lambda: gen.config3_cell(64, 8, 512, 3000), True)]:
        b = make()
        plan, _ = ps.ps_attn_plan(sh, b.prior, b.q_len, b.max_pages, opts())
        info = ps.ps_plan_get_info(plan)
        if mixed:
            assert info.decode_sms + info.prefill_sms == 148 and info.decode_sms >= 8 and info.prefill_sms >= 8
        else:
            assert info.decode_sms == 148 and info.prefill_sms == 148
        coverage_check(b, plan)
        ps.ps_plan_free(plan)
    big = gen.config4()
    plan, _ = ps.ps_attn_plan(ps.make_shape(64, 8, 128), big.prior, big.q_len, big.max_pages, opts())
    info = ps.ps_plan_get_info(plan)
    assert info.decode_sms + info.prefill_sms == 148 and info.prefill_sms > info.decode_sms  # prefill-heavy batch
    ps.ps_plan_free(plan)


def test_replanning_in_place_keeps_the_work_list_slots_where_they_are():
    """The two work-list slots of the workspace sit at a stride that only grows: a plan object rebuilt for a smaller
    batch keeps the stride of the larger one (so runs in flight find their slots), and asks for the same workspace
    again when the larger batch comes back."""
    s = ps.make_shape(32, 8, 128)
    big_prior, small_prior = [3000] * 64, [100] * 4
    plan, ws_big = ps.ps_attn_plan(s, big_prior, [1] * 64, 256, opts())
    try:
        fresh_small, ws_small_fresh = ps.ps_attn_plan(s, small_prior, [1] * 4, 256, opts())
        ps.ps_plan_free(fresh_small)
        _, ws_small = ps.ps_attn_plan(s, small_prior, [1] * 4, 256, opts(), plan)
        assert ws_small_fresh < ws_small <= ws_big
        _, ws_again = ps.ps_attn_plan(s, big_prior, [1] * 64, 256, opts(), plan)
        assert ws_again == ws_big
        info = ps.ps_plan_get_info(plan)
        assert info.n_decode_items >= 64 * 8
    finally:
        ps.ps_plan_free(plan)


def test_wait_limit_setter_validates_its_argument():
    s = ps.make_shape(32, 8, 128)
    plan, _ = ps.ps_attn_plan(s, [100], [1], 16, opts())
    try:
        ps.ps_plan_set_wait_limit(plan, 0)
        ps.ps_plan_set_wait_limit(plan, 4_000_000_000)
        for bad in (-1, 4_000_000_001):
            with pytest.raises(ps.PsError) as e:
                ps.ps_plan_set_wait_limit(plan, bad)
            assert e.value.status == B.PS_ERR_INVALID
    finally:
        ps.ps_plan_free(plan)


def test_fp8_cache_shapes_plan_decode_rows_only():
    s8 = ps.make_shape(32, 8, 128, 16, 1)
    assert ps.ps_kv_bytes(s8, 3) == 3 * 8 * (2 * 16 * 128 + 2 * 16 * 4)
    plan, ws = ps.ps_attn_plan(s8, [500, 40], [1, 1], 64, opts())
    ps.ps_plan_free(plan)
    with pytest.raises(ps.PsError) as e:
        ps.ps_attn_plan(s8, [500, 40], [1, 2], 64, opts())
    assert e.value.status == B.PS_ERR_UNSUPPORTED
    with pytest.raises(ps.PsError) as e:
        ps.ps_kv_bytes(ps.make_shape(8, 8, 64, 16, 1), 3)
    assert e.value.status == B.PS_ERR_UNSUPPORTED
