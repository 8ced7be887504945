"""Fixtures under tests/golden/: the paper's worked example of chunk schedules (section 4.7) and the oracle's stored
output for the tiny mixed batch (written by tests/golden/make_config0_oracle.py, which calls only oracle/)."""
import os

import numpy as np

import oracle
from workloads import gen

HERE = os.path.dirname(os.path.abspath(__file__))


def read_example():
    out = {}
    for line in open(os.path.join(HERE, "golden", "dynamic_chunking_example.txt")):
        line = line.strip()
        if line and not line.startswith("#"):
            name, *vals = line.split()
            out[name] = [int(v) for v in vals]
    return out


def test_paper_chunk_schedules_give_the_one_shot_rows():
    ex = read_example()
    budget, prompt = ex["budget"][0], ex["prompt"][0]
    assert budget == 1024 and prompt == 2050
    for name in ("one_shot", "static", "static_worst", "dynamic"):
        assert sum(ex[name]) == prompt
    # the rule of section 4.7: finish at once when fewer than two budgets remain
    assert ex["dynamic"] == [budget, prompt - budget] and prompt - budget < 2 * budget
    assert len(ex["static"]) == 3 and len(ex["static_worst"]) == 4 and len(ex["dynamic"]) == 2
    # attention rows are the same whichever schedule produced them (checked on sampled rows, small heads)
    hq, hkv, d = 2, 1, 16
    rng = np.random.default_rng(20)
    bits = lambda *s: gen.f32_to_bf16_bits(rng.standard_normal(s).astype(np.float32))
    q, k, v = bits(prompt, hq, d), bits(prompt, hkv, d), bits(prompt, hkv, d)
    pages = (prompt + 15) // 16
    bt = np.arange(pages, dtype=np.int32)[None]
    kp = oracle.plain_pool([k], bt, pages + 1, 16)
    vp = oracle.plain_pool([v], bt, pages + 1, 16)
    sample = sorted({0, 1, 1022, 1023, 1024, 1025, 2047, 2048, 2049})
    want, want_lse = oracle.attn_rows(q, kp, vp, bt, [0], [prompt], hq, hkv, d, 16, [0] * len(sample), sample)
    for name in ("static", "static_worst", "dynamic"):
        done = 0
        for c in ex[name]:
            rows = [s - done for s in sample if done <= s < done + c]
            if rows:
                got, got_lse = oracle.attn_rows(q[done : done + c], kp, vp, bt, [done], [c], hq, hkv, d, 16, [0] * len(rows), rows)
                idx = [sample.index(done + r) for r in rows]
                assert np.max(np.abs(got - want[idx])) < 1e-13 and np.max(np.abs(got_lse - want_lse[idx])) < 1e-13
            done += c


def test_oracle_output_for_config0_has_not_drifted():
    path = os.path.join(HERE, "golden", "config0_oracle.txt")
    stored = np.loadtxt(path, comments="#")
    b = gen.config0()
    s = b.shape
    ks, vs = zip(*[b.kv_bits(r) for r in range(b.n)])
    kp = oracle.plain_pool(ks, b.block_table, b.num_pages, s.page_size)
    vp = oracle.plain_pool(vs, b.block_table, b.num_pages, s.page_size)
    out, lse = oracle.attn_paged(b.q_bits(), kp, vp, b.block_table, b.prior, b.q_len, s.n_q_heads, s.n_kv_heads,
                                 s.head_dim, s.page_size)
    # stored: per (token, head): lse, then the first four and the last output element
    got = np.concatenate([lse.reshape(-1, 1), out.reshape(-1, s.head_dim)[:, [0, 1, 2, 3, -1]]], axis=1)
    assert stored.shape == got.shape
    assert np.max(np.abs(stored - got)) < 1e-12
