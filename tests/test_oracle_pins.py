"""Pins for the CPU oracle: every check compares it with something that is not
the oracle itself -- brute force of different structure, closed forms,
invariants of the definition, and torch's CPU attention routine.

The definition under test (paper section 2.1): Softmax(Q K^T / sqrt(d)) V over
the K, V of all previous tokens; chunked prefill (section 2.4) and dynamic
chunking (section 4.7, the 2050-token prompt under a 1024 budget) give the
chunk shapes used below.
"""
import math

import numpy as np
import pytest

import oracle
from workloads import gen

F = gen.bf16_bits_to_f64
B = gen.f32_to_bf16_bits


def identity_batch(kv_list, page_size, poison=True, shuffle_seed=None):
    """Pool + block table for given logical K/V lists; pages in order or shuffled."""
    need = [(x.shape[0] + page_size - 1) // page_size for x in kv_list]
    total = sum(need)
    num_pages = total + 5
    ids = np.arange(num_pages)
    if shuffle_seed is not None:
        ids = np.random.default_rng(shuffle_seed).permutation(num_pages)
    bt = np.full((len(kv_list), max(need)), -1, dtype=np.int32)
    off = 0
    for r, c in enumerate(need):
        bt[r, :c] = ids[off : off + c]
        off += c
    return bt, num_pages


def run(q, ks, vs, prior, q_len, hq, hkv, d, page=16, shuffle_seed=None):
    bt, num_pages = identity_batch(ks, page, shuffle_seed=shuffle_seed)
    kp = oracle.plain_pool(ks, bt, num_pages, page)
    vp = oracle.plain_pool(vs, bt, num_pages, page)
    return oracle.attn_paged(q, kp, vp, bt, prior, q_len, hq, hkv, d, page)


def rand_bits(rng, *shape, scale=1.0):
    return B((rng.standard_normal(shape) * scale).astype(np.float32))


def brute_force(q, k, v, prior, hq, hkv):
    """Dense reference of different structure: full score matrix, explicit
    boolean mask, normalise the whole matrix, one matmul -- extended precision."""
    qf = F(q).astype(np.longdouble)  # [c, hq, d]
    kf = F(k).astype(np.longdouble)  # [L, hkv, d]
    vf = F(v).astype(np.longdouble)
    c, _, d = qf.shape
    L = kf.shape[0]
    G = hq // hkv
    out = np.zeros((c, hq, d), dtype=np.longdouble)
    lse = np.zeros((c, hq), dtype=np.longdouble)
    rows = np.arange(c)[:, None]
    cols = np.arange(L)[None, :]
    visible = cols <= (prior + rows)
    for h in range(hq):
        g = h // G
        S = (qf[:, h, :] @ kf[:, g, :].T) / np.sqrt(np.longdouble(d))
        E = np.where(visible, np.exp(S), np.longdouble(0))
        Z = E.sum(axis=1, keepdims=True)
        out[:, h, :] = (E / Z) @ vf[:, g, :]
        lse[:, h] = np.log(Z[:, 0])
    return out.astype(np.float64), lse.astype(np.float64)


@pytest.mark.parametrize("hq,hkv,d,prior,c", [(4, 2, 64, 0, 9), (4, 2, 64, 21, 13), (8, 1, 32, 5, 1), (6, 6, 16, 37, 20)])
def test_brute_force_small(hq, hkv, d, prior, c):
    rng = np.random.default_rng(hq * 1000 + prior)
    L = prior + c
    q = rand_bits(rng, c, hq, d, scale=0.7)
    k = rand_bits(rng, L, hkv, d)
    v = rand_bits(rng, L, hkv, d)
    out, lse = run(q, [k], [v], [prior], [c], hq, hkv, d, shuffle_seed=1)
    want, want_lse = brute_force(q, k, v, prior, hq, hkv)
    assert np.max(np.abs(out - want)) < 1e-12
    assert np.max(np.abs(lse - want_lse)) < 1e-12


def test_brute_force_mixed_batch_rows_and_packing():
    """Several requests in one call: packed-Q offsets and per-request block-table rows."""
    rng = np.random.default_rng(3)
    hq, hkv, d = 4, 2, 32
    prior = [16, 0, 40, 7]
    q_len = [1, 5, 1, 18]
    ks = [rand_bits(rng, p + c, hkv, d) for p, c in zip(prior, q_len)]
    vs = [rand_bits(rng, p + c, hkv, d) for p, c in zip(prior, q_len)]
    qs = [rand_bits(rng, c, hq, d) for c in q_len]
    out, lse = run(np.concatenate(qs), ks, vs, prior, q_len, hq, hkv, d, shuffle_seed=5)
    off = 0
    for r in range(4):
        want, wl = brute_force(qs[r], ks[r], vs[r], prior[r], hq, hkv)
        assert np.max(np.abs(out[off : off + q_len[r]] - want)) < 1e-12
        assert np.max(np.abs(lse[off : off + q_len[r]] - wl)) < 1e-12
        off += q_len[r]


def test_constant_v_returns_v_and_zero_k_gives_log_length():
    rng = np.random.default_rng(1)
    hq, hkv, d, prior, c = 4, 2, 64, 30, 11
    L = prior + c
    q = rand_bits(rng, c, hq, d)
    k = rand_bits(rng, L, hkv, d)
    vrow = rand_bits(rng, 1, hkv, d)
    v = np.repeat(vrow, L, axis=0)
    out, _ = run(q, [k], [v], [prior], [c], hq, hkv, d)
    want = np.repeat(F(vrow), hq // hkv, axis=1)  # [1, hq, d]
    assert np.max(np.abs(out - want)) < 1e-14
    k0 = np.zeros_like(k)
    _, lse = run(q, [k0], [v], [prior], [c], hq, hkv, d)
    want_lse = np.log(prior + np.arange(c) + 1.0)[:, None] * np.ones((1, hq))
    assert np.max(np.abs(lse - want_lse)) < 1e-14


def test_single_key_and_one_hot_key():
    rng = np.random.default_rng(2)
    hq, hkv, d = 4, 2, 64
    q = rand_bits(rng, 1, hq, d)
    k = rand_bits(rng, 1, hkv, d)
    v = rand_bits(rng, 1, hkv, d)
    out, lse = run(q, [k], [v], [0], [1], hq, hkv, d)
    assert np.array_equal(out[0], np.repeat(F(v)[0], 2, axis=0))
    s = (F(q)[0].reshape(hkv, 2, d) * F(k)[0][:, None, :]).sum(-1).reshape(hq) / 8.0
    assert np.max(np.abs(lse[0] - s)) < 1e-13
    # one key scores +64 above the rest: output is that key's value up to e^-64
    L, hot = 50, 23
    kk = np.zeros((L, hkv, d), dtype=np.float32)
    kk[hot, :, 0] = 512.0
    qq = np.zeros((1, hq, d), dtype=np.float32)
    qq[0, :, 0] = 1.0
    vv = rand_bits(rng, L, hkv, d)
    out, _ = run(B(qq), [B(kk)], [vv], [L - 1], [1], hq, hkv, d)
    assert np.max(np.abs(out[0] - np.repeat(F(vv)[hot], 2, axis=0))) < 1e-20 + 50 * 5 * math.exp(-64)


def test_zero_q_gives_prefix_mean_of_v():
    rng = np.random.default_rng(4)
    hq, hkv, d, prior, c = 4, 2, 64, 19, 23
    L = prior + c
    q = np.zeros((c, hq, d), dtype=np.uint16)
    k = rand_bits(rng, L, hkv, d)
    v = rand_bits(rng, L, hkv, d)
    out, lse = run(q, [k], [v], [prior], [c], hq, hkv, d, shuffle_seed=9)
    vf = F(v)
    for i in range(c):
        mean = vf[: prior + i + 1].mean(axis=0)  # [hkv, d]
        assert np.max(np.abs(out[i] - np.repeat(mean, 2, axis=0))) < 1e-13
        assert abs(lse[i, 0] - math.log(prior + i + 1)) < 1e-13


@pytest.mark.parametrize("splits", [[40], [1, 39], [20, 20], [1, 19, 19, 1], [1] * 40])
def test_chunk_split_equals_unchunked(splits):
    """A prompt prefilled in chunks gives the rows of the one-shot prefill
    (the paper's 2050-token example scaled down: 1+19+19+1 vs 20+20 vs 40)."""
    rng = np.random.default_rng(6)
    hq, hkv, d, p = 4, 2, 64, 40
    q = rand_bits(rng, p, hq, d)
    k = rand_bits(rng, p, hkv, d)
    v = rand_bits(rng, p, hkv, d)
    full, full_lse = run(q, [k], [v], [0], [p], hq, hkv, d)
    done = 0
    for c in splits:
        part, part_lse = run(q[done : done + c], [k[: done + c]], [v[: done + c]], [done], [c], hq, hkv, d,
                             shuffle_seed=done)
        assert np.max(np.abs(part - full[done : done + c])) < 1e-13
        assert np.max(np.abs(part_lse - full_lse[done : done + c])) < 1e-13
        done += c
    assert done == p


def test_dynamic_chunk_lengths_1024_1026_small_heads():
    """Chunks {1024, 1026} of a 2050-token prompt (section 4.7's example) against the one-shot rows."""
    rng = np.random.default_rng(7)
    hq, hkv, d, p = 2, 1, 16, 2050
    q = rand_bits(rng, p, hq, d)
    k = rand_bits(rng, p, hkv, d)
    v = rand_bits(rng, p, hkv, d)
    bt, num_pages = identity_batch([k], 16)
    kp = oracle.plain_pool([k], bt, num_pages, 16)
    vp = oracle.plain_pool([v], bt, num_pages, 16)
    rows = np.array([0, 1, 1023, 1024, 1025, 2049], dtype=np.int32)
    full, _ = oracle.attn_rows(q, kp, vp, bt, [0], [p], hq, hkv, d, 16, np.zeros(6, dtype=np.int32), rows)
    second, _ = oracle.attn_rows(q[1024:], kp, vp, bt, [1024], [1026], hq, hkv, d, 16,
                                 np.zeros(3, dtype=np.int32), np.array([0, 1, 1025], dtype=np.int32))
    assert np.max(np.abs(second - full[3:])) < 1e-13
    want, _ = brute_force(q[2049:2050], k, v, 2049, hq, hkv)
    assert np.max(np.abs(full[5] - want[0])) < 1e-12


def test_decode_row_equals_last_prefill_row():
    rng = np.random.default_rng(8)
    hq, hkv, d, p = 4, 2, 64, 100
    q = rand_bits(rng, p, hq, d)
    k = rand_bits(rng, p, hkv, d)
    v = rand_bits(rng, p, hkv, d)
    full, full_lse = run(q, [k], [v], [0], [p], hq, hkv, d)
    dec, dec_lse = run(q[-1:], [k], [v], [p - 1], [1], hq, hkv, d, shuffle_seed=2)
    assert np.max(np.abs(dec[0] - full[-1])) < 1e-13
    assert np.max(np.abs(dec_lse[0] - full_lse[-1])) < 1e-13


def test_key_order_does_not_matter_for_a_decode_row():
    rng = np.random.default_rng(10)
    hq, hkv, d, L = 4, 2, 64, 77
    q = rand_bits(rng, 1, hq, d)
    k = rand_bits(rng, L, hkv, d)
    v = rand_bits(rng, L, hkv, d)
    a, la = run(q, [k], [v], [L - 1], [1], hq, hkv, d)
    perm = rng.permutation(L)
    b, lb = run(q, [k[perm]], [v[perm]], [L - 1], [1], hq, hkv, d)
    assert np.max(np.abs(a - b)) < 1e-13 and np.max(np.abs(la - lb)) < 1e-13


def test_gqa_consecutive_q_heads_share_a_kv_head():
    rng = np.random.default_rng(11)
    hq, hkv, d, L = 8, 2, 16, 33
    q = rand_bits(rng, 1, hq, d)
    k = rand_bits(rng, L, hkv, d)
    v = np.zeros((L, hkv, d), dtype=np.float32)
    for g in range(hkv):
        v[:, g, :] = g + 1
    out, _ = run(q, [k], [B(v)], [L - 1], [1], hq, hkv, d)
    for h in range(hq):
        assert np.max(np.abs(out[0, h] - (h // 4 + 1))) < 1e-14
    # and K's head mapping: scores of head h use K of kv head h // 4
    want, wl = brute_force(q, k, B(v), L - 1, hq, hkv)
    _, lse = run(q, [k], [B(v)], [L - 1], [1], hq, hkv, d)
    assert np.max(np.abs(lse - wl)) < 1e-12


@pytest.mark.parametrize("hq,hkv", [(4, 4), (8, 2)])
def test_matches_torch_cpu_causal_sdpa_fp64(hq, hkv):
    import torch

    rng = np.random.default_rng(12)
    d, p = 64, 75
    q = rand_bits(rng, p, hq, d)
    k = rand_bits(rng, p, hkv, d)
    v = rand_bits(rng, p, hkv, d)
    out, _ = run(q, [k], [v], [0], [p], hq, hkv, d)
    tq = torch.from_numpy(F(q)).permute(1, 0, 2)[None]  # [1, hq, p, d]
    tk = torch.from_numpy(F(k)).permute(1, 0, 2)[None].repeat_interleave(hq // hkv, dim=1)
    tv = torch.from_numpy(F(v)).permute(1, 0, 2)[None].repeat_interleave(hq // hkv, dim=1)
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0].permute(1, 0, 2).numpy()
    assert np.max(np.abs(out - want)) < 1e-10


def test_page_permutation_and_poison():
    """Same logical content under two page assignments gives identical bits;
    NaN in every unreferenced page and tail slot never reaches the output."""
    b = gen.config0()
    s = b.shape
    ks, vs = zip(*[b.kv_bits(r) for r in range(b.n)])
    kp = oracle.plain_pool(ks, b.block_table, b.num_pages, s.page_size)
    vp = oracle.plain_pool(vs, b.block_table, b.num_pages, s.page_size)
    assert np.any(kp == oracle.BF16_NAN)
    out, lse = oracle.attn_paged(b.q_bits(), kp, vp, b.block_table, b.prior, b.q_len, s.n_q_heads, s.n_kv_heads,
                                 s.head_dim, s.page_size)
    assert np.all(np.isfinite(out)) and np.all(np.isfinite(lse))
    bt2, n2 = gen.assign_pages(777, b.kv_len, s.page_size, spare=0.5)
    assert not np.array_equal(bt2, b.block_table)
    kp2 = oracle.plain_pool(ks, bt2, n2, s.page_size)
    vp2 = oracle.plain_pool(vs, bt2, n2, s.page_size)
    out2, lse2 = oracle.attn_paged(b.q_bits(), kp2, vp2, bt2, b.prior, b.q_len, s.n_q_heads, s.n_kv_heads,
                                   s.head_dim, s.page_size)
    assert np.array_equal(out, out2) and np.array_equal(lse, lse2)
    # gather returns the logical tensors bit for bit
    for r in range(b.n):
        assert np.array_equal(oracle.kv_gather(kp, b.block_table[r], int(b.kv_len[r])), ks[r])
        assert np.array_equal(oracle.kv_gather(vp2, bt2[r], int(b.kv_len[r])), vs[r])
    # reading one slot past a sequence's end hits the poison
    with np.errstate(invalid="ignore"):
        kv_len_bad = b.kv_len.copy()
        prior_bad = b.prior.copy()
        prior_bad[0] += 1  # 17 -> 18 tokens: slot 1 of page 1 is poisoned
        bad, _ = oracle.attn_paged(b.q_bits(), kp, vp, b.block_table, prior_bad, b.q_len, s.n_q_heads, s.n_kv_heads,
                                   s.head_dim, s.page_size)
    assert np.all(np.isnan(bad[0]))


def test_split_and_lse_merge_equals_unsplit():
    rng = np.random.default_rng(13)
    hq, hkv, d, L = 2, 1, 32, 90
    q = rand_bits(rng, 1, hq, d)
    k = rand_bits(rng, L, hkv, d)
    v = rand_bits(rng, L, hkv, d)
    full, full_lse = run(q, [k], [v], [L - 1], [1], hq, hkv, d)
    cuts = [0, 16, 48, 49, 90]
    parts, lses = [], []
    for a, b_ in zip(cuts[:-1], cuts[1:]):
        o, l = run(q, [k[a:b_]], [v[a:b_]], [b_ - a - 1], [1], hq, hkv, d)
        parts.append(o[0])
        lses.append(l[0])
    for h in range(hq):
        o, l = oracle.lse_merge(np.stack([p[h] for p in parts]), np.array([x[h] for x in lses]))
        assert np.max(np.abs(o - full[0, h])) < 1e-13
        assert abs(l - full_lse[0, h]) < 1e-13
    # closed form: two parts with equal mass average; a part with lse = -inf is ignored
    o, l = oracle.lse_merge(np.array([[1.0, 2.0], [3.0, 6.0]]), np.array([0.5, 0.5]))
    assert np.allclose(o, [2.0, 4.0]) and abs(l - (0.5 + math.log(2))) < 1e-15
    o, l = oracle.lse_merge(np.array([[1.0, 2.0], [3.0, 6.0]]), np.array([0.5, -np.inf]))
    assert np.allclose(o, [1.0, 2.0]) and abs(l - 0.5) < 1e-15


def test_rejects_bad_arguments():
    rng = np.random.default_rng(14)
    q = rand_bits(rng, 1, 4, 64)
    k = rand_bits(rng, 4, 2, 64)
    bt = np.array([[0]], dtype=np.int32)
    kp = oracle.plain_pool([k], bt, 2, 16)
    with pytest.raises(ValueError):
        oracle.attn_paged(q, kp, kp, bt, [20], [1], 4, 2, 64, 16)  # beyond the block table
    with pytest.raises(ValueError):
        oracle.attn_paged(q, kp, kp, np.array([[7]], dtype=np.int32), [3], [1], 4, 2, 64, 16)  # page id out of range
