"""Pins for the seeded input generator (integer hash, bf16 rounding, length laws)."""
import math

import numpy as np

from workloads import gen


def test_splitmix64_published_vectors():
    # First outputs of SplitMix64 for seeds 0 and 1234567 (reference implementation
    # by S. Vigna, public domain; values widely used as test vectors).
    assert int(gen.mix64(np.uint64(0))) == 0xE220A8397B1DCDAF
    assert int(gen.mix64(np.uint64(1234567))) == 6457827717110365317
    r = gen.raw_bits(0, 0, 3)
    assert [int(x) for x in r] == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]


def test_bf16_rounding_is_nearest_even():
    import torch

    x = np.random.default_rng(0).standard_normal(100000).astype(np.float32)
    x = np.concatenate([x, np.float32([1.00390625, 1.01171875, 0.0, -0.0, 3.0e38])])
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(gen.f32_to_bf16_bits(x), want)
    back = gen.bf16_bits_to_f64(want)
    assert np.array_equal(back, torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy())


def test_normal_table_moments_and_symmetry():
    t = gen.bf16_bits_to_f64(gen.normal_table())
    assert abs(t.mean()) < 1e-6
    assert abs(t.std() - 1.0) < 5e-3
    assert np.array_equal(t, -t[::-1])
    assert np.all(np.diff(t) >= 0)
    assert 4.0 < t.max() < 4.5


def test_streams_are_piecewise_reproducible_and_distinct():
    k1, v1 = gen.gen_kv(7, 3, 0, 40, 2, 64)
    k2, v2 = gen.gen_kv(7, 3, 16, 40, 2, 64)
    assert np.array_equal(k1[16:], k2) and np.array_equal(v1[16:], v2)
    assert not np.array_equal(k1, v1)
    k3, _ = gen.gen_kv(7, 4, 0, 40, 2, 64)
    assert not np.array_equal(k1, k3)
    q1 = gen.gen_q(7, 3, 10, 20, 4, 64)
    q2 = gen.gen_q(7, 3, 0, 20, 4, 64)
    assert np.array_equal(q1, q2[10:])
    x = gen.bf16_bits_to_f64(gen.normal_bf16(gen.stream_key(1, 2, 3), 0, 200000))
    assert abs(x.mean()) < 0.01 and abs(x.std() - 1.0) < 0.01


def test_uniform_int_bounds_and_spread():
    x = gen.uniform_int(gen.stream_key(5, gen.STREAM_LEN), 0, 50000, 512, 4096)
    assert x.min() == 512 and x.max() == 4096
    assert abs(x.mean() - 2304) < 20


def test_permutation_is_a_permutation():
    p = gen.permutation(gen.stream_key(9, gen.STREAM_PERM), 1000)
    assert sorted(p.tolist()) == list(range(1000))
    assert not np.array_equal(p, np.arange(1000))


def test_config_shapes():
    b0 = gen.config0()
    assert b0.kv_len.tolist() == [17, 33, 64, 100, 80]
    assert b0.total_q == 36 and b0.num_pages >= 2 + 3 + 4 + 7 + 5 + 8
    used = b0.block_table[b0.block_table >= 0]
    assert len(set(used.tolist())) == len(used) == 21
    b1 = gen.config1()
    assert b1.n == 64 and b1.kv_len.min() >= 512 and b1.kv_len.max() <= 4096
    assert np.all(b1.q_len == 1)
    b2 = gen.config2()
    assert b2.n == 513 and b2.total_q == 2048
    ctx = b2.kv_len[:512]
    assert ctx.min() >= 16 and ctx.max() <= 16384
    assert 800 < np.median(ctx) < 1300
    assert 0 <= b2.prior[512] <= 8192 and b2.q_len[512] == 1536
    b4 = gen.config4()
    assert b4.n == 258 and b4.kv_len[:256].min() >= 4096 and b4.kv_len[:256].max() <= 32768
    assert np.all((b4.prior[256:] >= 16384) & (b4.prior[256:] <= 30000))
    gib = b4.num_pages * 16 * b4.shape.kv_token_bytes / 2**30
    assert 14 < gib < 26
    cells = gen.grid_cells()
    assert len(cells) == 72
    c = gen.config3_cell(64, 8, 512, gen.grid_seed(0, 0))
    assert c.n == 9 and c.kv_len[:8].min() >= 256 and c.kv_len[:8].max() <= 768


def test_algorithmic_work_counters():
    b = gen.make_batch(gen.SHAPE_8B, 1, [9, 100], [1, 4])
    assert b.decode_bytes() == 10 * 4096
    assert b.prefill_flops() == 4 * 128 * 32 * (4 * 100 + 10)
