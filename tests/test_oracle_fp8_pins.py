"""Pins of the oracle's FP8 (E4M3) KV-cache path: the quantiser against the format's definition and a brute-force
nearest-value search, and the FP8 attention against the (separately pinned) bf16 attention on data E4M3 holds exactly."""
import numpy as np

import oracle
from oracle import fp8
from workloads import gen


def test_every_code_has_the_value_the_format_defines():
    t = fp8.decode_table()
    # spot values of the OCP FP8 E4M3 definition: bias 7, three mantissa bits, subnormals, no infinities
    assert t[0x00] == 0.0 and t[0x01] == 2.0 ** -9 and t[0x07] == 7 * 2.0 ** -9 and t[0x08] == 2.0 ** -6
    assert t[0x38] == 1.0 and t[0x3C] == 1.5 and t[0x40] == 2.0 and t[0x7E] == 448.0 and np.isnan(t[0x7F])
    assert t[0xB8] == -1.0 and t[0xFE] == -448.0 and np.isnan(t[0xFF])
    fin = ~np.isnan(t)
    assert np.all(np.diff(t[:0x7F]) > 0)  # positive codes are ordered
    # every finite code encodes back to itself (-0 keeps its sign bit)
    assert np.array_equal(fp8.encode(t[fin].astype(np.float32)), np.arange(256, dtype=np.uint8)[fin])


def test_encoder_is_round_to_nearest_even_with_saturation():
    t = fp8.decode_table()
    pos_codes = np.arange(0x7F)
    pos = t[pos_codes]
    rng = np.random.default_rng(3)
    y = np.concatenate([rng.normal(0, s, 4000) for s in (300.0, 20.0, 1.0, 0.05, 0.004)]).astype(np.float32)
    # exact midpoints between neighbouring values: ties go to the even code
    mid = ((pos[:-1] + pos[1:]) / 2).astype(np.float32)
    assert np.array_equal(mid.astype(np.float64), (pos[:-1] + pos[1:]) / 2)  # representable in fp32
    y = np.concatenate([y, mid, -mid, np.float32([448, 449, 464, 1e30, -1e30, 0.0, 2.0 ** -10, 2.0 ** -11])])
    got = fp8.encode(y)
    for v, c in zip(y.tolist(), got.tolist()):
        a = min(abs(v), 448.0)
        dist = np.abs(pos - a)
        best = np.nonzero(dist == dist.min())[0]
        want = int(best[0]) if len(best) == 1 else int([b for b in best if b % 2 == 0][0])
        assert (c & 0x7F) == want and bool(c & 0x80) == bool(np.signbit(np.float32(v))), (v, c, want)


def test_scale_is_amax_over_448_and_error_is_within_half_a_step():
    rng = np.random.default_rng(4)
    x = rng.normal(0, 1, (50, 3, 128)).astype(np.float32)
    bits = gen.f32_to_bf16_bits(x)
    xb = gen.bf16_bits_to_f64(bits)
    codes, scale = fp8.quantise(bits)
    amax = np.abs(xb).max(axis=-1)
    # the scale is amax / 448 rounded up to 8 significant bits: representable in bf16, at most 2^-7 above
    raw = amax.astype(np.float32) / np.float32(448.0)
    assert np.all(scale >= raw) and np.all(scale <= raw * (1 + 2.0 ** -7))
    assert np.array_equal(gen.bf16_bits_to_f64(gen.f32_to_bf16_bits(scale)), scale.astype(np.float64))
    assert np.all(np.abs(xb) / scale[..., None].astype(np.float64) <= 448.0)
    deq = fp8.dequantise(codes, scale)
    # E4M3 keeps 4 significant bits: relative error <= 2^-4 for normal values, absolute <= 2^-10 scale below
    err = np.abs(deq - xb)
    assert np.all(err <= np.maximum(np.abs(xb) * 2.0 ** -4, scale[..., None] * 2.0 ** -10) * (1 + 1e-6))
    z, s = fp8.quantise(np.zeros((2, 1, 8), dtype=np.uint16))
    assert np.all(z == 0) and np.all(s == 1.0)


def test_fp8_attention_equals_bf16_attention_on_data_e4m3_holds_exactly():
    """K and V drawn from E4M3's own value set (times 448 / amax = 1 by construction): quantisation is lossless, so
    the FP8 oracle must reproduce the bf16 oracle, which is pinned on its own."""
    rng = np.random.default_rng(5)
    t = fp8.decode_table()
    vals = t[np.arange(0x30, 0x50)]  # 0.5 .. 3.75
    Hq, Hkv, d, page = 4, 2, 64, 16
    prior, q_len = np.int32([20, 0, 37]), np.int32([1, 9, 3])
    ks, vs = [], []
    for L in (prior + q_len).tolist():
        k = rng.choice(vals, size=(L, Hkv, d)) * rng.choice([-1.0, 1.0], size=(L, Hkv, d))
        v = rng.choice(vals, size=(L, Hkv, d)) * rng.choice([-1.0, 1.0], size=(L, Hkv, d))
        k[:, :, 0] = 448.0  # amax = 448 exactly, so every scale is 1
        v[:, :, 0] = -448.0
        ks.append(gen.f32_to_bf16_bits(k.astype(np.float32)))
        vs.append(gen.f32_to_bf16_bits(v.astype(np.float32)))
    q = gen.f32_to_bf16_bits((rng.normal(0, 0.02, (int(q_len.sum()), Hq, d))).astype(np.float32))
    need = [(x.shape[0] + page - 1) // page for x in ks]
    bt = np.full((3, max(need)), -1, dtype=np.int32)
    perm = rng.permutation(sum(need) + 3)
    off = 0
    for r, c in enumerate(need):
        bt[r, :c] = perm[off : off + c]
        off += c
    n_pages = sum(need) + 3
    kp, vp = oracle.plain_pool(ks, bt, n_pages, page), oracle.plain_pool(vs, bt, n_pages, page)
    kc, ksc = oracle.plain_pool_fp8(ks, bt, n_pages, page)
    vc, vsc = oracle.plain_pool_fp8(vs, bt, n_pages, page)
    assert np.all(ksc[~np.isnan(ksc)] == 1.0)
    rows = [(r, i) for r in range(3) for i in range(int(q_len[r]))]
    rr, rt = [a for a, _ in rows], [b for _, b in rows]
    want, want_lse = oracle.attn_rows(q, kp, vp, bt, prior, q_len, Hq, Hkv, d, page, rr, rt)
    got, got_lse = oracle.attn_rows_fp8(q, kc, vc, ksc, vsc, bt, prior, q_len, Hq, Hkv, d, page, rr, rt)
    assert np.max(np.abs(got - want)) <= 1e-12 * 448 and np.max(np.abs(got_lse - want_lse)) <= 1e-12


def test_fp8_attention_on_random_data_is_the_bf16_attention_of_the_dequantised_cache():
    """On ordinary data the FP8 oracle equals a dense numpy evaluation of softmax(Q K'^T / sqrt(d)) V' with K', V'
    the dequantised tensors -- a different code path from the C loop."""
    rng = np.random.default_rng(6)
    Hq, Hkv, d, page = 4, 2, 64, 16
    L = 45
    kb = gen.f32_to_bf16_bits(rng.normal(0, 1, (L, Hkv, d)).astype(np.float32))
    vb = gen.f32_to_bf16_bits(rng.normal(0, 1, (L, Hkv, d)).astype(np.float32))
    qb = gen.f32_to_bf16_bits(rng.normal(0, 1, (1, Hq, d)).astype(np.float32))
    bt = np.int32([[2, 0, 1]])
    kc, ksc = oracle.plain_pool_fp8([kb], bt, 3, page)
    vc, vsc = oracle.plain_pool_fp8([vb], bt, 3, page)
    got, got_lse = oracle.attn_rows_fp8(qb, kc, vc, ksc, vsc, bt, np.int32([L - 1]), np.int32([1]), Hq, Hkv, d, page, [0], [0])
    kq = fp8.dequantise(*fp8.quantise(kb))
    vq = fp8.dequantise(*fp8.quantise(vb))
    qf = gen.bf16_bits_to_f64(qb)[0]
    for h in range(Hq):
        g = h // (Hq // Hkv)
        s = kq[:, g, :] @ qf[h] / np.sqrt(d)
        w = np.exp(s - s.max())
        assert np.allclose(got[0, h], (w / w.sum()) @ vq[:, g, :], rtol=0, atol=1e-12)
        assert abs(got_lse[0, h] - (s.max() + np.log(w.sum()))) <= 1e-12
