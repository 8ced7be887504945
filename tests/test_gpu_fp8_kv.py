"""The FP8 (E4M3) KV-cache variant of the decode path, through the C ABI: the stored cache bit for bit against the
oracle's quantiser, and decode attention against the oracle's FP8 attention (fp64 over the same dequantised values).

Tolerance.  Both sides see the same quantised K and V, so the quantisation itself cancels; what remains is the
kernel's arithmetic: fp32 scores and sums, weights times their V scale rounded to f16 (relative 2^-11 each, random
sign), bf16 output.  That is the budget of the bf16 cache's tests -- max-abs <= 1e-2 and mean-abs <= 1e-3 on outputs
that are convex mixes of N(0,1) values -- and the same bounds are used here (with the value-scaled bound of
parity_util.compare for rows of at most 8 keys and elements of 2.56 and more); lse to 2e-3."""
import numpy as np
import pytest

import oracle
from oracle import fp8 as oracle_fp8_mod
import paper_2507_17769_b200 as ps
from paper_2507_17769_b200 import binding as B
from workloads import gen

from parity_util import compare, kv_bits, q_bits

pytestmark = pytest.mark.gpu


def device_batch(batch, **kw):
    from workloads.device import DeviceBatch

    return DeviceBatch(batch, kv_dtype=1, **kw)


def oracle_fp8(batch):
    s = batch.shape
    ks, vs, qs = [], [], []
    for r in range(batch.n):
        k, v = kv_bits(batch, r)
        ks.append(k)
        vs.append(v)
        qs.append(q_bits(batch, r))
    kc, ksc = oracle.plain_pool_fp8(ks, batch.block_table, batch.num_pages, s.page_size)
    vc, vsc = oracle.plain_pool_fp8(vs, batch.block_table, batch.num_pages, s.page_size)
    rr = list(range(batch.n))
    return oracle.attn_rows_fp8(np.concatenate(qs), kc, vc, ksc, vsc, batch.block_table, batch.prior, batch.q_len, s.n_q_heads,
                                s.n_kv_heads, s.head_dim, s.page_size, rr, [0] * batch.n), (kc, vc, ksc, vsc)


def check(batch, opts=None, what=""):
    import torch

    db = device_batch(batch)
    info = db.plan(opts)
    out, lse = db.run()
    db.pa.check()
    (want, want_lse), pools = oracle_fp8(batch)
    # rows that see a handful of keys are as large as single V values: the bound scales there (see parity_util.compare)
    compare(out, lse, want, want_lse, what=what, few_key_rows=True, keys=batch.kv_len)
    out2, lse2 = db.run()
    db.pa.check()
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16)) and torch.equal(lse, lse2)
    return db, info, pools


def test_stored_cache_equals_the_reference_quantiser_bit_for_bit():
    b = gen.make_batch(gen.SHAPE_8B, 9101, [0, 16, 99, 300], [1, 1, 1, 1])
    db = device_batch(b)
    for r in range(b.n):
        L = int(b.kv_len[r])
        kc, vc, ks, vs = db.pa.gather_fp8(db.block_table[r], L)
        k, v = kv_bits(b, r)
        for bits, codes, scales in ((k, kc, ks), (v, vc, vs)):
            want_c, want_s = oracle_fp8_mod.quantise(bits)
            assert np.array_equal(codes.cpu().numpy(), want_c)
            assert np.array_equal(scales.cpu().numpy(), want_s)
    db.pa.check_pool()
    # appending token by token leaves earlier tokens' codes untouched and gives the same cache as one bulk write
    import torch
    from workloads import gen_cuda

    inc = ps.PagedAttention(32, 8, 128, b.num_pages, poison=True, kv_dtype=1)
    done = 0
    for step in (7, 1, 30, 62):
        k, v = gen_cuda.gen_kv(9101, 2, done, done + step, 8, 128)
        inc.write(k, v, db.block_table[2:3], [done], [step])
        done += step
    a = inc.gather_fp8(db.block_table[2], 100)
    w = db.pa.gather_fp8(db.block_table[2], 100)
    assert all(torch.equal(x, y) for x, y in zip(a, w))


@pytest.mark.parametrize("ctx", [[1], [2, 15, 16, 17], [31, 32, 33, 255, 256, 257], [1000, 4097]])
@pytest.mark.parametrize("shape", [gen.SHAPE_8B, gen.SHAPE_LARGE, gen.Shape(8, 8, 128), gen.Shape(16, 8, 128)])
def test_decode_rows_on_the_fp8_cache(ctx, shape):
    b = gen.make_batch(shape, 9111 + len(ctx), [c - 1 for c in ctx], [1] * len(ctx))
    check(b, what="fp8 decode %s" % ctx)


@pytest.mark.parametrize("seg", [16, 48, 512])
def test_split_kv_and_merge_on_the_fp8_cache(seg):
    b = gen.make_batch(gen.SHAPE_8B, 9121, [999, 16, 2047, 63], [1, 1, 1, 1])
    _, info, _ = check(b, ps.ps_plan_opts(seg, 0, 0), what="fp8 seg %d" % seg)
    assert info.n_merge_rows > 0


@pytest.mark.parametrize("case", range(16))
def test_random_decode_batches_on_the_fp8_cache(case):
    """Seeded batches of decode rows: group sizes 1 to 8, contexts around page and tile boundaries and long ones,
    default plans, forced segment sizes (split rows and merges) and plans for fewer SMs."""
    rng = np.random.default_rng(7300 + case)
    shape = [gen.Shape(8, 8, 128), gen.Shape(16, 8, 128), gen.SHAPE_8B, gen.SHAPE_LARGE][case % 4]
    ctx = [int(rng.choice([1, 2, 15, 16, 17, 63, 64, 65, 127, 128, 129, int(rng.integers(1, 700)), int(rng.integers(700, 6000))]))
           for _ in range(int(rng.integers(1, 24)))]
    opts = None
    if case % 3 == 1:
        opts = ps.ps_plan_opts(int(rng.choice([16, 32, 80])), 0, 0)
    elif case % 3 == 2:
        opts = ps.ps_plan_opts(0, 0, int(rng.choice([4, 33, 100])))
    b = gen.make_batch(shape, 7400 + case, [c - 1 for c in ctx], [1] * len(ctx))
    db, _, _ = check(b, opts, what="fp8 random case %d" % case)
    db.pa.close()


def test_config1_on_the_fp8_cache():
    check(gen.config1(), what="config1 on the fp8 cache")


def test_fp8_pools_refuse_what_they_do_not_serve():
    s8 = ps.make_shape(32, 8, 128, 16, 1)
    assert ps.ps_kv_bytes(s8, 10) == 10 * 8 * (2 * 16 * 128 + 128)
    with pytest.raises(ps.PsError) as e:
        ps.ps_attn_plan(s8, [100, 5], [1, 20], 16)
    assert e.value.status == B.PS_ERR_UNSUPPORTED
    with pytest.raises(ps.PsError) as e:
        ps.ps_kv_bytes(ps.make_shape(4, 2, 64, 16, 1), 4)
    assert e.value.status == B.PS_ERR_UNSUPPORTED
