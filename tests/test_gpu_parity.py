"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle
on the same seeded inputs.  Tolerance (bf16 in, fp32 accumulate, bf16 out):
max-abs <= 1e-2, mean-abs <= 1e-3; page gather and page-permutation
invariance are bit-exact."""
import numpy as np
import pytest

import oracle
import paper_2507_17769_b200 as ps
from paper_2507_17769_b200 import binding as B
from workloads import gen

from parity_util import compare, oracle_in_groups, oracle_subset

pytestmark = pytest.mark.gpu


def device_batch(batch, **kw):
    from workloads.device import DeviceBatch

    return DeviceBatch(batch, **kw)


def bits(t):
    import torch

    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def test_generator_twin_is_bit_identical():
    from workloads import gen_cuda

    k, v = gen_cuda.gen_kv(5, 3, 7, 300, 2, 64)
    hk, hv = gen.gen_kv(5, 3, 7, 300, 2, 64)
    assert np.array_equal(bits(k), hk) and np.array_equal(bits(v), hv)
    q = gen_cuda.gen_q(5, 3, 100, 140, 32, 128)
    assert np.array_equal(bits(q), gen.gen_q(5, 3, 100, 140, 32, 128))


def test_kv_write_then_gather_is_bit_exact():
    b = gen.config0()
    db = device_batch(b)
    ks, vs = zip(*[b.kv_bits(r) for r in range(b.n)])
    kp = oracle.plain_pool(ks, b.block_table, b.num_pages, 16)
    for r in range(b.n):
        k, v = db.pa.gather(db.block_table[r], int(b.kv_len[r]))
        assert np.array_equal(bits(k), ks[r]) and np.array_equal(bits(v), vs[r])
        assert np.array_equal(bits(k), oracle.kv_gather(kp, b.block_table[r], int(b.kv_len[r])))
    db.pa.check_pool()
    # appending tokens one iteration at a time gives the same pool content as one bulk write
    import torch
    from workloads import gen_cuda

    b2 = gen.make_batch(gen.SHAPE_8B, 77, [0, 0], [45, 130])
    one = device_batch(b2)
    inc = ps.PagedAttention(32, 8, 128, b2.num_pages, poison=True)
    bt = torch.from_numpy(b2.block_table).cuda()
    done = [0, 0]
    for step in ([20, 100], [24, 29], [1, 1]):
        kn, vn = [], []
        for r in range(2):
            k, v = gen_cuda.gen_kv(77, r, done[r], done[r] + step[r], 8, 128)
            kn.append(k)
            vn.append(v)
        inc.write(torch.cat(kn), torch.cat(vn), bt, done, step)
        done = [done[r] + step[r] for r in range(2)]
    for r in range(2):
        a = inc.gather(bt[r], int(b2.kv_len[r]))
        w = one.pa.gather(one.block_table[r], int(b2.kv_len[r]))
        assert torch.equal(a[0], w[0]) and torch.equal(a[1], w[1])


def full_parity(batch, opts=None, what=""):
    db = device_batch(batch)
    info = db.plan(opts)
    out, lse = db.run()
    db.pa.check()
    want, want_lse, _ = oracle_subset(batch, range(batch.n))
    return compare(out, lse, want, want_lse, what=what), info, db, out, lse


def test_config0_tiny_mixed_batch():
    (mx, mean), info, _, _, _ = full_parity(gen.config0(), what="config0")
    assert info.n_decode_items >= 8 and info.n_prefill_items >= 2


@pytest.mark.parametrize("ctx", [[1], [2, 15, 16, 17], [31, 32, 33, 255, 256, 257], [1000, 4097]])
@pytest.mark.parametrize("shape", [gen.SHAPE_TINY, gen.SHAPE_8B, gen.Shape(8, 8, 64), gen.Shape(16, 2, 128)])
def test_decode_rows(ctx, shape):
    b = gen.make_batch(shape, 11 + len(ctx), [c - 1 for c in ctx], [1] * len(ctx))
    full_parity(b, what="decode %s" % ctx)


@pytest.mark.parametrize("seg", [16, 48, 512])
def test_decode_split_kv_and_merge(seg):
    b = gen.make_batch(gen.SHAPE_8B, 21, [999, 16, 2047, 63], [1, 1, 1, 1])
    (mx, mean), info, _, _, _ = full_parity(b, ps.ps_plan_opts(seg, 0, 0), what="decode seg %d" % seg)
    assert info.n_merge_rows > 0


@pytest.mark.parametrize("prior,c", [(0, 2), (0, 33), (5, 31), (127, 128), (128, 129), (1000, 300), (48, 32), (0, 1026)])
@pytest.mark.parametrize("shape", [gen.SHAPE_TINY, gen.SHAPE_8B, gen.Shape(8, 8, 64), gen.SHAPE_LARGE])
def test_prefill_chunks(prior, c, shape):
    if shape.n_q_heads * c * (prior + c) > 2e8:
        pytest.skip("oracle would take too long")
    b = gen.make_batch(shape, 31 + c, [prior], [c])
    full_parity(b, what="prefill prior=%d c=%d" % (prior, c))


@pytest.mark.parametrize("shape", [gen.SHAPE_8B, gen.Shape(8, 8, 64), gen.SHAPE_LARGE])
def test_chunks_of_a_few_tokens_on_either_kernel(shape):
    """Chunks of 2 to 8 tokens run as decode rows by default and on the prefill kernel when segments are forced;
    both match the oracle."""
    b = gen.make_batch(shape, 45, [0, 5, 127, 1000, 300, 1200, 64], [2, 3, 8, 2, 1, 5, 9])
    (_, _), info, db, out_a, _ = full_parity(b, what="tiny chunks as decode rows")
    _, pre = ps.ps_plan_get_items(db.pa._plan)
    assert set(pre[:, 0].tolist()) == {6}  # only the 9-token chunk
    (_, _), info, db, out_b, _ = full_parity(b, ps.ps_plan_opts(0, 128, 0), what="tiny chunks on the prefill kernel")
    _, pre = ps.ps_plan_get_items(db.pa._plan)
    assert set(pre[:, 0].tolist()) == {0, 1, 2, 3, 5, 6}
    assert (out_a.float() - out_b.float()).abs().max().item() <= 1e-2


@pytest.mark.parametrize("seg", [128, 256])
def test_prefill_split_kv_and_merge(seg):
    b = gen.make_batch(gen.SHAPE_8B, 41, [700, 100], [40, 200])
    (mx, mean), info, _, _, _ = full_parity(b, ps.ps_plan_opts(0, seg, 0), what="prefill seg %d" % seg)
    assert info.n_merge_rows > 0


def test_chunked_prefill_matches_one_shot_on_gpu():
    """Rows of a prompt prefilled as chunks {1, 19, 45, 64, 1} equal the one-shot prefill's within tolerance."""
    import torch

    shape = gen.SHAPE_8B
    p = 130
    one = gen.make_batch(shape, 51, [0], [p])
    (_, _), _, _, full_out, _ = full_parity(one, what="one-shot")
    done = 0
    for c in [1, 19, 45, 64, 1]:
        part = gen.make_batch(shape, 51, [done], [c])
        db = device_batch(part)
        db.plan()
        out, _ = db.run()
        db.pa.check()
        diff = (out.float() - full_out[done : done + c].float()).abs().max().item()
        assert diff <= 1e-2
        done += c


def test_config1_decode_only_full_parity():
    (mx, mean), info, _, _, _ = full_parity(gen.config1(), what="config1")
    assert info.n_prefill_items == 0


def sampled_parity(batch, dec_reqs, chunk_rows, what):
    """Every output finite; the rows of ``dec_reqs`` (decode requests) and ``chunk_rows`` (request -> new-token
    indices) against the oracle, which computes them one by one."""
    db = device_batch(batch)
    db.plan()
    out, lse = db.run()
    db.pa.check()
    import torch

    assert bool(torch.isfinite(out.float()).all())
    rows = {r: toks for r, toks in chunk_rows.items()}
    want, want_lse, packed = oracle_in_groups(batch, list(dec_reqs) + list(chunk_rows.keys()), rows)
    return compare(out, lse, want, want_lse, packed, what=what), db


def chunk_sample(c, edge=8, every=64):
    return sorted(set(list(range(min(edge, c))) + list(range(max(0, c - edge), c)) + list(range(0, c, every))))


def test_config2_mixed_batch_full_parity():
    """Every row of config 2 -- all 512 decode rows and all 1536 rows of the chunk -- against the oracle."""
    import torch

    b = gen.config2()
    db = device_batch(b)
    info = db.plan()
    out, lse = db.run()
    db.pa.check()
    want, want_lse, packed = oracle_in_groups(b, range(b.n))
    assert np.array_equal(packed, np.arange(b.total_q))
    compare(out, lse, want, want_lse, packed, what="config2, all %d rows" % b.total_q)
    # the two kernels of this batch run side by side on disjoint SMs; the result is still the same bits every run
    assert 0 < info.decode_sms < info.decode_sms + info.prefill_sms and info.decode_sms != info.prefill_sms
    o2, l2 = db.run()
    db.pa.check()
    assert torch.equal(out, o2) and torch.equal(lse, l2)


def test_config3_every_cell_sampled_parity():
    """All 72 cells of the latency-table grid at seed index 0: every output finite, and against the oracle all
    heads of four decode sequences (first, last, longest, shortest) plus the first / last 8 and every 64th row
    of the chunk."""
    for cell, chunk, nd, m in gen.grid_cells():
        b = gen.config3_cell(chunk, nd, m, gen.grid_seed(cell, 0))
        dec = sorted({0, nd - 1, int(np.argmax(b.kv_len[:nd])), int(np.argmin(b.kv_len[:nd]))})
        sampled_parity(b, dec, {nd: chunk_sample(chunk)}, "config3 cell %d (%d/%d/%d)" % (cell, chunk, nd, m))


def test_config4_large_long_context_dense_parity():
    """Config 4: every one of the 256 decode rows, and of both 2048-token chunks the first and last 16 rows plus
    every 16th row, against the oracle; every other output finite."""
    b = gen.config4()
    rows = chunk_sample(2048, edge=16, every=16)
    sampled_parity(b, range(256), {256: rows, 257: rows}, "config4")


def test_page_permutation_gives_identical_bits_and_runs_repeat():
    import torch

    b = gen.config0()
    db = device_batch(b)
    db.plan()
    out1, lse1 = db.run()
    out1b, lse1b = db.run()
    db.pa.check()
    assert torch.equal(out1, out1b) and torch.equal(lse1, lse1b)
    bt2, n2 = gen.assign_pages(4242, b.kv_len, 16, spare=0.6)
    b2 = gen.Batch(b.shape, b.seed, b.prior, b.q_len, bt2, n2)
    db2 = device_batch(b2)
    db2.plan()
    out2, lse2 = db2.run()
    db2.pa.check()
    assert torch.equal(out1, out2) and torch.equal(lse1, lse2)
    # a larger mixed batch with forced splits, same property
    m = gen.make_batch(gen.SHAPE_8B, 61, [700, 99, 2000, 10], [1, 150, 1, 1])
    o = ps.ps_plan_opts(64, 256, 0)
    a = device_batch(m)
    a.plan(o)
    oa, la = a.run()
    bt3, n3 = gen.assign_pages(99, m.kv_len, 16, spare=1.0)
    c = device_batch(gen.Batch(m.shape, m.seed, m.prior, m.q_len, bt3, n3))
    c.plan(o)
    oc, lc = c.run()
    assert torch.equal(oa, oc) and torch.equal(la, lc)


def test_device_side_errors_are_reported_not_fatal():
    import torch

    b = gen.config0()
    db = device_batch(b)
    db.plan()
    with pytest.raises(ps.PsError) as e:
        B.ps_attn_run(db.pa._plan, db.pa.kv, db.q, db.block_table, torch.empty_like(db.q), None, db.pa._ws, 128)
    assert e.value.status == B.PS_ERR_WORKSPACE
    bad = db.block_table.clone()
    bad[0, 0] = b.num_pages + 5  # outside the pool: the page is skipped and the run is flagged
    db.pa.run(db.q, bad)
    with pytest.raises(ps.PsError) as e:
        db.pa.check()
    assert e.value.status == B.PS_ERR_BOUNDS
    out, _ = db.run()  # the context is still usable
    db.pa.check()
    want, want_lse, _ = oracle_subset(b, range(b.n))
    compare(out, None, want, want_lse, what="after error")
