"""Sizes at the edges of what a serving iteration can ask for, against the oracle on sampled rows: thousands of
short decode rows, one very long context, a chunk far above any token budget, and a batch of nothing but chunks."""
import numpy as np
import pytest

from workloads import gen
from workloads.device import DeviceBatch

from parity_util import compare, oracle_subset

pytestmark = pytest.mark.gpu


def sampled(batch, reqs, rows, what):
    import torch

    db = DeviceBatch(batch, poison=True)
    info = db.plan()
    out, lse = db.run()
    db.pa.check()
    assert bool(torch.isfinite(out.float()).all()) and bool(torch.isfinite(lse).all())
    want, want_lse, packed = oracle_subset(batch, reqs, rows)
    compare(out, lse, want, want_lse, packed, what=what)
    out2, lse2 = db.run()
    db.pa.check()
    assert torch.equal(out, out2) and torch.equal(lse, lse2)
    db.pa.close()
    return info


def test_four_thousand_short_decode_rows():
    rng = np.random.default_rng(1)
    ctx = rng.integers(1, 200, 4096)
    b = gen.make_batch(gen.SHAPE_8B, 501, ctx - 1, np.ones(4096, dtype=np.int32))
    pick = [0, 1, 4095, int(np.argmax(ctx)), int(np.argmin(ctx))] + rng.integers(0, 4096, 40).tolist()
    sampled(b, sorted(set(pick)), None, "4096 decode rows")


def test_one_very_long_context():
    b = gen.make_batch(gen.SHAPE_8B, 502, [200_000 - 1, 50], [1, 1])
    info = sampled(b, [0, 1], None, "200 k context")
    assert info.n_merge_rows >= 32  # the long row is cut over many warps and combined


def test_chunk_far_above_the_budget_and_chunks_only():
    b = gen.make_batch(gen.SHAPE_8B, 503, [100], [8192])
    rows = sorted(set(list(range(4)) + [4095, 4096, 8190, 8191] + list(range(0, 8192, 1024))))
    sampled(b, [0], {0: rows}, "8192-token chunk")
    b = gen.make_batch(gen.SHAPE_LARGE, 504, [0, 700, 3000, 16], [300, 129, 64, 2])
    sampled(b, [0, 1, 2, 3], {0: [0, 1, 150, 299], 1: [0, 64, 128], 2: [0, 63], 3: [0, 1]}, "chunks only")
