"""Randomised mixed batches against the oracle: shapes, row mix, lengths, planner segment sizes and SM counts drawn
from a seeded generator, pools poisoned with NaN.  Tolerance: that of the other parity tests (max-abs <= 1e-2,
mean-abs <= 1e-3 on bf16 outputs, lse to 2e-3), widened in proportion to the value only where a bf16 output cannot do
better (rows that see at most 8 keys, and elements of 2.56 and more; see parity_util.compare); every case also
runs twice and must repeat bit for bit."""
import os

import numpy as np
import pytest

import paper_2507_17769_b200 as ps
from workloads import gen
from workloads.device import DeviceBatch

from parity_util import compare, oracle_subset

pytestmark = pytest.mark.gpu

SHAPES = [gen.Shape(4, 2, 64, 16), gen.Shape(8, 8, 64, 16), gen.Shape(8, 1, 128, 16), gen.Shape(16, 2, 128, 16),
          gen.Shape(32, 8, 128, 16), gen.Shape(64, 8, 128, 16)]


def draw_batch(rng, case):
    shape = SHAPES[case % len(SHAPES)]
    n_dec = int(rng.integers(0, 12))
    n_chunk = int(rng.integers(0, 3)) if n_dec else int(rng.integers(1, 3))
    prior, q_len = [], []
    for _ in range(n_dec):
        # contexts around page and tile boundaries as well as long ones
        L = int(rng.choice([1, 2, 15, 16, 17, 127, 128, 129, int(rng.integers(1, 600)), int(rng.integers(600, 5000))]))
        prior.append(L - 1)
        q_len.append(1)
    for _ in range(n_chunk):
        c = int(rng.choice([2, 3, 31, 32, 33, 64, 127, 128, 129, 257, int(rng.integers(2, 700))]))
        pr = int(rng.choice([0, 1, 15, 16, 127, 128, 129, int(rng.integers(0, 1500))]))
        prior.append(pr)
        q_len.append(c)
    order = rng.permutation(len(prior))  # decode rows and chunks in any order
    return gen.make_batch(shape, 4000 + case, [prior[i] for i in order], [q_len[i] for i in order])


@pytest.mark.parametrize("case", range(int(os.environ.get("PS_FUZZ_CASES", "40"))))  # more cases: PS_FUZZ_CASES=300
def test_random_mixed_batch(case):
    import torch

    rng = np.random.default_rng(900 + case)
    batch = draw_batch(rng, case)
    opts = None
    if case % 3 == 1:  # forced segment sizes: many split rows and cut items
        opts = ps.ps_plan_opts(int(rng.choice([16, 32, 64])), int(rng.choice([128, 256])), 0)
    elif case % 3 == 2:  # plan for fewer SMs than the device has
        opts = ps.ps_plan_opts(0, 0, int(rng.choice([8, 40, 100])))
    db = DeviceBatch(batch, poison=True)
    db.plan(opts)
    out, lse = db.run()
    db.pa.check()
    want, want_lse, _, keys = oracle_subset(batch, range(batch.n), with_keys=True)
    compare(out, lse, want, want_lse, what="fuzz case %d" % case, few_key_rows=True, keys=keys)
    out2, lse2 = db.run()
    db.pa.check()
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16)) and torch.equal(lse, lse2)
    db.pa.close()
