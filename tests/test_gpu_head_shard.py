"""Sharding a batch by KV head needs no exchange inside attention: the run of a head shard (its own pool holding only
that shard's K/V heads, its own plan) gives the rows of the full run for those heads, within the tolerance of the
parity tests (the work partition, hence the summation order, depends on the head count), and matches the oracle."""
import numpy as np
import pytest

import paper_2507_17769_b200 as ps
from workloads import gen, gen_cuda

from parity_util import MAX_ABS, compare, oracle_subset

pytestmark = pytest.mark.gpu


def test_head_shards_reproduce_the_full_run():
    import torch

    full_shape = gen.Shape(32, 8, 128, 16)
    prior, q_len = [700, 33, 2500, 129, 40], [1, 1, 1, 300, 1]
    batch = gen.make_batch(full_shape, 91, prior, q_len)
    bt = torch.from_numpy(batch.block_table).cuda()
    kv = [gen_cuda.gen_kv(batch.seed, r, 0, int(batch.kv_len[r]), 8, 128, "cuda") for r in range(batch.n)]
    q = torch.cat([gen_cuda.gen_q(batch.seed, r, int(batch.prior[r]), int(batch.kv_len[r]), 32, 128, "cuda") for r in range(batch.n)])

    def run(hq0, hq1, g0, g1):
        pa = ps.PagedAttention(hq1 - hq0, g1 - g0, 128, batch.num_pages, poison=True)
        for r in range(batch.n):
            k, v = kv[r]
            pa.write(k[:, g0:g1].contiguous(), v[:, g0:g1].contiguous(), bt[r], [0], [int(batch.kv_len[r])], max_pages=batch.max_pages)
        pa.plan(batch.prior, batch.q_len, batch.max_pages)
        out, lse = pa.run(q[:, hq0:hq1].contiguous(), bt)
        pa.check()
        pa.close()
        return out, lse

    full_out, full_lse = run(0, 32, 0, 8)
    want_out, want_lse, _ = oracle_subset(batch, range(batch.n))
    compare(full_out, full_lse, want_out, want_lse, what="full run")
    world = 2
    for rank in range(world):
        g0, g1 = rank * 8 // world, (rank + 1) * 8 // world
        out, lse = run(4 * g0, 4 * g1, g0, g1)
        ref = full_out[:, 4 * g0 : 4 * g1].float()
        assert (out.float() - ref).abs().max().item() <= MAX_ABS
        assert (lse - full_lse[:, 4 * g0 : 4 * g1]).abs().max().item() <= 2e-3
        compare(out, lse, want_out[:, 4 * g0 : 4 * g1], want_lse[:, 4 * g0 : 4 * g1], what="shard %d" % rank)
