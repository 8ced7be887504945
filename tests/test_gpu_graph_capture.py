"""ps_attn_run inside a CUDA stream capture: the graph replays the plan bit for bit, and calls outside the capture
keep working afterwards."""
import pytest

import paper_2507_17769_b200 as ps
from workloads import gen

from parity_util import compare, oracle_subset

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("which", ["decode rows", "mixed batch", "cut prefill items"])
def test_captured_run_replays_the_plan(which):
    import torch
    from workloads.device import DeviceBatch

    if which == "decode rows":
        b, opts = gen.make_batch(gen.SHAPE_8B, 3, [511, 2047, 15, 999], [1, 1, 1, 1]), None
    elif which == "mixed batch":
        b, opts = gen.config0(), None
    else:
        b, opts = gen.make_batch(gen.SHAPE_8B, 4, [700, 100], [40, 200]), ps.ps_plan_opts(0, 128, 0)
    db = DeviceBatch(b)
    db.plan(opts)
    eager, eager_lse = db.run()
    db.pa.check()
    want, want_lse, _ = oracle_subset(b, range(b.n))
    compare(eager, eager_lse, want, want_lse, what=which)

    out, lse = torch.zeros_like(eager), torch.zeros_like(eager_lse)
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        db.pa.run(db.q, db.block_table, out=out, lse=lse)
    for _ in range(3):
        out.zero_()
        lse.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(out, eager) and torch.equal(lse, eager_lse)
    db.pa.check()
    # calls outside the capture are not disturbed by it, whichever image slot they land on
    for _ in range(4):
        again, again_lse = db.run()
        db.pa.check()
        assert torch.equal(again, eager) and torch.equal(again_lse, eager_lse)
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, eager)
