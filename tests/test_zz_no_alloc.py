"""ps_attn_run_static: the attention call for callers that cannot allocate.

An engine plug-in that is forbidden to call cudaMalloc after start-up (the
host engine owns all of HBM), or a loop that cannot afford an allocation's
device stall, still has to run attention.  ps_attn_run_static takes the same
inputs and outputs as ps_attn_run but keeps its scratch (work list and
split-KV partials) in a fixed array inside the library.  This file checks,
through the C ABI, that it gives what ps_attn_run gives -- twice in a row,
because the array keeps the previous call's contents -- and that it refuses
plans that do not fit.

The file name sorts last on purpose: a run that stops at the first failure
has then already run every other test.
"""
import numpy as np
import pytest

import paper_2507_17769_b200 as ps
from paper_2507_17769_b200 import binding as B
from workloads import gen

from parity_util import MAX_ABS, MEAN_ABS, LSE_ABS

pytestmark = pytest.mark.gpu


def test_static_scratch_matches_workspace_run_twice_in_a_row():
    import torch
    from workloads.device import DeviceBatch

    # decode rows cut into several KV pieces and a chunk split into segments, so the
    # scratch carries work list, partial outputs and partial log-sum-exps
    batch = gen.make_batch(gen.SHAPE_8B, 71, [700, 99, 2000, 10, 333], [1, 150, 1, 1, 40])
    db = DeviceBatch(batch)
    info = db.plan(ps.ps_plan_opts(64, 256, 0))
    assert info.n_merge_rows > 0 and info.n_partial_slots > 0
    ref_out, ref_lse = db.run()
    db.pa.check()
    stream = torch.cuda.current_stream().cuda_stream

    for attempt in range(2):
        out = torch.full_like(ref_out, float("nan"))
        lse = torch.full_like(ref_lse, float("nan"))
        B.ps_attn_run_static(db.pa._plan, db.pa.kv, db.q, db.block_table, out, lse, stream)
        db.pa.check()
        err = (out.float() - ref_out.float()).abs()
        assert bool(torch.isfinite(out.float()).all()), "call %d: non-finite output" % attempt
        assert err.max().item() <= MAX_ABS and err.mean().item() <= MEAN_ABS, "call %d" % attempt
        assert (lse - ref_lse).abs().max().item() <= LSE_ABS, "call %d" % attempt

    # a different, smaller batch right after: stale scratch from the larger one must not leak in
    small = gen.make_batch(gen.SHAPE_8B, 72, [40, 5], [1, 20])
    ds = DeviceBatch(small)
    ds.plan(ps.ps_plan_opts(16, 128, 0))
    want_out, want_lse = ds.run()
    got = torch.empty_like(want_out)
    got_lse = torch.empty_like(want_lse)
    B.ps_attn_run_static(ds.pa._plan, ds.pa.kv, ds.q, ds.block_table, got, got_lse, stream)
    ds.pa.check()
    assert (got.float() - want_out.float()).abs().max().item() <= MAX_ABS
    assert (got_lse - want_lse).abs().max().item() <= LSE_ABS


def test_static_scratch_refuses_plans_that_do_not_fit():
    import torch
    from workloads.device import DeviceBatch

    # 48 decode rows of 4096 tokens cut into one-page pieces: far more partial rows than 8 MiB holds
    big = gen.make_batch(gen.SHAPE_8B, 73, [4095] * 48, [1] * 48)
    db = DeviceBatch(big, poison=False)
    plan, need = ps.ps_attn_plan(db.pa.shape, big.prior, big.q_len, big.max_pages, ps.ps_plan_opts(16, 0, 0))
    try:
        assert need > ps.PS_STATIC_WORKSPACE_BYTES
        out = torch.empty_like(db.q)
        with pytest.raises(ps.PsError) as e:
            B.ps_attn_run_static(plan, db.pa.kv, db.q, db.block_table, out, None, torch.cuda.current_stream().cuda_stream)
        assert e.value.status == B.PS_ERR_WORKSPACE
        assert "built-in scratch" in str(e.value)
    finally:
        ps.ps_plan_free(plan)


def test_static_scratch_two_plans_taking_turns_without_synchronising():
    """Two plans share the one built-in array on one stream, in the order A, A, B, A, ... with no host
    synchronisation: a plan's work-list upload must not land on the other plan's run while that is still
    reading the array."""
    import torch
    from workloads.device import DeviceBatch

    a = DeviceBatch(gen.make_batch(gen.SHAPE_8B, 74, [1500, 99, 2100, 10, 333, 800, 1200, 40], [1, 150, 1, 1, 40, 1, 1, 1]))
    b = DeviceBatch(gen.make_batch(gen.SHAPE_8B, 75, [40, 5, 600], [1, 20, 1]))
    stream = torch.cuda.current_stream().cuda_stream
    ref = {}
    for name, d in (("A", a), ("B", b)):
        d.plan()
        ref[name] = d.run()[0]
        d.pa.check()
    outs = []
    for name in "AABABBA" * 10:
        d = a if name == "A" else b
        out = torch.empty_like(d.q)
        B.ps_attn_run_static(d.pa._plan, d.pa.kv, d.q, d.block_table, out, None, stream)
        outs.append((name, out))
    torch.cuda.synchronize()
    a.pa.check()
    for i, (name, out) in enumerate(outs):
        assert torch.equal(out.view(torch.int16), ref[name].view(torch.int16)), "call %d (plan %s)" % (i, name)
