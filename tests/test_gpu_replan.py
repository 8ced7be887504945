"""A serving loop re-plans every iteration with new lengths (paper section 2.4: each iteration batches the
running decode requests with a fresh prefill chunk).  These tests drive that loop through the C ABI with no host
synchronisation between one plan / run pair and the next, on one workspace, with batches whose work lists differ
in size and row mix, and check every iteration's output: against the CPU oracle on sampled rows, and bit for bit
against the same batch's earlier iterations."""
import numpy as np
import pytest

import paper_2507_17769_b200 as ps
from paper_2507_17769_b200 import binding as B
from workloads import gen

from parity_util import compare, oracle_subset

pytestmark = pytest.mark.gpu


def universe():
    """One pool holding the sequences of three batches: decode-only (A), mixed (B), tiny (C)."""
    rng = np.random.default_rng(5)
    a_ctx = rng.integers(300, 3000, size=48).tolist()
    b_ctx = rng.integers(100, 1500, size=24).tolist()
    prior = [c - 1 for c in a_ctx] + [c - 1 for c in b_ctx] + [1000, 40] + [20, 700, 5]
    q_len = [1] * 48 + [1] * 24 + [300, 37] + [1, 1, 2]
    u = gen.make_batch(gen.SHAPE_8B, 8101, prior, q_len)
    subsets = {"A": list(range(0, 48)), "B": list(range(48, 74)), "C": list(range(74, 77))}
    return u, subsets


def sub_inputs(u, db, idx):
    import torch

    q_start = u.q_start
    tok = np.concatenate([np.arange(q_start[r], q_start[r] + u.q_len[r]) for r in idx])
    q = db.q.index_select(0, torch.from_numpy(tok).to(db.q.device)).contiguous()
    bt = db.block_table.index_select(0, torch.tensor(idx, device=db.q.device)).contiguous()
    return q, bt, u.prior[idx], u.q_len[idx], tok


def test_replanning_between_unsynchronised_runs_on_one_workspace():
    import torch
    from workloads.device import DeviceBatch

    u, subsets = universe()
    db = DeviceBatch(u)
    pa = db.pa
    inputs = {k: sub_inputs(u, db, idx) for k, idx in subsets.items()}
    order = "ABC" * 67  # 201 iterations; neighbours always differ in work-list size and row mix
    outs = []
    torch.cuda.synchronize()
    for k in order:  # no host synchronisation inside this loop
        q, bt, prior, q_len, _ = inputs[k]
        pa.plan(prior, q_len, u.max_pages)
        out = torch.empty_like(q)
        lse = torch.empty((q.shape[0], u.shape.n_q_heads), dtype=torch.float32, device=q.device)
        pa.run(q, bt, out=out, lse=lse)
        outs.append((k, out, lse))
    pa.check()
    first = {}
    for i, (k, out, lse) in enumerate(outs):
        if k not in first:
            first[k] = (out, lse)
            continue
        assert torch.equal(out.view(torch.int16), first[k][0].view(torch.int16)), "iteration %d (batch %s) differs" % (i, k)
        assert torch.equal(lse, first[k][1]), "iteration %d (batch %s): lse differs" % (i, k)
    # the oracle on sampled rows of each batch kind: every decode row of a few requests, first / last / some
    # middle rows of the chunks
    for k, idx in subsets.items():
        reqs = idx if k == "C" else idx[:3] + idx[-2:]
        rows = {r: sorted(set(list(range(min(4, u.q_len[r]))) + list(range(max(0, u.q_len[r] - 4), u.q_len[r])) +
                              list(range(0, u.q_len[r], 61)))) for r in reqs}
        want, want_lse, packed_u = oracle_subset(u, reqs, rows)
        tok = inputs[k][4]
        pos = {int(t): j for j, t in enumerate(tok)}
        packed = np.asarray([pos[int(t)] for t in packed_u])
        compare(first[k][0], first[k][1], want, want_lse, packed, what="batch %s" % k)
    pa.close()


def test_two_plans_taking_turns_on_one_workspace():
    """Two plan objects share one workspace and one stream; neither may overwrite the other's work list or
    partial rows while that run is still in flight."""
    import torch
    from workloads.device import DeviceBatch

    u, subsets = universe()
    db = DeviceBatch(u)
    stream = torch.cuda.current_stream().cuda_stream
    plans, need = {}, 0
    for k in "AB":
        q, bt, prior, q_len, _ = sub_inputs(u, db, subsets[k])
        plan, ws = ps.ps_attn_plan(db.pa.shape, prior, q_len, u.max_pages)
        plans[k] = (plan, q, bt)
        need = max(need, ws)
    ws = torch.empty(need + 256, dtype=torch.uint8, device="cuda")
    ws_ptr = (ws.data_ptr() + 255) // 256 * 256
    try:
        ref = {}
        for k, (plan, q, bt) in plans.items():
            out = torch.empty_like(q)
            B.ps_attn_run(plan, db.pa.kv, q, bt, out, None, ws_ptr, need, stream)
            B.ps_plan_status(plan, stream)
            ref[k] = out
        outs = []
        for k in "AABABBA" * 12:  # no host synchronisation inside this loop
            plan, q, bt = plans[k]
            out = torch.empty_like(q)
            B.ps_attn_run(plan, db.pa.kv, q, bt, out, None, ws_ptr, need, stream)
            outs.append((k, out))
        torch.cuda.synchronize()
        for i, (k, out) in enumerate(outs):
            assert torch.equal(out.view(torch.int16), ref[k].view(torch.int16)), "run %d (plan %s)" % (i, k)
    finally:
        for plan, _, _ in plans.values():
            ps.ps_plan_free(plan)


@pytest.mark.parametrize("kind", ["decode", "prefill"])
def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable(kind):
    """With the wait limit at zero the first wait of an otherwise normal run gives up before its copy has landed:
    the run reports PS_ERR_TIMEOUT, nothing is left waiting, and the same plan runs correctly afterwards."""
    import torch
    from workloads.device import DeviceBatch

    if kind == "decode":
        b = gen.make_batch(gen.SHAPE_8B, 8201, [1999, 2500, 1200, 900, 3000, 1700, 2100, 800], [1] * 8)
    else:
        b = gen.make_batch(gen.SHAPE_8B, 8202, [700], [200])
    db = DeviceBatch(b)
    info = db.plan()
    assert (info.n_prefill_items == 0) == (kind == "decode")
    ps.ps_plan_set_wait_limit(db.pa._plan, 0)
    db.run()
    with pytest.raises(ps.PsError) as e:
        db.pa.check()
    assert e.value.status == B.PS_ERR_TIMEOUT
    with pytest.raises(ps.PsError) as e:
        ps.ps_plan_set_wait_limit(db.pa._plan, -1)
    assert e.value.status == B.PS_ERR_INVALID
    ps.ps_plan_set_wait_limit(db.pa._plan, 2_000_000_000)
    out, lse = db.run()
    db.pa.check()
    want, want_lse, _ = oracle_subset(b, range(b.n))
    compare(out, lse, want, want_lse, what="after a timed-out run (%s)" % kind)
    out2, lse2 = db.run()
    db.pa.check()
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16)) and torch.equal(lse, lse2)
