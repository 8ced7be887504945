"""The N > 1 path on CPU: two gloo ranks draw their own batches of the same
law (weak scaling, no data-path collective) and combine their measurements as
bench.py does: time = max over ranks, units = sum over ranks."""
import os
import socket
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import torch.distributed as dist

    import bench
    import paper_2507_17769_b200 as ps
    from workloads import gen

    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.dist_env() == (rank, rank, world)
    batch = gen.config1(1001 + 100 * rank)
    # each rank plans its own shard; no rank needs another rank's lengths
    plan, _ = ps.ps_attn_plan(ps.make_shape(32, 8, 128), batch.prior, batch.q_len, batch.max_pages, ps.ps_plan_opts(0, 0, 148))
    info = ps.ps_plan_get_info(plan)
    ps.ps_plan_free(plan)
    local_ms = 1.0 + rank  # stand-in for the device time
    ms, units = bench.reduce_over_ranks(local_ms, float(batch.decode_bytes()), world)
    # the other way to split the job: one batch, cut by KV head -- same lengths on every rank, half the heads each
    full = gen.config1(1001)
    part = bench.shard_batch(gen.config1, 1001, rank, world, "heads")
    assert (part.shape.n_q_heads, part.shape.n_kv_heads) == (16, 4) and (part.prior == full.prior).all()
    assert (part.block_table == full.block_table).all()
    _, head_units = bench.reduce_over_ranks(local_ms, float(part.decode_bytes()), world)
    assert head_units == float(full.decode_bytes())  # the shards' bytes add up to the whole batch's
    out.put((rank, ms, units, float(batch.decode_bytes()), info.n_decode_items))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_by_request_and_reduce():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, ms0, u0, b0, n0), (r1, ms1, u1, b1, n1) = res
    assert ms0 == ms1 == 2.0  # max over ranks
    assert u0 == u1 == b0 + b1  # whole-job units
    assert b0 != b1 and n0 > 0 and n1 > 0  # different batches of the same law
