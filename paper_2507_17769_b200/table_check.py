"""Build the scheduler's latency table from a sweep and check it on held-out batches (paper section 4.5).

    python -m paper_2507_17769_b200.table_check [--seeds 27] [--iters 10] [--quick] [--heads 32,8,128]

1. ps_profile_grid over the chunk x decode count x mean context grid -> ps_table_build (per token batch size one
   least-squares fit of latency over KV tokens and prefill-attention work).
2. A second sweep over batch shapes that are not on the grid, with other seeds; each of its draws is timed and
   compared with ps_table_predict(token_batch, kv_tokens, prefill_flops), and with the same table looked up by the
   paper's two keys alone (prefill work left out of the fit), and with the overlap form ps_table_build_overlap fits
   to the same sweep (base + max(decode term, prefill term): the two kernels of a mixed batch run side by side).
   Prints the relative prediction errors.
3. The host cost of the admission test (ps_admit) and of the chunk prediction (ps_chunk_predict) for an instance
   with 256 running requests, in decisions per second through this binding.
4. With --iteration: the whole-iteration table of the paper's model T_iter = GEMM(B) + decode attention + prefill
   attention (section 3.4; the two attention terms in the overlap form) for an 8B-class decoder (32 layers, hidden 4096, 32 q / 8 kv heads of 128, FFN 14336): the
   sweep is repeated with the KV append inside the timed region, the linear layers' time at each of the table's batch
   sizes is measured with library GEMMs (torch.matmul, bf16; weights of four layers in rotation so that none is found
   in L2) and added with ps_table_add_batch_term, and everything is scaled to 32 layers with ps_table_scale.

The paper's keys (token batch size, KV-cache size) do not carry the chunk's own prior context, so a table on those
two alone predicts prefill-heavy batches poorly; the report shows both tables and splits the batches by chunk size.
"""
from __future__ import annotations

import argparse
import json
import time

import numpy as np

from . import binding as B
from . import sched_binding as S

GRID = ((64, 128, 256, 512, 1024, 2048), (8, 32, 128, 256), (512, 2048, 8192))
HELD_OUT = ((96, 384, 768, 1536), (16, 64, 192), (1024, 4096))


def rel_errors(table, rows, with_prefill_work=True):
    out = []
    for r in rows:
        pred = S.ps_table_predict(table, r.token_batch, r.kv_tokens, r.prefill_flops if with_prefill_work else 0.0)
        out.append((pred - r.latency_us) / r.latency_us)
    return np.array(out)


def two_key_table(rows):
    """The same sweep fitted on the paper's two keys alone: the rows' prefill work is hidden from the fit."""
    blind = []
    for r in rows:
        c = B.ps_grid_row()
        c.token_batch, c.kv_tokens, c.prefill_flops, c.latency_us = r.token_batch, r.kv_tokens, 0.0, r.latency_us
        blind.append(c)
    return S.ps_table_build(blind)


def summary(err):
    a = np.abs(err)
    return {"n": int(a.size), "median_abs": float(np.median(a)), "p90_abs": float(np.quantile(a, 0.9)),
            "max_abs": float(a.max()), "mean_signed": float(err.mean())}


def host_rates(table, n_running=256, calls=20000, seed=7):
    rng = np.random.default_rng(seed)
    kv = rng.integers(64, 8192, n_running).astype(np.int32)
    rem = rng.integers(1, 512, n_running).astype(np.int32)
    t0 = time.perf_counter()
    for i in range(calls):
        S.ps_admit(table, kv, rem, 1000 + i % 97, 200, 0, 0, 0.0, 400.0)
    admit_s = (time.perf_counter() - t0) / calls
    n2 = max(calls // 20, 1)
    t0 = time.perf_counter()
    for i in range(n2):
        S.ps_chunk_predict(table, kv, rem, 6000 + i % 97, 2048, 4.0 * 128 * 32, 400.0)
    chunk_s = (time.perf_counter() - t0) / n2
    return {"n_running": n_running, "admit_per_s": 1.0 / admit_s, "chunk_predict_per_s": 1.0 / chunk_s}


LAYERS, HIDDEN, KV_DIM, FFN = 32, 4096, 1024, 14336


def layer_gemm_us(batches, reps=20):
    """Time of one decoder layer's linear layers (QKV, O, gate+up, down) on B tokens, per B, with torch.matmul."""
    import torch

    dev = torch.device("cuda")
    shapes = [(HIDDEN, HIDDEN + 2 * KV_DIM), (HIDDEN, HIDDEN), (HIDDEN, 2 * FFN), (FFN, HIDDEN)]
    weights = [[torch.randn(k, n, device=dev, dtype=torch.bfloat16) * 0.02 for k, n in shapes] for _ in range(4)]
    out = []
    for b in batches:
        xs = [torch.randn(int(b), k, device=dev, dtype=torch.bfloat16) for k, _ in shapes]
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        times = []
        for it in range(reps + 5):
            w = weights[it % 4]
            ev0.record()
            for x, m in zip(xs, w):
                torch.matmul(x, m)
            ev1.record()
            torch.cuda.synchronize()
            if it >= 5:
                times.append(ev0.elapsed_time(ev1) * 1e3)
        out.append(float(np.median(times)))
    return out


def iteration_table(shape, grid, seeds, warmup, iters):
    rows = B.ps_profile_grid(shape, *grid, seeds, warmup, iters, 3000, include_kv_write=True)
    table = S.ps_table_build_overlap(rows)  # the form that predicts held-out batches best; its base takes GEMM(B)
    b, _, _, _ = S.ps_table_get_lines(table)
    gemm = layer_gemm_us(b.tolist())
    S.ps_table_add_batch_term(table, b, gemm)
    S.ps_table_scale(table, float(LAYERS))
    print("whole-iteration table (%d layers; per layer: attention with KV append + linear layers):" % LAYERS)
    for bi, g in zip(b.tolist(), gemm):
        print("  token_batch %5d: linear layers %8.1f us per layer" % (bi, g))
    phi = 4.0 * shape.head_dim * shape.n_q_heads
    for n_dec, ctx, chunk, prior in [(64, 1024, 0, 0), (256, 2048, 0, 0), (256, 8192, 0, 0), (128, 2048, 512, 2048), (256, 2048, 1792, 4096)]:
        kv = n_dec * ctx + (chunk + prior if chunk else 0)
        pf = phi * (chunk * prior + 0.5 * chunk * (chunk + 1.0))
        t = S.ps_table_predict(table, n_dec + chunk, kv, pf)
        print("  %3d decodes at %5d tokens%s: predicted iteration %.2f ms" %
              (n_dec, ctx, " + %d-token chunk on %d" % (chunk, prior) if chunk else "", t / 1e3))
    return table


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--seeds", type=int, default=27)
    ap.add_argument("--held-out-seeds", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--iters", type=int, default=10)
    ap.add_argument("--quick", action="store_true", help="corner cells of the grid, 3 seeds; two held-out shapes")
    ap.add_argument("--heads", default="32,8,128", help="n_q_heads,n_kv_heads,head_dim")
    ap.add_argument("--iteration", action="store_true", help="also build the whole-iteration table of an 8B-class model")
    a = ap.parse_args()
    hq, hkv, d = (int(x) for x in a.heads.split(","))
    shape = B.make_shape(hq, hkv, d)
    grid, held, seeds = GRID, HELD_OUT, a.seeds
    if a.quick:
        grid, held, seeds = ((64, 2048), (8, 256), (512, 8192)), ((384,), (64,), (1024, 4096)), min(3, a.seeds)
    rows = B.ps_profile_grid(shape, *grid, seeds, a.warmup, a.iters, 3000)
    table = S.ps_table_build(rows)
    try:
        b, icpt, slope, slope_pf = S.ps_table_get_lines(table)
        print("table: %d lines from %d draws" % (len(b), len(rows)))
        for i in range(len(b)):
            print("  token_batch %5d: latency_us = %9.2f + %.4e * kv_tokens + %.4e * prefill_flops" % (b[i], icpt[i], slope[i], slope_pf[i]))
        test = B.ps_profile_grid(shape, *held, a.held_out_seeds, a.warmup, a.iters, 9000)
        heavy = np.array([r.chunk >= 768 for r in test])

        def split(err):
            return {"all": summary(err), "chunk_below_768": summary(err[~heavy]) if (~heavy).any() else None,
                    "chunk_768_up": summary(err[heavy]) if heavy.any() else None}

        blind = two_key_table(rows)
        overlap = S.ps_table_build_overlap(rows)
        try:
            _, _, o_s, o_q = S.ps_table_get_lines(overlap)
            o_ad, o_ap = S.ps_table_get_overlap(overlap)
            print("overlap form: latency_us = max(%.2f + %.4e * kv_tokens, %.2f + %.4e * prefill_flops)" % (o_ad[0], o_s[0], o_ap[0], o_q[0]))
            report = {"fit_rows": summary(rel_errors(table, rows)), "held_out": split(rel_errors(table, test)),
                      "fit_rows_two_keys": summary(rel_errors(blind, rows, False)),
                      "held_out_two_keys": split(rel_errors(blind, test, False)),
                      "fit_rows_overlap": summary(rel_errors(overlap, rows)), "held_out_overlap": split(rel_errors(overlap, test)),
                      "host": host_rates(table), "host_overlap": host_rates(overlap)}
        finally:
            S.ps_table_free(blind)
            S.ps_table_free(overlap)
        print(json.dumps(report))
        if a.iteration:
            S.ps_table_free(iteration_table(shape, grid, seeds, a.warmup, a.iters))
    finally:
        S.ps_table_free(table)


if __name__ == "__main__":
    main()
