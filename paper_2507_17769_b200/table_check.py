"""Build the scheduler's latency table from a sweep and check it on held-out batches (paper section 4.5).

    python -m paper_2507_17769_b200.table_check [--seeds 27] [--iters 10] [--quick] [--heads 32,8,128]

1. ps_profile_grid over the chunk x decode count x mean context grid -> ps_table_build (per token batch size one
   least-squares fit of latency over KV tokens and prefill-attention work).
2. A second sweep over batch shapes that are not on the grid, with other seeds; each of its draws is timed and
   compared with ps_table_predict(token_batch, kv_tokens, prefill_flops), and with the same table looked up by the
   paper's two keys alone (prefill work left out of the fit).  Prints the relative prediction errors.
3. The host cost of the admission test (ps_admit) and of the chunk prediction (ps_chunk_predict) for an instance
   with 256 running requests, in decisions per second through this binding.

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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--seeds", type=int, default=27)
    ap.add_argument("--held-out-seeds", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--iters", type=int, default=10)
    ap.add_argument("--quick", action="store_true", help="corner cells of the grid, 3 seeds; two held-out shapes")
    ap.add_argument("--heads", default="32,8,128", help="n_q_heads,n_kv_heads,head_dim")
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
        try:
            report = {"fit_rows": summary(rel_errors(table, rows)), "held_out": split(rel_errors(table, test)),
                      "fit_rows_two_keys": summary(rel_errors(blind, rows, False)),
                      "held_out_two_keys": split(rel_errors(blind, test, False)), "host": host_rates(table)}
        finally:
            S.ps_table_free(blind)
        print(json.dumps(report))
    finally:
        S.ps_table_free(table)


if __name__ == "__main__":
    main()
