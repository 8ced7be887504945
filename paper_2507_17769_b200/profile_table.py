"""Emit the iteration-latency table the scheduler consults (paper section 4.5).

    python -m paper_2507_17769_b200.profile_table [--out table.csv] [--seeds 27] [--iters 10] [--quick]
                                                  [--peaks hbm_gbs,bf16_tflops] [--cpu-times cells.csv]

Runs ps_profile_grid over chunk size x decode count x mean context (default:
the 6 x 4 x 3 grid with 27 seeded length draws per cell) and prints, per cell,
the median latency over the draws plus the table's two keys in the paper's
terms: token batch size (chunk + decode rows) and KV-cache size (sum of
kv_len).  Also reports how well latency at a fixed decode count is explained
by an affine function of total KV tokens (the paper models decode attention
time as a function of KV-cache size, section 3.4).  ``--peaks`` sets the
denominators of the rows' roofline fraction (default: the nominal 8000 GB/s and
2250 TFLOP/s); ``--cpu-times`` takes the CSV that ``bench.py --workload 3``
writes (seconds a CPU reference needs for seed 0 of each cell) and prints that
time beside each cell.
"""
from __future__ import annotations

import argparse
import statistics

import numpy as np

from . import binding as B

CHUNKS = (64, 128, 256, 512, 1024, 2048)
DECODES = (8, 32, 128, 256)
CTXS = (512, 2048, 8192)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--out", default=None, help="CSV with one row per (cell, seed) draw")
    ap.add_argument("--seeds", type=int, default=27)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--iters", type=int, default=10)
    ap.add_argument("--quick", action="store_true", help="2 x 2 x 2 corner cells, 3 seeds")
    ap.add_argument("--heads", default="32,8,128", help="n_q_heads,n_kv_heads,head_dim")
    ap.add_argument("--peaks", default="0,0", help="hbm GB/s, bf16 TFLOP/s for roofline_frac (0 = nominal)")
    ap.add_argument("--cpu-times", default=None, help="CSV of per-cell CPU reference times (chunk,n_decode,mean_ctx,...,cpu_seconds)")
    a = ap.parse_args()
    hq, hkv, d = (int(x) for x in a.heads.split(","))
    chunks, decodes, ctxs, seeds = CHUNKS, DECODES, CTXS, a.seeds
    if a.quick:
        chunks, decodes, ctxs, seeds = (64, 2048), (8, 256), (512, 8192), min(3, a.seeds)
    hbm, tensor = (float(x) for x in a.peaks.split(","))
    rows = B.ps_profile_grid(B.make_shape(hq, hkv, d), chunks, decodes, ctxs, seeds, a.warmup, a.iters, 3000, a.out,
                             hbm_peak_gbs=hbm, bf16_peak_tflops=tensor)
    cpu = {}
    if a.cpu_times:
        import csv

        with open(a.cpu_times) as f:
            for rec in csv.DictReader(f):
                cpu[(int(rec["chunk"]), int(rec["n_decode"]), int(rec["mean_ctx"]))] = float(rec["cpu_seconds"])
    cells = {}
    for r in rows:
        cells.setdefault((r.chunk, r.n_decode, r.mean_ctx), []).append(r)
    print("chunk n_dec mean_ctx | token_batch kv_tokens(med) | latency_us med [min..max over draws] | decode TB/s  prefill TFLOP/s  "
          "roofline frac (medians of the rows' fields)" + ("  | CPU reference s (seed 0)" if cpu else ""))
    for (c, n, m), rs in cells.items():
        lat = [r.latency_us for r in rs]
        med = statistics.median(lat)
        kv = statistics.median([r.kv_tokens for r in rs])
        line = "%5d %5d %8d | %11d %14d | %9.1f [%8.1f .. %8.1f] | %6.2f %8.1f %6.3f" % (
            c, n, m, c + n, kv, med, min(lat), max(lat), statistics.median([r.decode_TBps for r in rs]),
            statistics.median([r.prefill_TFLOPs for r in rs]), statistics.median([r.roofline_frac for r in rs]))
        if cpu:
            line += "  | %9.3f" % cpu.get((c, n, m), float("nan"))
        print(line)
    # structural check: at fixed (chunk, decode count), latency ~ affine in total KV tokens
    for c in chunks:
        for n in decodes:
            pts = [(r.kv_tokens, r.latency_us) for r in rows if r.chunk == c and r.n_decode == n]
            if len(pts) >= 3:
                x = np.array([p[0] for p in pts], dtype=np.float64)
                y = np.array([p[1] for p in pts], dtype=np.float64)
                A = np.stack([x, np.ones_like(x)], axis=1)
                coef, res, _, _ = np.linalg.lstsq(A, y, rcond=None)
                ss_tot = float(((y - y.mean()) ** 2).sum())
                r2 = 1.0 - float(((A @ coef - y) ** 2).sum()) / ss_tot if ss_tot > 0 else 1.0
                print("affine fit chunk=%4d n_dec=%3d: latency_us = %.4g * kv_tokens + %.3g   R^2 = %.4f" % (c, n, coef[0], coef[1], r2))
    print("%d draws" % len(rows))


if __name__ == "__main__":
    main()
