"""Host-side logic of bench.py that needs no GPU: the bounded sample the CPU baseline is timed on, the extrapolation
from the sample's two rates to a whole step, the per-kernel roofline record, the peaks file and its fallback, and the
reference arm's line (the oracle timed on this machine's cores on the smallest perf workload)."""
import json
import os
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from workloads import gen  # noqa: E402


def test_sample_is_bounded_and_covers_every_chunk():
    b = gen.config4()
    dec, rows = bench.oracle_sample(b, dec_flops=4e10, pf_flops=8e10)
    s = b.shape
    phi = 4.0 * s.head_dim * s.n_q_heads
    # decode requests: a prefix of the batch's decode rows, within the budget
    dec_rows = [r for r in range(b.n) if b.q_len[r] == 1]
    assert dec == dec_rows[: len(dec)] and 1 <= len(dec) < len(dec_rows)
    assert sum(phi * (b.prior[r] + 1.0) for r in dec) <= 4e10
    nxt = dec_rows[len(dec)]
    assert sum(phi * (b.prior[r] + 1.0) for r in dec) + phi * (b.prior[nxt] + 1.0) > 4e10
    # chunk rows: every chunk is sampled, first and last row included, evenly spaced, within its share of the budget
    chunks = [r for r in range(b.n) if b.q_len[r] > 1]
    assert sorted(rows) == chunks and len(chunks) == 2
    for r in chunks:
        sel = rows[r]
        assert sel[0] == 0 and sel[-1] == b.q_len[r] - 1 and len(set(sel)) == len(sel)
        gaps = np.diff(sel)
        assert gaps.max() - gaps.min() <= 1
        work = sum(phi * (b.prior[r] + i + 1.0) for i in sel)
        assert work <= 1.05 * 8e10 / len(chunks)
    txt = bench.sample_text(b, dec, rows)
    assert "%d of 256 decode requests" % len(dec) in txt and "of 4096 chunk rows" in txt and "2 chunks" in txt


def test_sample_of_a_decode_only_batch_has_no_chunk_part():
    b = gen.config1()
    dec, rows = bench.oracle_sample(b)
    assert rows == {} and len(dec) >= 1
    assert "chunk" not in bench.sample_text(b, dec, rows).split(";")[0]


def test_whole_step_extrapolation_and_baseline_record():
    b = gen.config2()

    class Sample:  # the two attributes the record reads, and the method under test
        batch, dec, rows = b, [0, 1], {b.n - 1: [0, 5]}
        whole_step = bench.OracleSample.whole_step

    # a sample that ran at 2 GB/s on decode rows and 4 GFLOP/s on chunk rows
    timing = (0.5, 1.0e9, 0.25, 1.0e9, 7)
    rec = bench.cpu_baseline_record(b, Sample(), timing)
    full = b.decode_bytes() / 2.0e9 + b.prefill_flops() / 4.0e9
    assert abs(rec["whole_step_seconds_extrapolated"] - full) <= 1e-9 * full
    assert abs(rec["value"] - b.decode_bytes() / full / 1e12) <= 1e-12
    assert rec["cores"] == 7 and rec["kind"] == "oracle" and rec["unit"] == "TB/s"
    assert abs(rec["decode_TBps"] - 2.0e-3) < 1e-12 and abs(rec["prefill_TFLOPs"] - 4.0e-3) < 1e-12
    assert abs(rec["sample_seconds"] - 0.75) < 1e-12


def test_kernel_records_divide_algorithmic_units_by_the_launch_time():
    peaks = {"hbm_gbs": 6000.0, "bf16_tflops": 1600.0, "bf16_tflops_sustained": 1400.0}
    d = bench.kernel_record("decode_kernel", "alone", 0.5, 1.5e9, peaks, step_ms=0.6)
    assert d["bound"] == "hbm" and d["unit"] == "GB/s" and abs(d["achieved"] - 3000.0) < 1e-9 and abs(d["frac"] - 0.5) < 1e-12
    assert d["step_ms"] == 0.6 and d["algorithmic_bytes_per_launch"] == 1.5e9
    p = bench.kernel_record("prefill_kernel", "alone", 2.0, 1.6e12, peaks)
    assert p["bound"] == "tensor" and p["unit"] == "TFLOP/s" and abs(p["achieved"] - 800.0) < 1e-9
    assert abs(p["frac"] - 0.5) < 1e-12 and abs(p["frac_of_sustained"] - 800.0 / 1400.0) < 1e-12 and "step_ms" not in p
    assert bench.kernel_record("decode_kernel", "x", 0.0, 1.0, peaks)["achieved"] == 0.0
    # traffic: the committed capture's ratio times the launch's algorithmic bytes; no capture, no figure
    assert bench.ncu_traffic("decode_kernel", 2.0e9) == bench.NCU_TRAFFIC_RATIO["decode_kernel"] * 2.0e9
    assert bench.ncu_traffic("prefill_kernel", 2.0e9) is None


def test_peaks_come_from_the_file_or_the_stated_fallback(tmp_path, monkeypatch):
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    fb = bench.measured_peaks()
    assert fb["source"] == "fallback" and fb["hbm_gbs"] == 6650.0 and fb["bf16_tflops"] == 1590.0
    (tmp_path / "MEASURED_PEAKS.json").write_text(json.dumps({"hbm_gbs": 6500, "bf16_tflops": 1600}))
    got = bench.measured_peaks()
    assert got == {"hbm_gbs": 6500.0, "bf16_tflops": 1600.0, "bf16_tflops_sustained": 1600.0, "source": "measured"}
    (tmp_path / "MEASURED_PEAKS.json").write_text(json.dumps({"hbm_gbs": 6500, "bf16_tflops": 1600, "bf16_tflops_sustained": 1380}))
    assert bench.measured_peaks()["bf16_tflops_sustained"] == 1380.0


def test_reference_arm_prints_one_line_with_the_contract_keys():
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "1", "--steps", "1",
                        "--warmup", "0"], capture_output=True, text=True, timeout=600, env=env, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["metric"] == bench.METRIC and line["unit"] == "TB/s"
    assert line["higher_is_better"] is True and line["dtype"] == "f64" and line["vs_baseline"] is None
    assert line["config"]["workload"].startswith("config1") and line["steps"] == 1 and line["n_gpus"] == 1
    cb = line["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] == line["value"] > 0 and "decode requests" in cb["sample"]
    assert line["e2e"] == {"value": line["value"], "unit": "TB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
