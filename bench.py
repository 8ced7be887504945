#!/usr/bin/env python
"""Benchmark of one serving iteration's mixed-batch paged-KV attention.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload 1|2|3|4]

A step is one pass of the whole path over one synthetic batch: host work
partition (ps_attn_plan), then ps_attn_run (work-list upload, prefill, decode
and merge kernels).  The default workload is the largest single-GPU batch:
256 decode sequences with contexts uniform on [4096, 32768] beside two
2048-token prefill chunks on 16 k - 30 k prior tokens, 64 q / 8 kv heads (about
19 GB of KV; the two kernels run side by side).  The headline value is the KV
bytes the decode rows must stream divided by the step time; the prefill rows'
TFLOP/s over the same step, the roofline fraction of the step and of each
kernel, and the CPU oracle's rates on a bounded sample are in the same line.  With N > 1 (torchrun) every rank runs its own batch of the same
law (weak scaling, no data-path collective); the step time is the maximum over
ranks and the value the sum of all ranks' bytes over that time.  With
``--shard heads`` the ranks instead split ONE batch by KV head (rank k takes kv
heads [k Hkv / N, (k + 1) Hkv / N) and their q heads; attention needs no
exchange between heads), which is strong scaling.

Prints one JSON line.  ``--impl reference`` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from workloads import gen  # noqa: E402

METRIC = "mixed-batch attn: decode HBM TB/s, prefill TFLOP/s, % roofline, iter latency"
WORKLOADS = {
    1: ("config1: decode-only, 32q/8kv heads, d=128, page 16, 64 seqs, ctx U[512,4096]", gen.config1, 1001),
    2: ("config2: 2048-token budget, 1536-token chunk + 512 decode seqs lognormal ctx", gen.config2, 1002),
    4: ("config4: 64q/8kv heads, 256 decode seqs ctx U[4096,32768] + two 2048-token chunks", gen.config4, 1004),
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# dram__bytes_read.sum + dram__bytes_write.sum of one launch, as a multiple of the launch's algorithmic bytes, from the
# ncu captures summarised under profiles/ (small cases of the same kernels; DRAM traffic of both kernels grows in
# proportion to the KV a launch reads, so a full launch is the ratio times its algorithmic bytes).  The decode
# kernel's algorithmic bytes are the KV it streams; for the prefill kernel the ratio is per KV byte of its chunks'
# sequences (its K/V tiles are re-read from L2, not from DRAM).  Re-captured whenever a kernel changes.
NCU_TRAFFIC_RATIO = {"decode_kernel": 1.009}
NCU_TRAFFIC_SOURCE = "profiles/mixed_step_config2.md"


def ncu_traffic(kernel, algorithmic_units):
    """DRAM bytes per launch of ``kernel`` scaled from the committed capture, or None where no capture exists."""
    ratio = NCU_TRAFFIC_RATIO.get(kernel)
    return None if ratio is None else ratio * algorithmic_units


class ClockSampler:
    """Samples SM clocks and throttle reasons while the timed region runs: through NVML (read-only queries, every
    few milliseconds) when its Python binding is there, else by polling nvidia-smi."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index: int):
        self.index = index
        self.samples = []  # (sm_mhz, sm_max_mhz, [flags in the order of NAMES])
        self.source = "nvidia-smi"
        self._stop = threading.Event()
        self._nvml = None
        try:
            import pynvml

            pynvml.nvmlInit()
            # torch numbers the visible devices; NVML numbers all of them
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = index
            if visible:
                ids = [v.strip() for v in visible.split(",") if v.strip()]
                if index < len(ids) and ids[index].isdigit():
                    phys = int(ids[index])
            self._handle = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self._max = float(pynvml.nvmlDeviceGetMaxClockInfo(self._handle, pynvml.NVML_CLOCK_SM))
            self._nvml = pynvml
            self.source = "nvml"
        except Exception:
            self._nvml = None
        self._thread = threading.Thread(target=self._run_nvml if self._nvml else self._run_smi, daemon=True)

    def _run_nvml(self):
        n = self._nvml
        masks = [n.nvmlClocksEventReasonHwSlowdown, n.nvmlClocksEventReasonHwThermalSlowdown,
                 n.nvmlClocksEventReasonSwThermalSlowdown, n.nvmlClocksEventReasonSwPowerCap]
        while not self._stop.is_set():
            try:
                mhz = float(n.nvmlDeviceGetClockInfo(self._handle, n.NVML_CLOCK_SM))
                reasons = int(n.nvmlDeviceGetCurrentClocksEventReasons(self._handle))
                self.samples.append((mhz, self._max, [bool(reasons & m) for m in masks]))
            except Exception:
                pass
            self._stop.wait(0.002)

    def _run_smi(self):
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                                      "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=5).stdout
                parts = [x.strip() for x in out.strip().split(",")]
                if len(parts) >= 6 and parts[0].replace(".", "").isdigit() and parts[1].replace(".", "").isdigit():
                    self.samples.append((float(parts[0]), float(parts[1]), [x.lower().startswith("active") for x in parts[2:6]]))
            except Exception:
                pass
            self._stop.wait(0.1)

    def __enter__(self):
        self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._thread.join(timeout=10)

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no clock samples"], "source": self.source}
        reasons = [nm for k, nm in enumerate(self.NAMES) if any(s[2][k] for s in self.samples)]
        return {"sm_mhz": statistics.median(s[0] for s in self.samples), "sm_max_mhz": max(s[1] for s in self.samples),
                "reasons": reasons, "samples": len(self.samples), "source": self.source}


def dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def reduce_over_ranks(local_ms: float, local_units: float, world: int, device=None):
    """(max over ranks of the time, sum over ranks of the units) via torch.distributed."""
    if world == 1:
        return local_ms, local_units
    import torch
    import torch.distributed as dist

    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    u = torch.tensor([local_units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def shard_batch(make, seed, rank, world, shard):
    """This rank's share of the job.  "requests": its own batch of the same law (replicas, weak scaling).  "heads":
    the one batch of `seed`, cut by KV head -- same lengths and pages on every rank, Hkv / world kv heads and
    their q heads each (strong scaling; head slices never exchange anything inside attention)."""
    if shard == "requests" or world == 1:
        return make(seed + 100 * rank)
    full = make(seed)
    s = full.shape
    if s.n_kv_heads % world != 0:
        raise SystemExit("--shard heads: %d kv heads do not divide over %d ranks" % (s.n_kv_heads, world))
    part = gen.Shape(s.n_q_heads // world, s.n_kv_heads // world, s.head_dim, s.page_size)
    return gen.make_batch(part, seed, full.prior, full.q_len)


def oracle_sample(batch, dec_flops=4e10, pf_flops=8e10):
    """A bounded sample of ``batch`` for the CPU oracle: decode requests from the front of the batch up to
    ``dec_flops`` of fp64 work, and new-token rows spread evenly over every prefill chunk up to ``pf_flops``.
    Returns (decode requests, {chunk request: row indices})."""
    s = batch.shape
    phi = 4.0 * s.head_dim * s.n_q_heads
    dec, tot = [], 0.0
    for r in range(batch.n):
        if batch.q_len[r] > 1:
            continue
        cost = phi * (float(batch.prior[r]) + 1.0)
        if dec and tot + cost > dec_flops:
            break
        dec.append(r)
        tot += cost
    chunks = [r for r in range(batch.n) if batch.q_len[r] > 1]
    rows = {}
    for r in chunks:
        per_row = phi * (float(batch.prior[r]) + 0.5 * float(batch.q_len[r]))
        k = int(max(1, min(int(batch.q_len[r]), pf_flops / len(chunks) / per_row)))
        rows[r] = sorted(set(np.linspace(0, int(batch.q_len[r]) - 1, k).astype(int).tolist()))
    return dec, rows


def sample_text(batch, dec, rows):
    n_dec = int((batch.q_len == 1).sum())
    txt = "%d of %d decode requests" % (len(dec), n_dec)
    if rows:
        txt += " + %d of %d chunk rows (evenly spaced over %d chunk%s)" % (
            sum(len(v) for v in rows.values()), int(batch.q_len[batch.q_len > 1].sum()), len(rows), "s" if len(rows) > 1 else "")
    return txt + "; the whole step's time is extrapolated from the two measured rates by algorithmic work"


def host_bits(batch, r, device):
    """K, V and Q bit patterns of request r on the host.  With a CUDA device they come from the input generator's
    device twin (bit-identical to the numpy generator, which needs minutes for the large configs)."""
    import torch

    s = batch.shape
    lo, hi = int(batch.prior[r]), int(batch.kv_len[r])
    if device is not None:
        from workloads import gen_cuda

        def bits(t):
            return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)

        k, v = gen_cuda.gen_kv(batch.seed, r, 0, hi, s.n_kv_heads, s.head_dim, device)
        return bits(k), bits(v), bits(gen_cuda.gen_q(batch.seed, r, lo, hi, s.n_q_heads, s.head_dim, device))
    k, v = batch.kv_bits(r)
    return k, v, gen.gen_q(batch.seed, r, lo, hi, s.n_q_heads, s.head_dim)


class OracleSample:
    """Inputs of a bounded sample, built once; ``time()`` runs the oracle on them and returns the two rates."""

    def __init__(self, batch, dec, rows, device=None):
        import oracle

        self.batch, self.dec, self.rows = batch, dec, rows
        s = batch.shape
        self.parts = []
        for reqs, row_sel in ((dec, None), (sorted(rows), rows)):
            if not reqs:
                self.parts.append(None)
                continue
            ks, vs, qs = [], [], []
            for r in reqs:
                k, v, q = host_bits(batch, r, device)
                ks.append(k)
                vs.append(v)
                qs.append(q)
            need = [(x.shape[0] + s.page_size - 1) // s.page_size for x in ks]
            bt = np.full((len(reqs), max(need)), -1, dtype=np.int32)
            off = 0
            for a, c in enumerate(need):
                bt[a, :c] = np.arange(off, off + c)
                off += c
            kp = oracle.plain_pool(ks, bt, off + 1, s.page_size)
            vp = oracle.plain_pool(vs, bt, off + 1, s.page_size)
            row_req, row_tok, work = [], [], 0.0
            for a, r in enumerate(reqs):
                for i in (range(int(batch.q_len[r])) if row_sel is None else row_sel[r]):
                    row_req.append(a)
                    row_tok.append(i)
                    work += float(batch.prior[r]) + i + 1.0  # keys this row sees
            self.parts.append((np.concatenate(qs), kp, vp, bt, batch.prior[reqs], batch.q_len[reqs], row_req, row_tok, work))

    def time(self):
        """(seconds on the decode sample, its KV bytes, seconds on the chunk-row sample, its flops, threads)."""
        import oracle

        s = self.batch.shape
        res = []
        for part in self.parts:
            if part is None:
                res.append((0.0, 0.0))
                continue
            q, kp, vp, bt, prior, q_len, row_req, row_tok, work = part
            t0 = time.perf_counter()
            oracle.attn_rows(q, kp, vp, bt, prior, q_len, s.n_q_heads, s.n_kv_heads, s.head_dim, s.page_size, row_req, row_tok)
            res.append((time.perf_counter() - t0, work))
        (dt_d, keys_d), (dt_p, keys_p) = res
        return dt_d, keys_d * s.kv_token_bytes, dt_p, keys_p * 4.0 * s.head_dim * s.n_q_heads, oracle.num_threads()

    def whole_step(self, dt_d, bytes_d, dt_p, flops_p):
        """Seconds the oracle would need for the whole batch, from the two measured rates."""
        full = 0.0
        if bytes_d > 0:
            full += float(self.batch.decode_bytes()) * dt_d / bytes_d
        if flops_p > 0:
            full += float(self.batch.prefill_flops()) * dt_p / flops_p
        return full


def cpu_baseline_record(batch, sample, timing):
    dt_d, bytes_d, dt_p, flops_p, threads = timing
    full = sample.whole_step(dt_d, bytes_d, dt_p, flops_p)
    return {"value": float(batch.decode_bytes()) / full / 1e12, "unit": "TB/s", "cores": threads, "kind": "oracle",
            "sample": sample_text(batch, sample.dec, sample.rows), "sample_seconds": dt_d + dt_p,
            "whole_step_seconds_extrapolated": full,
            "decode_TBps": bytes_d / dt_d / 1e12 if dt_d > 0 else None,
            "prefill_TFLOPs": flops_p / dt_p / 1e12 if dt_p > 0 else None}


def components_alone(pa, batch, db, out, steps, peaks):
    """Decode rows alone and prefill rows alone (each planned by itself on all SMs), for attribution in mixed batches.
    Returns one record per row class for the roofline's kernel list."""
    import torch
    import paper_2507_17769_b200 as ps

    res = []
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    q_start = batch.q_start
    stream = torch.cuda.current_stream(db.q.device)
    for name, mask in (("decode", batch.q_len == 1), ("prefill", batch.q_len > 1)):
        idx = np.nonzero(mask)[0]
        rows = torch.from_numpy(idx).to(db.block_table.device)
        bt = db.block_table.index_select(0, rows).contiguous()
        tok = np.concatenate([np.arange(q_start[r], q_start[r] + batch.q_len[r]) for r in idx])
        q = db.q.index_select(0, torch.from_numpy(tok).to(db.q.device)).contiguous()
        o = torch.empty_like(q)
        prior, q_len = batch.prior[idx], batch.q_len[idx]

        def step():
            pa.plan(prior, q_len, batch.max_pages)
            pa.run(q, bt, out=o, want_lse=False)

        for _ in range(3):
            step()
        torch.cuda.synchronize()
        n = max(3, min(steps, 100))
        ev0.record()
        for _ in range(n):
            step()
        ev1.record()
        torch.cuda.synchronize()
        step_ms = ev0.elapsed_time(ev1) / n
        ps.ps_plan_set_timing(pa._plan, n)
        for _ in range(n):
            step()
        pre_ms, dec_ms, _, _ = ps.ps_plan_get_timing(pa._plan, stream.cuda_stream)
        ps.ps_plan_set_timing(pa._plan, 0)
        if name == "decode":
            res.append(kernel_record("decode_kernel", "decode rows alone on all SMs", dec_ms, float(batch.decode_bytes()), peaks,
                                     step_ms=step_ms))
        else:
            res.append(kernel_record("prefill_kernel", "prefill rows alone on all SMs", pre_ms, float(batch.prefill_flops()), peaks,
                                     step_ms=step_ms))
    pa.plan(batch.prior, batch.q_len, batch.max_pages)  # back to the full batch
    return res


def kernel_record(kernel, where, launch_ms, units, peaks, step_ms=None):
    """One entry of the roofline's kernel list: algorithmic units of one launch over its CUDA-event duration."""
    if kernel == "decode_kernel":
        ach = units / (launch_ms * 1e-3) / 1e9 if launch_ms > 0 else 0.0
        rec = {"kernel": kernel, "where": where, "bound": "hbm", "launch_ms": launch_ms, "algorithmic_bytes_per_launch": units,
               "achieved": ach, "unit": "GB/s", "peak": peaks["hbm_gbs"], "frac": ach / peaks["hbm_gbs"]}
    else:
        ach = units / (launch_ms * 1e-3) / 1e12 if launch_ms > 0 else 0.0
        rec = {"kernel": kernel, "where": where, "bound": "tensor", "launch_ms": launch_ms, "algorithmic_flops_per_launch": units,
               "achieved": ach, "unit": "TFLOP/s", "peak": peaks["bf16_tflops"], "frac": ach / peaks["bf16_tflops"],
               "peak_sustained": peaks["bf16_tflops_sustained"], "frac_of_sustained": ach / peaks["bf16_tflops_sustained"]}
    if step_ms is not None:
        rec["step_ms"] = step_ms
    return rec


def run_reference(args):
    rank, _, _ = dist_env()
    if rank != 0:
        return 0
    desc, make, seed = WORKLOADS[args.workload]
    batch = make(seed)
    device = None
    try:
        import torch

        if torch.cuda.is_available():
            device = torch.device("cuda", 0)
    except ImportError:
        pass
    dec, rows = oracle_sample(batch)
    sample = OracleSample(batch, dec, rows, device)
    for _ in range(min(args.warmup, 1)):
        sample.time()
    acc = None
    for _ in range(args.steps):
        t = sample.time()
        acc = t if acc is None else tuple(a + b for a, b in zip(acc[:4], t[:4])) + (t[4],)
    timing = tuple(x / args.steps for x in acc[:4]) + (acc[4],)
    rec = cpu_baseline_record(batch, sample, timing)
    line = {
        "impl": "reference", "metric": METRIC, "value": rec["value"], "unit": "TB/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * rec["sample_seconds"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": desc, "sample": rec["sample"],
                   "note": "a step is one oracle pass over the sample; value = the batch's decode KV bytes over the "
                           "whole-step time extrapolated from the sample's rates"},
        "cpu_baseline": rec,
        "e2e": {"value": rec["value"], "unit": "TB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))
    return 0


def run_ours(args):
    import torch
    import paper_2507_17769_b200 as ps
    from workloads import gen_cuda
    from workloads.device import DeviceBatch

    rank, local_rank, world = dist_env()
    if world != args.gpus:
        raise SystemExit("--gpus %d but WORLD_SIZE=%d: launch N > 1 with torch.distributed.run" % (args.gpus, world))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=dev)

    desc, make, seed = WORKLOADS[args.workload]
    batch = shard_batch(make, seed, rank, world, args.shard)
    s = batch.shape
    fp8 = args.kv_cache == "fp8"
    if fp8 and float(batch.prefill_flops()) > 0:
        raise SystemExit("--kv-cache fp8: the FP8 cache variant serves decode rows only (use --workload 1)")
    db = DeviceBatch(batch, poison=False, device=dev, kv_dtype=1 if fp8 else 0)
    pa = db.pa
    info = db.plan()
    stream = torch.cuda.current_stream(dev)
    out = torch.empty_like(db.q)
    warmup = max(args.warmup, 3)

    def step():
        pa.plan(batch.prior, batch.q_len, batch.max_pages)
        pa.run(db.q, db.block_table, out=out, want_lse=False)

    for _ in range(warmup):
        step()
    pa.check()

    def barrier():
        torch.cuda.synchronize(dev)
        if world > 1:
            import torch.distributed as dist

            dist.barrier()
            torch.cuda.synchronize(dev)

    # ---- device-resident timing ----
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    with ClockSampler(local_rank) as clocks:
        # pass 1: the K timed steps (two events around the whole region)
        ev0.record(stream)
        t_host = time.perf_counter()
        for _ in range(args.steps):
            step()
        host_ms = (time.perf_counter() - t_host) * 1e3 / args.steps
        ev1.record(stream)
        barrier()
        local_ms = ev0.elapsed_time(ev1) / args.steps
        # pass 2: the same steps again with events around every kernel launch (on the stream each kernel is
        # launched on), for the per-kernel durations of the roofline (kept out of pass 1: each extra event costs
        # device time)
        n_kernel_steps = min(args.steps, 1000)
        ps.ps_plan_set_timing(pa._plan, n_kernel_steps)
        for _ in range(n_kernel_steps):
            step()
        pre_ms, dec_ms, mrg_ms, n_timed = ps.ps_plan_get_timing(pa._plan, stream.cuda_stream)
        ps.ps_plan_set_timing(pa._plan, 0)
    pa.check()
    dec_bytes, pf_flops = float(batch.decode_bytes()), float(batch.prefill_flops())
    if fp8:  # one byte per element plus an fp32 scale per (token, kv head) for K and for V
        dec_bytes = float(batch.decode_kv_tokens()) * (2 * s.n_kv_heads * s.head_dim + 2 * s.n_kv_heads * 4)
    ms, units = reduce_over_ranks(local_ms, dec_bytes, world, dev)
    value = units / (ms * 1e-3) / 1e12

    # ---- end to end: host buffers in, host result out, every step ----
    # Inputs of step i + 1 cross to the device, and the output of step i - 1 crosses back, under the kernels of step
    # i: two device input buffers and two output buffers, one stream per copy direction, events for the ordering.
    new_k, new_v = [], []
    for r in range(batch.n):
        k, v = gen_cuda.gen_kv(batch.seed, r, int(batch.prior[r]), int(batch.kv_len[r]), s.n_kv_heads, s.head_dim, dev)
        new_k.append(k)
        new_v.append(v)
    # one pinned staging buffer and one device buffer hold the step's inputs back to back (Q | K | V | block table,
    # each 256-byte aligned), so that a step's inputs cross in a single copy
    parts = [db.q.cpu().contiguous().view(torch.uint8).reshape(-1), torch.cat(new_k).cpu().contiguous().view(torch.uint8).reshape(-1),
             torch.cat(new_v).cpu().contiguous().view(torch.uint8).reshape(-1),
             torch.from_numpy(batch.block_table).contiguous().view(torch.uint8).reshape(-1)]
    del new_k, new_v
    offs, total = [], 0
    for t in parts:
        offs.append(total)
        total += (t.numel() + 255) // 256 * 256
    h_in = torch.zeros(total, dtype=torch.uint8).pin_memory()
    for t, o in zip(parts, offs):
        h_in[o : o + t.numel()] = t
    d_in = [torch.empty(total, dtype=torch.uint8, device=dev) for _ in range(2)]
    d_out = [torch.empty_like(db.q) for _ in range(2)]

    def view(buf, i, dtype, shape):
        return buf[offs[i] : offs[i] + parts[i].numel()].view(dtype).reshape(shape)

    n_new = int(batch.q_len.sum())
    views = [(view(b, 0, torch.bfloat16, db.q.shape), view(b, 1, torch.bfloat16, (n_new, s.n_kv_heads, s.head_dim)),
              view(b, 2, torch.bfloat16, (n_new, s.n_kv_heads, s.head_dim)), view(b, 3, torch.int32, db.block_table.shape))
             for b in d_in]
    h_out = torch.empty(out.shape, dtype=out.dtype).pin_memory()
    h2d = sum(t.numel() for t in parts)
    d2h = h_out.numel() * 2
    s_in, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev)

    def e2e_loop(n):
        """n steps; returns when the last output copy has been ordered into the compute stream."""
        ev_in = [torch.cuda.Event() for _ in range(2)]      # inputs of the step using buffer b are on the device
        ev_read = [torch.cuda.Event() for _ in range(2)]    # the step using buffer b has finished (inputs read, output written)
        ev_back = [torch.cuda.Event() for _ in range(2)]    # output buffer b has been copied to the host
        s_in.wait_stream(stream)

        def send(i):
            b = i & 1
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(ev_read[b])
                d_in[b].copy_(h_in, non_blocking=True)
                ev_in[b].record(s_in)

        send(0)
        for i in range(n):
            b = i & 1
            if i + 1 < n:
                send(i + 1)
            d_q, d_k, d_v, d_bt = views[b]
            stream.wait_event(ev_in[b])
            if i >= 2:
                stream.wait_event(ev_back[b])
            pa.write(d_k, d_v, d_bt, batch.prior, batch.q_len, max_pages=batch.max_pages)
            pa.plan(batch.prior, batch.q_len, batch.max_pages)
            pa.run(d_q, d_bt, out=d_out[b], want_lse=False)
            ev_read[b].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_read[b])
                h_out.copy_(d_out[b], non_blocking=True)
                ev_back[b].record(s_out)
        stream.wait_event(ev_back[(n - 1) & 1])

    e2e_loop(3)
    barrier()
    ev0.record(stream)
    e2e_loop(args.steps)
    ev1.record(stream)
    barrier()
    e2e_ms, e2e_units = reduce_over_ranks(ev0.elapsed_time(ev1) / args.steps, dec_bytes, world, dev)
    pa.check()
    pa.plan(batch.prior, batch.q_len, batch.max_pages)

    line = None
    if rank == 0:
        peaks = measured_peaks()
        # the step against the resource that bounds it when its two kernels overlap perfectly
        t_hbm = dec_bytes / (peaks["hbm_gbs"] * 1e9)
        t_tensor = pf_flops / (peaks["bf16_tflops"] * 1e12)
        mixed = pf_flops > 0 and dec_bytes > 0
        side_by_side = bool(mixed and info.decode_sms != info.prefill_sms)
        where = "mixed step, beside the other kernel" if side_by_side else "whole step"
        kernels = []
        if dec_bytes > 0:
            kernels.append(kernel_record("decode_kernel", where + " (%d SMs)" % info.decode_sms, dec_ms, dec_bytes, peaks))
        if pf_flops > 0:
            kernels.append(kernel_record("prefill_kernel", where + " (%d SMs)" % info.prefill_sms, pre_ms, pf_flops, peaks))
        if mixed:
            kernels.extend(components_alone(pa, batch, db, out, args.steps, peaks))
        if t_hbm >= t_tensor:
            ach = dec_bytes / (ms * 1e-3) / 1e9
            roof = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"],
                    "traffic": None if fp8 else ncu_traffic("decode_kernel", dec_bytes), "dominant_kernel": "decode_kernel"}
        else:
            ach = pf_flops / (ms * 1e-3) / 1e12
            roof = {"bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                    "frac": ach / peaks["bf16_tflops"], "traffic": ncu_traffic("prefill_kernel", pf_flops),
                    "dominant_kernel": "prefill_kernel"}
        roof.update({"peak_source": peaks["source"], "of": "the whole step (ms_per_step)",
                     "bound_times_ms": {"hbm": t_hbm * 1e3, "tensor": t_tensor * 1e3},
                     "traffic_source": NCU_TRAFFIC_SOURCE, "launches_timed": n_timed, "merge_kernel_ms": mrg_ms,
                     "kernels": kernels})
        line = {
            "metric": METRIC, "value": value, "unit": "TB/s", "n_gpus": world, "steps": args.steps, "warmup": warmup,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "strong" if args.shard == "heads" and world > 1 else "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": desc + (" [KV cache in FP8 E4M3 with per-token scales]" if fp8 else ""),
                       "kv_cache": args.kv_cache, "kv_bytes_per_step_per_gpu": dec_bytes, "prefill_flops_per_step_per_gpu": pf_flops,
                       "l2": "inputs larger than L2 (%.0f MB of KV per step), no flush" % (dec_bytes / 1e6),
                       "decode_items": info.n_decode_items, "prefill_items": info.n_prefill_items,
                       "merge_rows": info.n_merge_rows, "decode_sms": info.decode_sms, "prefill_sms": info.prefill_sms,
                       "side_by_side": side_by_side,
                       "parallelism": ("kv heads x%d" if args.shard == "heads" and world > 1 else "replicas x%d") % world},
            "prefill_TFLOPs": pf_flops / (ms * 1e-3) / 1e12 if pf_flops > 0 else None,
            "host_issue_ms_per_step": host_ms,
            "clocks": clocks.summary(),
            "e2e": {"value": e2e_units / (e2e_ms * 1e-3) / 1e12, "unit": "TB/s", "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "note": "per step: new tokens' Q/K/V and block table from pinned host memory, ps_kv_write, plan, run, "
                            "output back to pinned host memory; the next step's input copy and the previous step's output "
                            "copy run on their own streams under this step's kernels; the KV cache of earlier iterations "
                            "stays in HBM"},
            "gpu_launches": args.steps * info.n_launches,
            "roofline": roof,
        }
        # ---- CPU baseline: the oracle as it stands, on the host's cores, on a bounded sample ----
        if world == 1 and not args.no_cpu_baseline and not fp8:
            dec, rows = oracle_sample(batch)
            sample = OracleSample(batch, dec, rows, dev)
            line["cpu_baseline"] = cpu_baseline_record(batch, sample, sample.time())
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist

        dist.barrier()
        dist.destroy_process_group()
    return 0


def run_grid(args):
    """--workload 3: seed 0 of each of the 72 cells of the latency-table grid (the scheduler's profile of section
    4.5): the GPU latency of one ps_attn_run and, beside it, the seconds the CPU oracle needs for the same cell (run in
    full while a cell's fp64 work stays under the sample budgets, else on a bounded sample and extrapolated by work)."""
    import torch
    import paper_2507_17769_b200 as ps  # noqa: F401
    from workloads.device import DeviceBatch

    rank, local_rank, world = dist_env()
    if rank != 0:
        return 0
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; the library has no CPU path")
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    rows, tot_bytes, tot_ms, tot_cpu, threads = [], 0.0, 0.0, 0.0, 1
    for cell, chunk, nd, m in gen.grid_cells():
        batch = gen.config3_cell(chunk, nd, m, gen.grid_seed(cell, 0))
        db = DeviceBatch(batch, poison=False, device=dev)
        db.plan()
        out = torch.empty_like(db.q)
        for _ in range(max(3, args.warmup)):
            db.pa.run(db.q, db.block_table, out=out, want_lse=False)
        n = max(5, min(args.steps, 50))
        torch.cuda.synchronize(dev)
        ev0.record()
        for _ in range(n):
            db.pa.run(db.q, db.block_table, out=out, want_lse=False)
        ev1.record()
        torch.cuda.synchronize(dev)
        db.pa.check()
        gpu_us = ev0.elapsed_time(ev1) / n * 1e3
        cpu_s, sampled = float("nan"), 0
        if not args.no_cpu_baseline:
            dec, rws = oracle_sample(batch)
            sampled = int(len(dec) < nd or sum(len(v) for v in rws.values()) < chunk)
            sample = OracleSample(batch, dec, rws, dev)
            dt_d, bytes_d, dt_p, flops_p, threads = sample.time()
            cpu_s = sample.whole_step(dt_d, bytes_d, dt_p, flops_p)
            tot_cpu += cpu_s
        rows.append((chunk, nd, m, batch.seed, int(batch.kv_len.sum()), batch.decode_bytes(), batch.prefill_flops(), gpu_us,
                     cpu_s, sampled, threads))
        tot_bytes += float(batch.decode_bytes())
        tot_ms += gpu_us * 1e-3
        db.pa.close()
        del db, out
    if args.grid_csv:
        with open(args.grid_csv, "w") as f:
            f.write("chunk,n_decode,mean_ctx,seed,kv_tokens,decode_bytes,prefill_flops,gpu_latency_us,cpu_seconds,cpu_sampled,cpu_cores\n")
            for r in rows:
                f.write("%d,%d,%d,%d,%d,%d,%d,%.3f,%.4f,%d,%d\n" % r)
    line = {"metric": METRIC, "value": tot_bytes / (tot_ms * 1e-3) / 1e12, "unit": "TB/s", "n_gpus": 1, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": tot_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "config3: latency-table grid, seed 0 of each of %d cells (a step = one run of every cell)" % len(rows),
                       "cells": len(rows), "csv": args.grid_csv},
            "cpu_baseline": {"value": tot_bytes / tot_cpu / 1e12 if tot_cpu > 0 else None, "unit": "TB/s", "cores": threads,
                             "kind": "oracle", "seconds_all_cells": tot_cpu,
                             "sample": "every cell; cells above the sample budgets are timed on a bounded sample and extrapolated"}}
    print(json.dumps(line))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=4, choices=sorted(WORKLOADS) + [3])
    ap.add_argument("--grid-csv", default=None, help="--workload 3: write one row per grid cell (GPU latency, CPU oracle seconds)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--kv-cache", default="bf16", choices=["bf16", "fp8"],
                    help="fp8: the E4M3 cache variant of the decode path (decode-only workloads; bytes counted at one per "
                         "element plus the scales)")
    ap.add_argument("--shard", default="requests", choices=["requests", "heads"],
                    help="what N > 1 ranks split: requests (each rank its own batch; default) or the KV heads of one batch")
    args = ap.parse_args()
    if args.workload == 3:
        if args.impl == "reference" or args.gpus != 1:
            raise SystemExit("--workload 3 (the per-cell grid) runs on one GPU with --impl ours")
        return run_grid(args)
    if args.impl == "reference":
        args.steps = min(args.steps, 3)  # each step is seconds of CPU work
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
