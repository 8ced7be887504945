#!/usr/bin/env python
"""Benchmark of one serving iteration's mixed-batch paged-KV attention.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload 1|2|4]

A step is one pass of the whole path over one synthetic batch: host work
partition (ps_attn_plan), then ps_attn_run (work-list upload, prefill, decode
and merge kernels).  The default workload is the decode-only 8B-class batch
(64 sequences, contexts uniform on [512, 4096], about 0.6 GB of KV, larger than
L2); the headline value is the KV bytes the decode rows must stream divided by
the step time.  With N > 1 (torchrun) every rank runs its own batch of the same
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


# dram__bytes_read.sum + dram__bytes_write.sum per launch of the decode kernel from one ncu capture (see
# profiles/decode_kernel_config1.md), valid only for the kernel source it was taken on.
NCU_TRAFFIC = {1: {"decode_cu_sha256_prefix": "740814e60edf27c5", "bytes_per_launch": 600.8e6}}


def ncu_traffic(workload):
    """Measured DRAM traffic per launch, or None if the kernel changed since the counters were taken."""
    import hashlib

    rec = NCU_TRAFFIC.get(workload)
    if rec is None:
        return None
    src = os.path.join(ROOT, "paper_2507_17769_b200", "csrc", "decode.cu")
    try:
        with open(src, "rb") as f:
            digest = hashlib.sha256(f.read()).hexdigest()
    except OSError:
        return None
    return rec["bytes_per_launch"] if digest.startswith(rec["decode_cu_sha256_prefix"]) else None


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


def oracle_sample(batch, budget_flops=6e10):
    """Decode requests of ``batch`` for the CPU oracle, bounded by an fp64 flop budget."""
    s = batch.shape
    cost = 4.0 * s.head_dim * s.n_q_heads * (batch.prior.astype(np.float64) + 1.0)
    picked, tot = [], 0.0
    for r in range(batch.n):
        if batch.q_len[r] > 1:
            continue  # decode rows carry the headline metric
        if tot + cost[r] > budget_flops and picked:
            break
        picked.append(r)
        tot += cost[r]
    return picked


def time_oracle(batch, reqs):
    """Seconds the oracle takes on the given requests (inputs built outside the timed part)."""
    import oracle

    s = batch.shape
    ks, vs, qs = [], [], []
    for r in reqs:
        k, v = batch.kv_bits(r)
        ks.append(k)
        vs.append(v)
        qs.append(gen.gen_q(batch.seed, r, int(batch.prior[r]), int(batch.prior[r] + batch.q_len[r]), s.n_q_heads, s.head_dim))
    need = [(x.shape[0] + s.page_size - 1) // s.page_size for x in ks]
    bt = np.full((len(reqs), max(need)), -1, dtype=np.int32)
    off = 0
    for a, c in enumerate(need):
        bt[a, :c] = np.arange(off, off + c)
        off += c
    kp = oracle.plain_pool(ks, bt, off + 1, s.page_size)
    vp = oracle.plain_pool(vs, bt, off + 1, s.page_size)
    q = np.concatenate(qs)
    args = (q, kp, vp, bt, batch.prior[reqs], batch.q_len[reqs], s.n_q_heads, s.n_kv_heads, s.head_dim, s.page_size)
    t0 = time.perf_counter()
    oracle.attn_paged(*args)
    dt = time.perf_counter() - t0
    nbytes = float((batch.kv_len[reqs][batch.q_len[reqs] == 1]).sum()) * s.kv_token_bytes
    return dt, nbytes, oracle.num_threads()


def components_alone(pa, batch, db, out, steps, peaks):
    """Decode rows alone and prefill rows alone (each on all SMs), for attribution in mixed batches."""
    import torch

    res = {}
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    q_start = batch.q_start
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
        ms = ev0.elapsed_time(ev1) / n
        if name == "decode":
            res["decode_rows_alone_ms"] = ms
            res["decode_rows_alone_TBps"] = float(batch.decode_bytes()) / (ms * 1e-3) / 1e12
        else:
            tf = float(batch.prefill_flops()) / (ms * 1e-3) / 1e12
            res["prefill_rows_alone_ms"] = ms
            res["prefill_rows_alone_TFLOPs"] = tf
            res["prefill_rows_alone_frac_of_bf16_peak"] = tf / peaks["bf16_tflops"]
    pa.plan(batch.prior, batch.q_len, batch.max_pages)  # back to the full batch
    return res


def run_reference(args):
    rank, _, _ = dist_env()
    if rank != 0:
        return 0
    desc, make, seed = WORKLOADS[args.workload]
    batch = make(seed)
    reqs = oracle_sample(batch)
    if args.warmup > 0:
        time_oracle(batch, reqs[:2])
    times, nbytes, threads = [], 0.0, 1
    for _ in range(args.steps):
        dt, nbytes, threads = time_oracle(batch, reqs)
        times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    value = nbytes / (ms * 1e-3) / 1e12
    sample = "%d of %d decode requests (%.1f MB of KV) per step" % (len(reqs), batch.n, nbytes / 1e6)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TB/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": {"workload": desc, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "TB/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
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
    db = DeviceBatch(batch, poison=False, device=dev)
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
        # pass 2: the same steps again with events around every kernel launch, for the per-kernel
        # durations of the roofline (kept out of pass 1: each extra event costs device time)
        n_kernel_steps = min(args.steps, 1000)
        ps.ps_plan_set_timing(pa._plan, n_kernel_steps)
        for _ in range(n_kernel_steps):
            step()
        pre_ms, dec_ms, mrg_ms, n_timed = ps.ps_plan_get_timing(pa._plan, stream.cuda_stream)
        ps.ps_plan_set_timing(pa._plan, 0)
    pa.check()
    dec_bytes, pf_flops = float(batch.decode_bytes()), float(batch.prefill_flops())
    ms, units = reduce_over_ranks(local_ms, dec_bytes, world, dev)
    value = units / (ms * 1e-3) / 1e12

    # ---- end to end: host buffers in, host result out, every step ----
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
    offs, total = [], 0
    for t in parts:
        offs.append(total)
        total += (t.numel() + 255) // 256 * 256
    h_in = torch.zeros(total, dtype=torch.uint8).pin_memory()
    for t, o in zip(parts, offs):
        h_in[o : o + t.numel()] = t
    d_in = torch.empty(total, dtype=torch.uint8, device=dev)

    def view(i, dtype, shape):
        return d_in[offs[i] : offs[i] + parts[i].numel()].view(dtype).reshape(shape)

    n_new = int(batch.q_len.sum())
    d_q = view(0, torch.bfloat16, db.q.shape)
    d_k = view(1, torch.bfloat16, (n_new, s.n_kv_heads, s.head_dim))
    d_v = view(2, torch.bfloat16, (n_new, s.n_kv_heads, s.head_dim))
    d_bt = view(3, torch.int32, db.block_table.shape)
    h_out = torch.empty(out.shape, dtype=out.dtype).pin_memory()
    h2d = sum(t.numel() for t in parts)
    d2h = h_out.numel() * 2

    def e2e_step():
        d_in.copy_(h_in, non_blocking=True)
        pa.write(d_k, d_v, d_bt, batch.prior, batch.q_len, max_pages=batch.max_pages)
        pa.plan(batch.prior, batch.q_len, batch.max_pages)
        pa.run(d_q, d_bt, out=out, want_lse=False)
        h_out.copy_(out, non_blocking=True)

    for _ in range(3):
        e2e_step()
    barrier()
    ev0.record(stream)
    for _ in range(args.steps):
        e2e_step()
    ev1.record(stream)
    barrier()
    e2e_ms, e2e_units = reduce_over_ranks(ev0.elapsed_time(ev1) / args.steps, dec_bytes, world, dev)
    pa.check()

    line = None
    if rank == 0:
        peaks = measured_peaks()
        achieved = dec_bytes / (dec_ms * 1e-3) / 1e9 if dec_ms > 0 else 0.0
        roof = {"kernel": "decode_kernel", "bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "traffic": ncu_traffic(args.workload), "peak_source": peaks["source"],
                "launch_ms": dec_ms, "algorithmic_bytes_per_launch": dec_bytes, "launches_timed": n_timed}
        pf_tf = pf_flops / (pre_ms * 1e-3) / 1e12 if pf_flops > 0 and pre_ms > 0 else None
        extra = {"decode_kernel_ms": dec_ms, "prefill_kernel_ms": pre_ms, "merge_kernel_ms": mrg_ms,
                 "decode_TBps_kernel": achieved / 1e3, "prefill_TFLOPs_kernel": pf_tf,
                 "prefill_frac_of_bf16_peak": pf_tf / peaks["bf16_tflops"] if pf_tf else None,
                 "value_frac_of_nominal_8TBps": value / world / 8.0, "host_issue_ms_per_step": host_ms,
                 "decode_sms": info.decode_sms, "prefill_sms": info.prefill_sms,
                 "side_by_side": bool(pf_flops > 0 and dec_bytes > 0 and info.decode_sms + info.prefill_sms <= 148
                                      and info.decode_sms != info.prefill_sms)}
        if pf_flops > 0 and dec_bytes > 0:
            extra.update(components_alone(pa, batch, db, out, args.steps, peaks))
        line = {
            "metric": METRIC, "value": value, "unit": "TB/s", "n_gpus": world, "steps": args.steps, "warmup": warmup,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "strong" if args.shard == "heads" and world > 1 else "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": desc, "kv_bytes_per_step_per_gpu": dec_bytes, "prefill_flops_per_step_per_gpu": pf_flops,
                       "l2": "inputs larger than L2 (%.0f MB of KV per step), no flush" % (dec_bytes / 1e6),
                       "decode_items": info.n_decode_items, "prefill_items": info.n_prefill_items,
                       "merge_rows": info.n_merge_rows,
                       "parallelism": ("kv heads x%d" if args.shard == "heads" and world > 1 else "replicas x%d") % world},
            "clocks": clocks.summary(),
            "e2e": {"value": e2e_units / (e2e_ms * 1e-3) / 1e12, "unit": "TB/s", "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "note": "per step: new tokens' Q/K/V and block table from pinned host memory, ps_kv_write, plan, run, "
                            "output back to host; the KV cache of earlier iterations stays in HBM"},
            "gpu_launches": args.steps * info.n_launches,
            "roofline": roof,
            "kernels": extra,
        }
        # ---- CPU baseline: the oracle as it stands, on the host's cores ----
        if world == 1 and not args.no_cpu_baseline:
            reqs = oracle_sample(batch)
            dt, nbytes, threads = time_oracle(batch, reqs)
            line["cpu_baseline"] = {"value": nbytes / dt / 1e12, "unit": "TB/s", "cores": threads, "kind": "oracle",
                                    "seconds": dt, "sample": "%d of %d decode requests (%.1f MB of KV), one pass"
                                    % (len(reqs), batch.n, nbytes / 1e6)}
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist

        dist.barrier()
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=1, choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--shard", default="requests", choices=["requests", "heads"],
                    help="what N > 1 ranks split: requests (each rank its own batch; default) or the KV heads of one batch")
    args = ap.parse_args()
    if args.impl == "reference":
        args.steps = min(args.steps, 5)  # each step is seconds of CPU work
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
