"""ctypes binding of ``libpolyserve_attn.so`` -- argument marshalling only.

Every function has the name and argument order of its C declaration in
``include/polyserve_attn.h``; all arithmetic runs in the CUDA kernels behind
the C ABI.  Device pointers may be given as integers or as objects with a
``data_ptr()`` method (torch tensors); host arrays are converted to contiguous
int32 numpy arrays.  A non-zero status raises :class:`PsError`.

There is no CPU path: if the shared library cannot be loaded the import of
this module fails.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

from .build import LIB, build_library

PS_OK, PS_ERR_INVALID, PS_ERR_OOM, PS_ERR_CUDA, PS_ERR_UNSUPPORTED, PS_ERR_WORKSPACE, PS_ERR_BOUNDS, PS_ERR_TIMEOUT = range(8)
_STATUS_NAMES = ["PS_OK", "PS_ERR_INVALID", "PS_ERR_OOM", "PS_ERR_CUDA", "PS_ERR_UNSUPPORTED", "PS_ERR_WORKSPACE",
                 "PS_ERR_BOUNDS", "PS_ERR_TIMEOUT"]


class PsError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__("%s: %s" % (_STATUS_NAMES[status] if 0 <= status < 8 else status, message))
        self.status = status


class ps_shape(ctypes.Structure):
    _fields_ = [("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("page_size", ctypes.c_int32), ("dtype", ctypes.c_int32)]


class ps_plan_opts(ctypes.Structure):
    _fields_ = [("decode_segment_tokens", ctypes.c_int32), ("prefill_segment_tokens", ctypes.c_int32),
                ("num_sms", ctypes.c_int32)]


class ps_plan_info(ctypes.Structure):
    _fields_ = [("n_decode_items", ctypes.c_int32), ("n_prefill_items", ctypes.c_int32), ("n_merge_rows", ctypes.c_int32),
                ("decode_segment_tokens", ctypes.c_int32), ("prefill_segment_tokens", ctypes.c_int32),
                ("n_partial_slots", ctypes.c_int64), ("total_q_tokens", ctypes.c_int64), ("n_launches", ctypes.c_int32),
                ("decode_sms", ctypes.c_int32), ("prefill_sms", ctypes.c_int32)]


class ps_grid_spec(ctypes.Structure):
    _fields_ = [("chunk_sizes", ctypes.POINTER(ctypes.c_int32)), ("n_chunk_sizes", ctypes.c_int32),
                ("decode_counts", ctypes.POINTER(ctypes.c_int32)), ("n_decode_counts", ctypes.c_int32),
                ("mean_ctxs", ctypes.POINTER(ctypes.c_int32)), ("n_mean_ctxs", ctypes.c_int32),
                ("seeds_per_cell", ctypes.c_int32), ("warmup", ctypes.c_int32), ("iters", ctypes.c_int32),
                ("seed_base", ctypes.c_uint64), ("include_kv_write", ctypes.c_int32),
                ("hbm_peak_gbs", ctypes.c_double), ("bf16_peak_tflops", ctypes.c_double)]


class ps_grid_row(ctypes.Structure):
    _fields_ = [("chunk", ctypes.c_int32), ("n_decode", ctypes.c_int32), ("mean_ctx", ctypes.c_int32),
                ("seed_index", ctypes.c_int32), ("seed", ctypes.c_uint64), ("token_batch", ctypes.c_int32),
                ("prefill_prior", ctypes.c_int32), ("kv_tokens", ctypes.c_int64), ("decode_bytes", ctypes.c_double),
                ("prefill_flops", ctypes.c_double), ("latency_us", ctypes.c_float), ("latency_min_us", ctypes.c_float),
                ("latency_max_us", ctypes.c_float), ("plan_us", ctypes.c_float), ("decode_TBps", ctypes.c_float),
                ("prefill_TFLOPs", ctypes.c_float), ("roofline_frac", ctypes.c_float)]


EXPORTS = ["ps_kv_bytes", "ps_kv_alloc", "ps_kv_free", "ps_kv_write", "ps_kv_gather", "ps_kv_gather_fp8", "ps_kv_status", "ps_attn_plan",
           "ps_plan_free", "ps_plan_get_info", "ps_plan_get_items", "ps_attn_run", "ps_plan_status",
           "ps_plan_set_timing", "ps_plan_get_timing", "ps_plan_set_wait_limit", "ps_profile_grid", "ps_attn_run_static",
           "ps_last_error", "ps_version"]

_lib = None
_vp, _i32, _i64, _sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
_i32p = ctypes.POINTER(ctypes.c_int32)


def load() -> ctypes.CDLL:
    """Load (building first if the sources are newer) the shared library."""
    global _lib
    if _lib is not None:
        return _lib
    path = LIB
    if os.environ.get("PS_ATTN_NO_BUILD") != "1":
        path = build_library()
    lib = ctypes.CDLL(path)
    sp = ctypes.POINTER(ps_shape)
    lib.ps_kv_bytes.argtypes = [sp, _i64, ctypes.POINTER(_sz)]
    lib.ps_kv_alloc.argtypes = [sp, _i64, _vp, _sz, ctypes.POINTER(_vp)]
    lib.ps_kv_free.argtypes = [_vp]
    lib.ps_kv_write.argtypes = [_vp, _vp, _vp, _vp, _i32, _i32p, _i32p, _i32, _vp]
    lib.ps_kv_gather.argtypes = [_vp, _vp, _i32, _vp, _vp, _vp]
    lib.ps_kv_gather_fp8.argtypes = [_vp, _vp, _i32, _vp, _vp, _vp, _vp, _vp]
    lib.ps_kv_status.argtypes = [_vp, _vp]
    lib.ps_attn_plan.argtypes = [sp, _i32p, _i32p, _i32, _i32, ctypes.POINTER(ps_plan_opts), ctypes.POINTER(_vp),
                                 ctypes.POINTER(_sz)]
    lib.ps_plan_free.argtypes = [_vp]
    lib.ps_plan_get_info.argtypes = [_vp, ctypes.POINTER(ps_plan_info)]
    lib.ps_plan_get_items.argtypes = [_vp, _i32p, _i64, _i32p, _i64]
    lib.ps_attn_run.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
    lib.ps_plan_status.argtypes = [_vp, _vp]
    lib.ps_attn_run_static.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp]
    lib.ps_plan_set_timing.argtypes = [_vp, _i32]
    lib.ps_plan_set_wait_limit.argtypes = [_vp, _i64]
    fp = ctypes.POINTER(ctypes.c_float)
    lib.ps_plan_get_timing.argtypes = [_vp, _vp, fp, fp, fp, ctypes.POINTER(_i32)]
    lib.ps_profile_grid.argtypes = [sp, ctypes.POINTER(ps_grid_spec), ctypes.POINTER(ps_grid_row), _i64,
                                    ctypes.POINTER(_i64), ctypes.c_char_p, _vp]
    for name in EXPORTS:
        getattr(lib, name).restype = ctypes.c_int
    lib.ps_last_error.restype = ctypes.c_char_p
    lib.ps_last_error.argtypes = []
    lib.ps_version.restype = ctypes.c_char_p
    lib.ps_version.argtypes = []
    _lib = lib
    return lib


def _check(status: int):
    if status != PS_OK:
        raise PsError(status, load().ps_last_error().decode())


def _ptr(x):
    if x is None:
        return None
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    return int(x)


def _host_i32(a):
    arr = np.ascontiguousarray(a, dtype=np.int32)
    return arr, arr.ctypes.data_as(_i32p)


def make_shape(n_q_heads, n_kv_heads, head_dim, page_size=16, dtype=0) -> ps_shape:
    return ps_shape(n_q_heads, n_kv_heads, head_dim, page_size, dtype)


def ps_last_error() -> str:
    return load().ps_last_error().decode()


def ps_version() -> str:
    return load().ps_version().decode()


def ps_kv_bytes(shape: ps_shape, num_pages: int) -> int:
    out = _sz(0)
    _check(load().ps_kv_bytes(ctypes.byref(shape), num_pages, ctypes.byref(out)))
    return out.value


def ps_kv_alloc(shape: ps_shape, num_pages: int, dev_mem=None, dev_bytes: int = 0):
    """Returns the opaque pool handle (an integer)."""
    out = _vp(0)
    _check(load().ps_kv_alloc(ctypes.byref(shape), num_pages, _ptr(dev_mem), dev_bytes, ctypes.byref(out)))
    return out.value


def ps_kv_free(kv):
    _check(load().ps_kv_free(kv))


def ps_kv_write(kv, k_new_dev, v_new_dev, block_table_dev, max_pages, prior_host, q_len_host, stream=None):
    pr, prp = _host_i32(prior_host)
    ql, qlp = _host_i32(q_len_host)
    _check(load().ps_kv_write(kv, _ptr(k_new_dev), _ptr(v_new_dev), _ptr(block_table_dev), max_pages, prp, qlp,
                              pr.shape[0], _ptr(stream)))


def ps_kv_gather(kv, block_table_row_dev, length, k_out_dev, v_out_dev, stream=None):
    _check(load().ps_kv_gather(kv, _ptr(block_table_row_dev), length, _ptr(k_out_dev), _ptr(v_out_dev), _ptr(stream)))


def ps_kv_gather_fp8(kv, block_table_row_dev, length, k_codes_out_dev, v_codes_out_dev, k_scale_out_dev, v_scale_out_dev, stream=None):
    _check(load().ps_kv_gather_fp8(kv, _ptr(block_table_row_dev), length, _ptr(k_codes_out_dev), _ptr(v_codes_out_dev),
                                   _ptr(k_scale_out_dev), _ptr(v_scale_out_dev), _ptr(stream)))


def ps_kv_status(kv, stream=None):
    _check(load().ps_kv_status(kv, _ptr(stream)))


def ps_attn_plan(shape: ps_shape, prior_host, q_len_host, max_pages_per_seq, opts: ps_plan_opts | None = None, plan=None):
    """Returns (plan handle, workspace bytes).  Pass ``plan`` to rebuild an existing handle in place."""
    pr, prp = _host_i32(prior_host)
    ql, qlp = _host_i32(q_len_host)
    handle = _vp(plan or 0)
    ws = _sz(0)
    _check(load().ps_attn_plan(ctypes.byref(shape), prp, qlp, pr.shape[0], max_pages_per_seq,
                               ctypes.byref(opts) if opts is not None else None, ctypes.byref(handle), ctypes.byref(ws)))
    return handle.value, ws.value


def ps_plan_free(plan):
    _check(load().ps_plan_free(plan))


def ps_plan_get_info(plan) -> ps_plan_info:
    info = ps_plan_info()
    _check(load().ps_plan_get_info(plan, ctypes.byref(info)))
    return info


def ps_plan_get_items(plan):
    """Returns (decode items [Nd, 8], prefill items [Np, 8]) as int32 arrays."""
    info = ps_plan_get_info(plan)
    dec = np.zeros((info.n_decode_items, 8), dtype=np.int32)
    pre = np.zeros((info.n_prefill_items, 8), dtype=np.int32)
    _check(load().ps_plan_get_items(plan, dec.ctypes.data_as(_i32p), dec.shape[0], pre.ctypes.data_as(_i32p), pre.shape[0]))
    return dec, pre


def ps_attn_run(plan, kv, q_dev, block_table_dev, out_dev, lse_out_dev, workspace_dev, workspace_bytes, stream=None):
    _check(load().ps_attn_run(plan, kv, _ptr(q_dev), _ptr(block_table_dev), _ptr(out_dev), _ptr(lse_out_dev),
                              _ptr(workspace_dev), workspace_bytes, _ptr(stream)))


PS_STATIC_WORKSPACE_BYTES = 8 << 20


def ps_attn_run_static(plan, kv, q_dev, block_table_dev, out_dev, lse_out_dev, stream=None):
    """ps_attn_run on the library's built-in scratch array: no workspace argument, no allocation.

    For callers that may not allocate device memory when they need attention.
    Plans needing more than PS_STATIC_WORKSPACE_BYTES raise PS_ERR_WORKSPACE.
    Calls on one device share the array: do not let two of them overlap on the GPU.
    """
    _check(load().ps_attn_run_static(plan, kv, _ptr(q_dev), _ptr(block_table_dev), _ptr(out_dev), _ptr(lse_out_dev),
                                     _ptr(stream)))


def ps_plan_status(plan, stream=None):
    _check(load().ps_plan_status(plan, _ptr(stream)))


def ps_plan_set_wait_limit(plan, limit_ns: int):
    _check(load().ps_plan_set_wait_limit(plan, limit_ns))


def ps_plan_set_timing(plan, max_runs: int):
    _check(load().ps_plan_set_timing(plan, max_runs))


def ps_plan_get_timing(plan, stream=None):
    """Returns (prefill_ms, decode_ms, merge_ms, n_runs): mean per-kernel time of the recorded runs."""
    a, b, c, n = ctypes.c_float(0), ctypes.c_float(0), ctypes.c_float(0), _i32(0)
    _check(load().ps_plan_get_timing(plan, _ptr(stream), ctypes.byref(a), ctypes.byref(b), ctypes.byref(c), ctypes.byref(n)))
    return a.value, b.value, c.value, n.value


def ps_profile_grid(shape: ps_shape, chunk_sizes, decode_counts, mean_ctxs, seeds_per_cell, warmup, iters, seed_base,
                    csv_path=None, stream=None, include_kv_write=False, hbm_peak_gbs=0.0, bf16_peak_tflops=0.0):
    """Returns the list of ps_grid_row in sweep order."""
    ca, cp = _host_i32(chunk_sizes)
    da, dp = _host_i32(decode_counts)
    ma, mp = _host_i32(mean_ctxs)
    spec = ps_grid_spec(cp, ca.shape[0], dp, da.shape[0], mp, ma.shape[0], seeds_per_cell, warmup, iters, seed_base,
                        int(bool(include_kv_write)), float(hbm_peak_gbs), float(bf16_peak_tflops))
    n = ca.shape[0] * da.shape[0] * ma.shape[0] * seeds_per_cell
    rows = (ps_grid_row * n)()
    n_out = _i64(0)
    _check(load().ps_profile_grid(ctypes.byref(shape), ctypes.byref(spec), rows, n, ctypes.byref(n_out),
                                  csv_path.encode() if csv_path else None, _ptr(stream)))
    return [rows[i] for i in range(n_out.value)]
