"""ctypes binding of the scheduler-side entry points (``include/polyserve_sched.h``) -- argument marshalling only.

Same shared library as the attention entry points, same names and argument
order as the C declarations.  These calls are host code: no device is needed.
"""
from __future__ import annotations

import ctypes

import numpy as np

from . import binding as B

EXPORTS = ["ps_table_build", "ps_table_build_overlap", "ps_table_get_overlap", "ps_table_from_lines", "ps_table_free", "ps_table_add_batch_term", "ps_table_scale", "ps_table_size",
           "ps_table_get_lines",
           "ps_table_predict", "ps_peak_kv", "ps_admit", "ps_chunk_next", "ps_chunk_schedule", "ps_chunk_predict"]

_vp, _i32, _i64, _f64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_double
_i32p, _f64p = ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_double)
_ready = False


def _lib():
    global _ready
    lib = B.load()
    if not _ready:
        lib.ps_table_build.argtypes = [ctypes.POINTER(B.ps_grid_row), _i64, ctypes.POINTER(_vp)]
        lib.ps_table_build_overlap.argtypes = [ctypes.POINTER(B.ps_grid_row), _i64, ctypes.POINTER(_vp)]
        lib.ps_table_get_overlap.argtypes = [_vp, ctypes.POINTER(_i32), _f64p, _f64p, _i32]
        lib.ps_table_from_lines.argtypes = [_i32p, _f64p, _f64p, _f64p, _i32, ctypes.POINTER(_vp)]
        lib.ps_table_free.argtypes = [_vp]
        lib.ps_table_add_batch_term.argtypes = [_vp, _i32p, _f64p, _i32]
        lib.ps_table_scale.argtypes = [_vp, _f64]
        lib.ps_table_size.argtypes = [_vp, ctypes.POINTER(_i32)]
        lib.ps_table_get_lines.argtypes = [_vp, _i32p, _f64p, _f64p, _f64p, _i32]
        lib.ps_table_predict.argtypes = [_vp, _i32, _i64, _f64, _f64p]
        lib.ps_peak_kv.argtypes = [_i32p, _i32p, _i32, ctypes.POINTER(_i64), ctypes.POINTER(_i32)]
        lib.ps_admit.argtypes = [_vp, _i32p, _i32p, _i32, _i32, _i32, _i32, _i64, _f64, _f64, ctypes.POINTER(_i32), _f64p,
                                 ctypes.POINTER(_i64)]
        lib.ps_chunk_next.argtypes = [_i32p, _i32, _i32, _i32, _i32, _i32p]
        lib.ps_chunk_schedule.argtypes = [_i32, _i32, _i32, _i32, _i32p, _i32, ctypes.POINTER(_i32)]
        lib.ps_chunk_predict.argtypes = [_vp, _i32p, _i32p, _i32, _i32, _i32, _f64, _f64, ctypes.POINTER(_i32),
                                         ctypes.POINTER(_i32), _f64p, ctypes.POINTER(_i32)]
        for name in EXPORTS:
            getattr(lib, name).restype = ctypes.c_int
        _ready = True
    return lib


def _host_f64(a):
    arr = np.ascontiguousarray(a, dtype=np.float64)
    return arr, arr.ctypes.data_as(_f64p)


def ps_table_build(rows):
    """rows: a sequence of ps_grid_row (as ps_profile_grid returns).  Returns the opaque table handle."""
    arr = (B.ps_grid_row * len(rows))(*rows)
    out = _vp(0)
    B._check(_lib().ps_table_build(arr, len(rows), ctypes.byref(out)))
    return out.value


def ps_table_build_overlap(rows):
    """The sweep fitted as base + max(decode term, prefill term) (one set of parameters for all lines)."""
    arr = (B.ps_grid_row * len(rows))(*rows)
    out = _vp(0)
    B._check(_lib().ps_table_build_overlap(arr, len(rows), ctypes.byref(out)))
    return out.value


def ps_table_get_overlap(table):
    """Returns None for a sum-form table, else (decode_intercept_us, prefill_intercept_us: float64[n])."""
    flag = _i32(0)
    B._check(_lib().ps_table_get_overlap(table, ctypes.byref(flag), None, None, 0))
    if not flag.value:
        return None
    n = ps_table_size(table)
    a_d, a_p = np.zeros(n, np.float64), np.zeros(n, np.float64)
    B._check(_lib().ps_table_get_overlap(table, ctypes.byref(flag), a_d.ctypes.data_as(_f64p), a_p.ctypes.data_as(_f64p), n))
    return a_d, a_p


def ps_table_from_lines(token_batch, intercept_us, slope_us_per_token, slope_us_per_flop=None):
    b, bp = B._host_i32(token_batch)
    a, ap = _host_f64(intercept_us)
    s, sp = _host_f64(slope_us_per_token)
    q, qp = _host_f64(slope_us_per_flop) if slope_us_per_flop is not None else (None, None)
    out = _vp(0)
    B._check(_lib().ps_table_from_lines(bp, ap, sp, qp, b.shape[0], ctypes.byref(out)))
    return out.value


def ps_table_free(table):
    B._check(_lib().ps_table_free(table))


def ps_table_add_batch_term(table, token_batch, term_us):
    """Adds a batch-size-only term (the model's GEMM time at the sampled batch sizes) to every line, in place."""
    b, bp = B._host_i32(token_batch)
    t, tp = _host_f64(term_us)
    B._check(_lib().ps_table_add_batch_term(table, bp, tp, b.shape[0]))


def ps_table_scale(table, factor: float):
    B._check(_lib().ps_table_scale(table, factor))


def ps_table_size(table) -> int:
    n = _i32(0)
    B._check(_lib().ps_table_size(table, ctypes.byref(n)))
    return n.value


def ps_table_get_lines(table):
    """Returns (token_batch int32[n], intercept_us, slope_us_per_token, slope_us_per_flop: float64[n]), sorted by batch size."""
    n = ps_table_size(table)
    b, a, s, q = np.zeros(n, np.int32), np.zeros(n, np.float64), np.zeros(n, np.float64), np.zeros(n, np.float64)
    B._check(_lib().ps_table_get_lines(table, b.ctypes.data_as(_i32p), a.ctypes.data_as(_f64p), s.ctypes.data_as(_f64p),
                                       q.ctypes.data_as(_f64p), n))
    return b, a, s, q


def ps_table_predict(table, token_batch: int, kv_tokens: int, prefill_flops: float = 0.0) -> float:
    out = _f64(0.0)
    B._check(_lib().ps_table_predict(table, token_batch, kv_tokens, prefill_flops, ctypes.byref(out)))
    return out.value


def ps_peak_kv(kv_len, remaining):
    """Returns (peak KV tokens, first iteration where it occurs)."""
    kv, kvp = B._host_i32(kv_len)
    rm, rmp = B._host_i32(remaining)
    peak, when = _i64(0), _i32(0)
    B._check(_lib().ps_peak_kv(kvp, rmp, kv.shape[0], ctypes.byref(peak), ctypes.byref(when)))
    return peak.value, when.value


def ps_admit(table, kv_len, remaining, new_kv_len, new_remaining, extra_tokens, extra_kv_tokens, extra_prefill_flops, tpot_us):
    """Returns (admitted: bool, predicted_us, peak_kv of the decode requests)."""
    kv, kvp = B._host_i32(kv_len)
    rm, rmp = B._host_i32(remaining)
    ok, pred, peak = _i32(0), _f64(0.0), _i64(0)
    B._check(_lib().ps_admit(table, kvp, rmp, kv.shape[0], new_kv_len, new_remaining, extra_tokens, extra_kv_tokens,
                             extra_prefill_flops, tpot_us,
                             ctypes.byref(ok), ctypes.byref(pred), ctypes.byref(peak)))
    return bool(ok.value), pred.value, peak.value


def ps_chunk_next(remaining, budget, used, dynamic):
    rm, rmp = B._host_i32(remaining)
    out = np.zeros(rm.shape[0], np.int32)
    B._check(_lib().ps_chunk_next(rmp, rm.shape[0], budget, used, int(bool(dynamic)), out.ctypes.data_as(_i32p)))
    return out


def ps_chunk_schedule(prompt_len, budget, first_free, dynamic, capacity=None):
    cap = capacity if capacity is not None else prompt_len // max(budget, 1) + 4
    out, n = np.zeros(max(cap, 1), np.int32), _i32(0)
    B._check(_lib().ps_chunk_schedule(prompt_len, budget, first_free, int(bool(dynamic)), out.ctypes.data_as(_i32p), cap,
                                      ctypes.byref(n)))
    return out[: n.value]


def ps_chunk_predict(table, kv_len, remaining, prompt_len, max_chunk, flops_per_pair, tpot_us):
    """Returns (chunk, iterations, completion_us, maintained: bool)."""
    kv, kvp = B._host_i32(kv_len)
    rm, rmp = B._host_i32(remaining)
    c, it, tot, kept = _i32(0), _i32(0), _f64(0.0), _i32(0)
    B._check(_lib().ps_chunk_predict(table, kvp, rmp, kv.shape[0], prompt_len, max_chunk, flops_per_pair, tpot_us, ctypes.byref(c),
                                     ctypes.byref(it), ctypes.byref(tot), ctypes.byref(kept)))
    return c.value, it.value, tot.value, bool(kept.value)
