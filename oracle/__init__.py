"""CPU fp64 oracle for mixed-batch paged-KV attention (test infrastructure).

Only the tests, the smoke check and the bench's CPU-baseline leg may import
this package; the CUDA library and its Python binding never do.

``attn_oracle.c`` holds the arithmetic; this file compiles it with gcc on
first use, marshals numpy arrays through ctypes, and builds the oracle's own
paged layout ``[num_pages][page_size][Hkv][d]`` from logical K/V.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "attn_oracle.c")
_LIB = os.path.join(_HERE, "liboracle_attn.so")
_lib = None

_I32P = ctypes.POINTER(ctypes.c_int32)
_U16P = ctypes.POINTER(ctypes.c_uint16)
_F64P = ctypes.POINTER(ctypes.c_double)
_U8P = ctypes.POINTER(ctypes.c_uint8)
_F32P = ctypes.POINTER(ctypes.c_float)


def build(force: bool = False) -> str:
    """Compile attn_oracle.c into a shared library next to it (gcc, OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.oracle_attn_rows.restype = ctypes.c_int
        lib.oracle_attn_rows.argtypes = [
            _U16P, _U16P, _U16P, ctypes.c_int64, _I32P, ctypes.c_int32, _I32P, _I32P, ctypes.c_int32,
            ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
            _I32P, _I32P, ctypes.c_int64, _F64P, _F64P,
        ]
        lib.oracle_attn_paged.restype = ctypes.c_int
        lib.oracle_attn_paged.argtypes = [
            _U16P, _U16P, _U16P, ctypes.c_int64, _I32P, ctypes.c_int32, _I32P, _I32P, ctypes.c_int32,
            ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, _F64P, _F64P,
        ]
        lib.oracle_attn_rows_fp8.restype = ctypes.c_int
        lib.oracle_attn_rows_fp8.argtypes = [
            _U16P, _U8P, _U8P, _F32P, _F32P, _F64P, ctypes.c_int64, _I32P, ctypes.c_int32, _I32P, _I32P, ctypes.c_int32,
            ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
            _I32P, _I32P, ctypes.c_int64, _F64P, _F64P,
        ]
        lib.oracle_kv_gather.restype = ctypes.c_int
        lib.oracle_kv_gather.argtypes = [
            _U16P, ctypes.c_int64, _I32P, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, _U16P,
        ]
        lib.oracle_lse_merge.restype = ctypes.c_int
        lib.oracle_lse_merge.argtypes = [_F64P, _F64P, ctypes.c_int32, ctypes.c_int32, _F64P, _F64P]
        lib.oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def _p(a, ptype):
    return a.ctypes.data_as(ptype)


def attn_rows(q, k_pool, v_pool, block_table, prior, q_len, n_q_heads, n_kv_heads, head_dim, page_size,
              row_req, row_tok):
    """Oracle attention for selected rows.  Returns (out [R,Hq,d], lse [R,Hq]) float64."""
    lib = _load()
    q = _c(q, np.uint16)
    k_pool = _c(k_pool, np.uint16)
    v_pool = _c(v_pool, np.uint16)
    block_table = _c(block_table, np.int32)
    prior = _c(prior, np.int32)
    q_len = _c(q_len, np.int32)
    row_req = _c(row_req, np.int32)
    row_tok = _c(row_tok, np.int32)
    n = prior.shape[0]
    assert q.shape == (int(q_len.sum()), n_q_heads, head_dim), q.shape
    assert k_pool.shape[1:] == (page_size, n_kv_heads, head_dim), k_pool.shape
    assert v_pool.shape == k_pool.shape
    assert block_table.ndim == 2 and block_table.shape[0] == n
    R = row_req.shape[0]
    out = np.empty((R, n_q_heads, head_dim), dtype=np.float64)
    lse = np.empty((R, n_q_heads), dtype=np.float64)
    rc = lib.oracle_attn_rows(
        _p(q, _U16P), _p(k_pool, _U16P), _p(v_pool, _U16P), k_pool.shape[0],
        _p(block_table, _I32P), block_table.shape[1], _p(prior, _I32P), _p(q_len, _I32P), n,
        n_q_heads, n_kv_heads, head_dim, page_size, _p(row_req, _I32P), _p(row_tok, _I32P), R,
        _p(out, _F64P), _p(lse, _F64P),
    )
    if rc != 0:
        raise ValueError("oracle_attn_rows failed with code %d" % rc)
    return out, lse


def attn_rows_fp8(q, k_codes, v_codes, k_scale, v_scale, block_table, prior, q_len, n_q_heads, n_kv_heads, head_dim,
                  page_size, row_req, row_tok):
    """Oracle attention over an FP8 (E4M3) cache: codes uint8 [pages, page, Hkv, d], scales float32 [pages, page, Hkv]
    (see ``oracle.fp8``).  Returns (out [R,Hq,d], lse [R,Hq]) float64."""
    from . import fp8

    lib = _load()
    q = _c(q, np.uint16)
    k_codes = _c(k_codes, np.uint8)
    v_codes = _c(v_codes, np.uint8)
    k_scale = _c(k_scale, np.float32)
    v_scale = _c(v_scale, np.float32)
    block_table = _c(block_table, np.int32)
    prior = _c(prior, np.int32)
    q_len = _c(q_len, np.int32)
    row_req = _c(row_req, np.int32)
    row_tok = _c(row_tok, np.int32)
    table = _c(fp8.decode_table(), np.float64)
    n = prior.shape[0]
    assert q.shape == (int(q_len.sum()), n_q_heads, head_dim), q.shape
    assert k_codes.shape[1:] == (page_size, n_kv_heads, head_dim) and v_codes.shape == k_codes.shape
    assert k_scale.shape == k_codes.shape[:3] and v_scale.shape == k_scale.shape
    R = row_req.shape[0]
    out = np.empty((R, n_q_heads, head_dim), dtype=np.float64)
    lse = np.empty((R, n_q_heads), dtype=np.float64)
    rc = lib.oracle_attn_rows_fp8(
        _p(q, _U16P), _p(k_codes, _U8P), _p(v_codes, _U8P), _p(k_scale, _F32P), _p(v_scale, _F32P), _p(table, _F64P),
        k_codes.shape[0], _p(block_table, _I32P), block_table.shape[1], _p(prior, _I32P), _p(q_len, _I32P), n,
        n_q_heads, n_kv_heads, head_dim, page_size, _p(row_req, _I32P), _p(row_tok, _I32P), R,
        _p(out, _F64P), _p(lse, _F64P),
    )
    if rc != 0:
        raise ValueError("oracle_attn_rows_fp8 failed with code %d" % rc)
    return out, lse


def plain_pool_fp8(kv_bits_per_request, block_table, num_pages, page_size):
    """Quantise logical bf16 tensors (uint16 [kv_len_r, Hkv, d] each) token by token and lay them out in the oracle's
    paged form: (codes uint8 [pages, page, Hkv, d], scales float32 [pages, page, Hkv]).  Slots nobody references hold
    the E4M3 NaN code and a NaN scale."""
    from . import fp8

    hkv, d = kv_bits_per_request[0].shape[1:]
    codes = np.full((num_pages, page_size, hkv, d), 0x7F, dtype=np.uint8)
    scales = np.full((num_pages, page_size, hkv), np.nan, dtype=np.float32)
    for r, x in enumerate(kv_bits_per_request):
        c, s = fp8.quantise(x)
        L = x.shape[0]
        for pi in range((L + page_size - 1) // page_size):
            lo = pi * page_size
            hi = min(L, lo + page_size)
            codes[int(block_table[r, pi]), : hi - lo] = c[lo:hi]
            scales[int(block_table[r, pi]), : hi - lo] = s[lo:hi]
    return codes, scales


def attn_paged(q, k_pool, v_pool, block_table, prior, q_len, n_q_heads, n_kv_heads, head_dim, page_size):
    """Oracle attention for every row of the batch: (out [T,Hq,d], lse [T,Hq]) float64."""
    lib = _load()
    q = _c(q, np.uint16)
    k_pool = _c(k_pool, np.uint16)
    v_pool = _c(v_pool, np.uint16)
    block_table = _c(block_table, np.int32)
    prior = _c(prior, np.int32)
    q_len = _c(q_len, np.int32)
    n = prior.shape[0]
    T = int(q_len.sum())
    assert q.shape == (T, n_q_heads, head_dim), q.shape
    assert k_pool.shape[1:] == (page_size, n_kv_heads, head_dim), k_pool.shape
    assert v_pool.shape == k_pool.shape
    assert block_table.ndim == 2 and block_table.shape[0] == n
    out = np.empty((T, n_q_heads, head_dim), dtype=np.float64)
    lse = np.empty((T, n_q_heads), dtype=np.float64)
    rc = lib.oracle_attn_paged(
        _p(q, _U16P), _p(k_pool, _U16P), _p(v_pool, _U16P), k_pool.shape[0],
        _p(block_table, _I32P), block_table.shape[1], _p(prior, _I32P), _p(q_len, _I32P), n,
        n_q_heads, n_kv_heads, head_dim, page_size, _p(out, _F64P), _p(lse, _F64P),
    )
    if rc != 0:
        raise ValueError("oracle_attn_paged failed with code %d" % rc)
    return out, lse


def kv_gather(pool, block_table_row, length):
    """Contiguous [length, Hkv, d] copy of a sequence's tokens from the oracle's paged pool."""
    lib = _load()
    pool = _c(pool, np.uint16)
    row = _c(block_table_row, np.int32)
    _, page_size, hkv, d = pool.shape
    dst = np.empty((length, hkv, d), dtype=np.uint16)
    rc = lib.oracle_kv_gather(_p(pool, _U16P), pool.shape[0], _p(row, _I32P), length, hkv, d, page_size,
                              _p(dst, _U16P))
    if rc != 0:
        raise ValueError("oracle_kv_gather failed with code %d" % rc)
    return dst


def lse_merge(o_parts, lse_parts):
    """Merge partial results over disjoint key subsets: o_parts [S,d], lse_parts [S]."""
    lib = _load()
    o = _c(o_parts, np.float64)
    l = _c(lse_parts, np.float64)
    S, d = o.shape
    out = np.empty(d, dtype=np.float64)
    lo = np.empty(1, dtype=np.float64)
    rc = lib.oracle_lse_merge(_p(o, _F64P), _p(l, _F64P), S, d, _p(out, _F64P), _p(lo, _F64P))
    if rc != 0:
        raise ValueError("oracle_lse_merge failed with code %d" % rc)
    return out, float(lo[0])


BF16_NAN = np.uint16(0x7FC1)


def plain_pool(kv_per_request, block_table, num_pages, page_size, poison=True):
    """Build the oracle's paged pool from logical tensors.

    ``kv_per_request[r]`` is a uint16 array [kv_len_r, Hkv, d].  Pages nobody
    references and tail slots past a sequence's length hold a bf16 NaN when
    ``poison`` is set, so any read of a wrong page or slot shows in the output.
    """
    hkv, d = kv_per_request[0].shape[1:]
    pool = np.full((num_pages, page_size, hkv, d), BF16_NAN if poison else 0, dtype=np.uint16)
    for r, x in enumerate(kv_per_request):
        L = x.shape[0]
        for pi in range((L + page_size - 1) // page_size):
            lo = pi * page_size
            hi = min(L, lo + page_size)
            pool[int(block_table[r, pi]), : hi - lo] = x[lo:hi]
    return pool
