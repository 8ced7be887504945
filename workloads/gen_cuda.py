"""Device-side twin of :mod:`workloads.gen`'s bf16 normal streams.

Large configs hold tens of GB of K/V; drawing them on the host would take
minutes, so the same integer hash and table lookup run as a CUDA kernel and
give bit-identical tensors.  torch is used for device memory only.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

from . import gen

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen_cuda.cu")
_LIB = os.path.join(_HERE, "libpsgen.so")
_lib = None
_table = {}


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        nvcc = "/usr/local/cuda/bin/nvcc" if os.path.exists("/usr/local/cuda/bin/nvcc") else "nvcc"
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-Xcompiler", "-fPIC",
                               "-shared", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.psgen_normal_bf16.restype = ctypes.c_int
        lib.psgen_normal_bf16.argtypes = [ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint64, ctypes.c_uint64,
                                          ctypes.c_void_p, ctypes.c_void_p]
        _lib = lib
    return _lib


def _table_dev(device):
    import torch

    key = str(device)
    if key not in _table:
        _table[key] = torch.from_numpy(gen.normal_table().view(np.int16).copy()).to(device)
    return _table[key]


def normal_bf16_into(dst, key: int, idx0: int):
    """Fill the contiguous 2-byte-element tensor ``dst`` (bf16 or int16) with the stream's values."""
    import torch

    assert dst.is_cuda and dst.is_contiguous() and dst.element_size() == 2
    rc = _load().psgen_normal_bf16(dst.data_ptr(), key, idx0, dst.numel(), _table_dev(dst.device).data_ptr(),
                                   torch.cuda.current_stream(dst.device).cuda_stream)
    if rc != 0:
        raise RuntimeError("psgen_normal_bf16 failed with CUDA error %d" % rc)
    return dst


def gen_kv(seed: int, seq: int, tok0: int, tok1: int, n_kv_heads: int, head_dim: int, device="cuda"):
    """Device K, V (bf16 [tok1 - tok0, Hkv, d]); same bits as :func:`workloads.gen.gen_kv`."""
    import torch

    per_tok = n_kv_heads * head_dim
    k = torch.empty((tok1 - tok0, n_kv_heads, head_dim), dtype=torch.bfloat16, device=device)
    v = torch.empty_like(k)
    normal_bf16_into(k, gen.stream_key(seed, gen.TENSOR_K, seq), tok0 * per_tok)
    normal_bf16_into(v, gen.stream_key(seed, gen.TENSOR_V, seq), tok0 * per_tok)
    return k, v


def gen_q(seed: int, seq: int, pos0: int, pos1: int, n_q_heads: int, head_dim: int, device="cuda"):
    import torch

    q = torch.empty((pos1 - pos0, n_q_heads, head_dim), dtype=torch.bfloat16, device=device)
    return normal_bf16_into(q, gen.stream_key(seed, gen.TENSOR_Q, seq), pos0 * n_q_heads * head_dim)
