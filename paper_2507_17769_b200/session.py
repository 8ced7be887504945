"""PagedAttention: pool + plan + workspace of one serving instance.

torch supplies device memory and the current stream; every computation is a
call through the C ABI.
"""
from __future__ import annotations

import numpy as np

from . import binding as B


class PagedAttention:
    """A paged K/V pool with the per-iteration plan / run cycle.

    >>> pa = PagedAttention(32, 8, 128, num_pages)
    >>> pa.write(k_new, v_new, block_table_dev, prior, q_len)   # cache the new tokens
    >>> pa.plan(prior, q_len, max_pages)                        # host partition
    >>> out, lse = pa.run(q, block_table_dev)                   # attention
    """

    def __init__(self, n_q_heads, n_kv_heads, head_dim, num_pages, page_size=16, device="cuda", poison=False, kv_dtype=0):
        """``kv_dtype``: 0 = bf16 cache, 1 = FP8 (E4M3) cache with a scale per (token, kv head); see ps_shape."""
        import torch

        self.torch = torch
        self.device = torch.device(device)
        self.shape = B.make_shape(n_q_heads, n_kv_heads, head_dim, page_size, kv_dtype)
        self.num_pages = int(num_pages)
        nbytes = B.ps_kv_bytes(self.shape, self.num_pages)
        # 0xFF bytes are bf16 NaN: any read of a slot nobody wrote shows in the output
        if poison:
            self.pool = torch.full((nbytes + 1024,), 0xFF, dtype=torch.uint8, device=self.device)
        else:
            self.pool = torch.empty((nbytes + 1024,), dtype=torch.uint8, device=self.device)
        base = (self.pool.data_ptr() + 1023) // 1024 * 1024  # the pool must start on a 1024-byte boundary
        self.kv = B.ps_kv_alloc(self.shape, self.num_pages, base, nbytes)
        self._plan = None
        self._ws = None
        self._ws_bytes = 0
        self._total_q = 0

    def close(self):
        if self._plan is not None:
            B.ps_plan_free(self._plan)
            self._plan = None
        if self.kv is not None:
            B.ps_kv_free(self.kv)
            self.kv = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _stream(self):
        return self.torch.cuda.current_stream(self.device).cuda_stream

    def write(self, k_new, v_new, block_table_dev, prior, q_len, max_pages=None):
        """Scatter new tokens' K, V (bf16 [T, Hkv, d]) into their pages."""
        if max_pages is None:
            max_pages = block_table_dev.shape[-1]
        assert k_new.is_contiguous() and v_new.is_contiguous() and block_table_dev.is_contiguous()
        B.ps_kv_write(self.kv, k_new, v_new, block_table_dev, int(max_pages), prior, q_len, self._stream())

    def gather_fp8(self, block_table_row_dev, length):
        """FP8 cache: logical tokens [0, length) of one sequence as (K codes, V codes) uint8 [length, Hkv, d] and
        (K scales, V scales) float32 [length, Hkv]."""
        t = self.torch
        kc = t.empty((length, self.shape.n_kv_heads, self.shape.head_dim), dtype=t.uint8, device=self.device)
        vc = t.empty_like(kc)
        ks = t.empty((length, self.shape.n_kv_heads), dtype=t.float32, device=self.device)
        vs = t.empty_like(ks)
        B.ps_kv_gather_fp8(self.kv, block_table_row_dev, int(length), kc, vc, ks, vs, self._stream())
        return kc, vc, ks, vs

    def gather(self, block_table_row_dev, length):
        """Logical tokens [0, length) of one sequence as contiguous (K, V) bf16 [length, Hkv, d] (bf16 cache)."""
        t = self.torch
        assert self.shape.dtype == 0, "use gather_fp8 on an FP8 cache"
        k = t.empty((length, self.shape.n_kv_heads, self.shape.head_dim), dtype=t.bfloat16, device=self.device)
        v = t.empty_like(k)
        B.ps_kv_gather(self.kv, block_table_row_dev, int(length), k, v, self._stream())
        return k, v

    def check_pool(self):
        B.ps_kv_status(self.kv, self._stream())

    def plan(self, prior, q_len, max_pages, opts=None):
        """Partition the batch; grows the workspace if the plan needs more."""
        self._plan, need = B.ps_attn_plan(self.shape, prior, q_len, int(max_pages), opts, self._plan)
        if need > self._ws_bytes:
            self._ws = self.torch.empty(int(need * 1.25) + 256, dtype=self.torch.uint8, device=self.device)
            self._ws_bytes = self._ws.numel()
        self._total_q = int(np.asarray(q_len).sum())
        return B.ps_plan_get_info(self._plan)

    def items(self):
        return B.ps_plan_get_items(self._plan)

    def run(self, q, block_table_dev, out=None, lse=None, want_lse=True):
        """Attention for the planned batch.  q: bf16 [T, Hq, d].  Returns (out, lse)."""
        t = self.torch
        assert self._plan is not None, "call plan() first"
        assert q.is_contiguous() and q.shape[0] == self._total_q and block_table_dev.is_contiguous()
        if out is None:
            out = t.empty_like(q)
        if lse is None and want_lse:
            lse = t.empty((q.shape[0], self.shape.n_q_heads), dtype=t.float32, device=self.device)
        B.ps_attn_run(self._plan, self.kv, q, block_table_dev, out, lse, self._ws, self._ws_bytes, self._stream())
        return out, lse

    def check(self):
        """Synchronise and raise if the last run saw a device-side error."""
        B.ps_plan_status(self._plan, self._stream())
