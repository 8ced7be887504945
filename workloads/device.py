"""Put a synthetic :class:`workloads.gen.Batch` on the GPU through the library's own write path."""
from __future__ import annotations

from . import gen, gen_cuda


class DeviceBatch:
    """Pool filled with the batch's K/V (drawn on the device, scattered with
    ``ps_kv_write``), its block table and packed Q as device tensors."""

    def __init__(self, batch: gen.Batch, poison: bool = True, device="cuda", kv_dtype: int = 0):
        import torch
        from paper_2507_17769_b200 import PagedAttention

        s = batch.shape
        self.batch = batch
        self.pa = PagedAttention(s.n_q_heads, s.n_kv_heads, s.head_dim, batch.num_pages, s.page_size, device, poison=poison,
                                 kv_dtype=kv_dtype)
        self.block_table = torch.from_numpy(batch.block_table).to(device)
        for r in range(batch.n):
            L = int(batch.kv_len[r])
            k, v = gen_cuda.gen_kv(batch.seed, r, 0, L, s.n_kv_heads, s.head_dim, device)
            self.pa.write(k, v, self.block_table[r], [0], [L], max_pages=batch.max_pages)
        qs = [gen_cuda.gen_q(batch.seed, r, int(batch.prior[r]), int(batch.prior[r] + batch.q_len[r]), s.n_q_heads,
                             s.head_dim, device) for r in range(batch.n)]
        self.q = torch.cat(qs, dim=0).contiguous()
        self.pa.check_pool()

    def plan(self, opts=None):
        return self.pa.plan(self.batch.prior, self.batch.q_len, self.batch.max_pages, opts)

    def run(self, **kw):
        return self.pa.run(self.q, self.block_table, **kw)
