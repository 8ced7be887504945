"""Writes tests/golden/config0_oracle.txt: the CPU oracle's result for the tiny mixed batch (4 decode rows with
contexts 17, 33, 64, 100 and one 32-token chunk on 48 prior tokens; 4 q heads / 2 kv heads, head_dim 64).
Calls only oracle/ and the seeded input generator.  Run from the repository root:

    python tests/golden/make_config0_oracle.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from workloads import gen  # noqa: E402

b = gen.config0()
s = b.shape
ks, vs = zip(*[b.kv_bits(r) for r in range(b.n)])
kp = oracle.plain_pool(ks, b.block_table, b.num_pages, s.page_size)
vp = oracle.plain_pool(vs, b.block_table, b.num_pages, s.page_size)
out, lse = oracle.attn_paged(b.q_bits(), kp, vp, b.block_table, b.prior, b.q_len, s.n_q_heads, s.n_kv_heads, s.head_dim,
                             s.page_size)
rows = np.concatenate([lse.reshape(-1, 1), out.reshape(-1, s.head_dim)[:, [0, 1, 2, 3, -1]]], axis=1)
path = os.path.join(ROOT, "tests", "golden", "config0_oracle.txt")
np.savetxt(path, rows, fmt="%.17g",
           header="oracle (fp64) for workloads.gen.config0(seed 1000): one line per (token, q head) in packed order: "
                  "lse out[0] out[1] out[2] out[3] out[63]")
print("wrote", path, rows.shape)
