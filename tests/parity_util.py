"""Helpers shared by the GPU parity tests: oracle inputs for a batch (or a
subset of its requests) and the comparison with the tolerance the target
states: max-abs <= 1e-2 and mean-abs <= 1e-3 on bf16 outputs."""
import numpy as np

import oracle
from workloads import gen

MAX_ABS = 1e-2
MEAN_ABS = 1e-3
LSE_ABS = 2e-3


def oracle_subset(batch, reqs, rows=None):
    """Oracle output for the given requests of ``batch``.

    ``rows``: optional dict request -> list of new-token indices; default all
    tokens.  Returns (out [R, Hq, d], lse [R, Hq], packed q-token indices [R]).
    """
    s = batch.shape
    reqs = list(reqs)
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
    row_req, row_tok, packed = [], [], []
    q_start = batch.q_start
    for a, r in enumerate(reqs):
        toks = range(int(batch.q_len[r])) if rows is None or r not in rows else rows[r]
        for i in toks:
            row_req.append(a)
            row_tok.append(i)
            packed.append(int(q_start[r]) + i)
    out, lse = oracle.attn_rows(np.concatenate(qs), kp, vp, bt, batch.prior[reqs], batch.q_len[reqs], s.n_q_heads,
                                s.n_kv_heads, s.head_dim, s.page_size, row_req, row_tok)
    return out, lse, np.asarray(packed)


def compare(gpu_out, gpu_lse, want_out, want_lse, packed=None, what="", few_key_rows=False):
    """gpu_out: torch bf16 [T, Hq, d] (device), gpu_lse: torch fp32 [T, Hq] or None.

    ``few_key_rows``: for batches made mostly of rows that see one or two keys.  Such a row's output is as
    large as a single V value (up to 4 and more for N(0,1) data), and a bf16 result cannot be closer to the exact
    one than half a unit in its last place, |x| 2^-8 at worst: 0.016 at |x| = 4.1 however the kernel computes.
    The bounds then scale with the values: per element max(1e-2, |want| 2^-7) (the output's own rounding plus as
    much again for the bf16-rounded weights), and for the mean max(1e-3, mean|want| 2^-8).  Batches shaped like
    the target's configs average over many keys and are held to the plain 1e-2 / 1e-3."""
    got = gpu_out.float().cpu().numpy().astype(np.float64)
    if packed is not None:
        got = got[packed]
    assert np.all(np.isfinite(got)), "%s: non-finite output" % what
    err = np.abs(got - want_out)
    if few_key_rows:
        bound = np.maximum(MAX_ABS, np.abs(want_out) * 2.0 ** -7)
        worst = np.unravel_index(np.argmax(err - bound), err.shape)
        assert np.all(err <= bound), "%s: error %.3e at a value of %.4f" % (what, err[worst], want_out[worst])
        assert err.mean() <= max(MEAN_ABS, np.abs(want_out).mean() * 2.0 ** -8), "%s: mean-abs %.3e" % (what, err.mean())
    else:
        assert err.max() <= MAX_ABS, "%s: max-abs %.3e" % (what, err.max())
        assert err.mean() <= MEAN_ABS, "%s: mean-abs %.3e" % (what, err.mean())
    if gpu_lse is not None:
        gl = gpu_lse.cpu().numpy().astype(np.float64)
        if packed is not None:
            gl = gl[packed]
        lerr = np.abs(gl - want_lse)
        assert lerr.max() <= LSE_ABS, "%s: lse max-abs %.3e" % (what, lerr.max())
    return float(err.max()), float(err.mean())
