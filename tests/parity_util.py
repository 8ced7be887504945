"""Helpers shared by the GPU parity tests: oracle inputs for a batch (or a
subset of its requests) and the comparison with the tolerance the target
states: max-abs <= 1e-2 and mean-abs <= 1e-3 on bf16 outputs."""
import numpy as np

import oracle
from workloads import gen

MAX_ABS = 1e-2
MEAN_ABS = 1e-3
LSE_ABS = 2e-3


def _bits(t):
    import torch

    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def kv_bits(batch, r):
    """Logical K, V bit patterns of request r for the oracle.  With a CUDA device they are drawn by the input
    generator's device twin (bit-identical to the numpy generator, which takes minutes on the large configs) and
    copied back; they never pass through the attention library."""
    s = batch.shape
    try:
        import torch

        if torch.cuda.is_available():
            from workloads import gen_cuda

            k, v = gen_cuda.gen_kv(batch.seed, r, 0, int(batch.kv_len[r]), s.n_kv_heads, s.head_dim)
            return _bits(k), _bits(v)
    except ImportError:
        pass
    return batch.kv_bits(r)


def q_bits(batch, r):
    s = batch.shape
    lo, hi = int(batch.prior[r]), int(batch.prior[r] + batch.q_len[r])
    try:
        import torch

        if torch.cuda.is_available():
            from workloads import gen_cuda

            return _bits(gen_cuda.gen_q(batch.seed, r, lo, hi, s.n_q_heads, s.head_dim))
    except ImportError:
        pass
    return gen.gen_q(batch.seed, r, lo, hi, s.n_q_heads, s.head_dim)


def oracle_subset(batch, reqs, rows=None, with_keys=False):
    """Oracle output for the given requests of ``batch``.

    ``rows``: optional dict request -> list of new-token indices; default all
    tokens.  Returns (out [R, Hq, d], lse [R, Hq], packed q-token indices [R])
    and, with ``with_keys``, the number of keys each of the R rows sees.
    """
    s = batch.shape
    reqs = list(reqs)
    ks, vs, qs = [], [], []
    for r in reqs:
        k, v = kv_bits(batch, r)
        ks.append(k)
        vs.append(v)
        qs.append(q_bits(batch, r))
    need = [(x.shape[0] + s.page_size - 1) // s.page_size for x in ks]
    bt = np.full((len(reqs), max(need)), -1, dtype=np.int32)
    off = 0
    for a, c in enumerate(need):
        bt[a, :c] = np.arange(off, off + c)
        off += c
    kp = oracle.plain_pool(ks, bt, off + 1, s.page_size)
    vp = oracle.plain_pool(vs, bt, off + 1, s.page_size)
    row_req, row_tok, packed, keys = [], [], [], []
    q_start = batch.q_start
    for a, r in enumerate(reqs):
        toks = range(int(batch.q_len[r])) if rows is None or r not in rows else rows[r]
        for i in toks:
            row_req.append(a)
            row_tok.append(i)
            packed.append(int(q_start[r]) + i)
            keys.append(int(batch.prior[r]) + i + 1)
    out, lse = oracle.attn_rows(np.concatenate(qs), kp, vp, bt, batch.prior[reqs], batch.q_len[reqs], s.n_q_heads,
                                s.n_kv_heads, s.head_dim, s.page_size, row_req, row_tok)
    if with_keys:
        return out, lse, np.asarray(packed), np.asarray(keys)
    return out, lse, np.asarray(packed)


FEW_KEYS = 8      # rows that see at most this many keys ...
LARGE_VALUE = 2.56  # ... and elements at least this large may exceed 1e-2 by bf16 rounding alone (2.56 * 2^-8 = 1e-2)


def compare(gpu_out, gpu_lse, want_out, want_lse, packed=None, what="", few_key_rows=False, keys=None):
    """gpu_out: torch bf16 [T, Hq, d] (device), gpu_lse: torch fp32 [T, Hq] or None.

    ``few_key_rows`` (with ``keys`` [R], the number of keys each compared row sees): for batches with rows that
    see a handful of keys.  Such a row's output is as large as a single V value (up to 4 and more for N(0,1) data),
    and a bf16 result cannot be closer to the exact one than half a unit in its last place, |x| 2^-8 at worst:
    0.016 at |x| = 4.1 however the kernel computes.  For the elements this can touch -- rows that see at most
    FEW_KEYS keys, and elements with |want| >= LARGE_VALUE anywhere -- the bound scales with the value:
    max(1e-2, |want| 2^-7) (the output's own rounding plus as much again for the bf16-rounded weights).  Every
    other element keeps the plain 1e-2; the mean bound is max(1e-3, mean|want| 2^-8).  Batches shaped like the
    target's configs are held to the plain 1e-2 / 1e-3 throughout."""
    got = gpu_out.float().cpu().numpy().astype(np.float64)
    if packed is not None:
        got = got[packed]
    assert np.all(np.isfinite(got)), "%s: non-finite output" % what
    err = np.abs(got - want_out)
    if few_key_rows:
        assert keys is not None and len(keys) == err.shape[0]
        scaled = (np.asarray(keys) <= FEW_KEYS)[:, None, None] | (np.abs(want_out) >= LARGE_VALUE)
        bound = np.where(scaled, np.maximum(MAX_ABS, np.abs(want_out) * 2.0 ** -7), MAX_ABS)
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


def oracle_in_groups(batch, reqs, rows=None, max_tokens=400_000):
    """oracle_subset over ``reqs`` in groups of at most ``max_tokens`` KV tokens, so that the host copies of a
    large config's K/V (config 4 holds 19 GB) never exist all at once.  Returns the concatenated results."""
    outs, lses, packs = [], [], []
    group, tokens = [], 0
    for r in list(reqs) + [None]:
        if r is not None and (not group or tokens + int(batch.kv_len[r]) <= max_tokens):
            group.append(r)
            tokens += int(batch.kv_len[r])
            continue
        if group:
            o, l, p = oracle_subset(batch, group, rows)
            outs.append(o)
            lses.append(l)
            packs.append(p)
        group, tokens = ([r], int(batch.kv_len[r])) if r is not None else ([], 0)
    return np.concatenate(outs), np.concatenate(lses), np.concatenate(packs)
