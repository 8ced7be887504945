"""Seeded synthetic inputs for mixed-batch paged-KV attention.

This module only *draws inputs*: bf16 bit patterns for Q/K/V, request lengths,
and block tables.  It holds none of the attention arithmetic and is the one
piece of code shared by the CPU oracle's tests and the CUDA path's tests.

Every value is a pure function of (seed, tensor id, sequence id, logical
index), so a tensor can be regenerated piecewise (one sequence, one token
range) on the host, or by the integer-only CUDA twin in ``gen_cuda.cu``, with
bit-identical results.  Values are indexed by *logical* coordinates
(sequence, token position, head, dim): permuting physical pages never changes
the content a request sees.

The counter-based generator is SplitMix64 (Steele, Lea, Flood 2014): the
k-th draw (k = 0, 1, ...) of a stream with key ``s`` is the published
finaliser applied to ``s + (k + 1) * gamma`` (gamma = the golden-ratio
increment), i.e. exactly the k-th output of SplitMix64 seeded with ``s``,
reachable at any k without stepping.  Normal
deviates come from the top 16 bits through a 65 536-entry table of the inverse
normal CDF at the bin mid-points, rounded to bf16 (round-to-nearest-even).

The batches stand in for the serving traces the paper samples (Table 1), which
are not redistributable here: lengths follow the laws listed per config in
``CONFIGS`` below; Q/K/V are N(0,1) in bf16.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np

U64 = np.uint64
_GAMMA = U64(0x9E3779B97F4A7C15)
_M1 = U64(0xBF58476D1CE4E5B9)
_M2 = U64(0x94D049BB133111EB)

TENSOR_Q, TENSOR_K, TENSOR_V = 1, 2, 3
STREAM_LEN, STREAM_PERM, STREAM_PRIOR = 11, 12, 13


def _finalise(z) -> np.ndarray:
    with np.errstate(over="ignore"):
        z = np.asarray(z, dtype=U64)
        z = (z ^ (z >> U64(30))) * _M1
        z = (z ^ (z >> U64(27))) * _M2
        return z ^ (z >> U64(31))


def mix64(x) -> np.ndarray:
    """First SplitMix64 output for state ``x``: finalise(x + gamma)."""
    with np.errstate(over="ignore"):
        return _finalise(np.asarray(x, dtype=U64) + _GAMMA)


def stream_key(seed: int, tensor_id: int, seq: int = 0) -> int:
    """Key of the stream (seed, tensor id, sequence id); a Python int < 2**64."""
    k = int(mix64(U64(seed & 0xFFFFFFFFFFFFFFFF))) ^ (tensor_id & 0xFFFFFFFFFFFFFFFF)
    k = int(mix64(U64(k))) ^ (seq & 0xFFFFFFFFFFFFFFFF)
    return int(mix64(U64(k)))


def raw_bits(key: int, idx0: int, count: int) -> np.ndarray:
    """``count`` consecutive 64-bit draws of stream ``key`` starting at counter ``idx0``."""
    with np.errstate(over="ignore"):
        ctr = U64(key) + (np.arange(count, dtype=U64) + U64(idx0 + 1)) * _GAMMA
    return _finalise(ctr)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest even); returns uint16 bit patterns."""
    u = np.asarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns exactly to float64."""
    u = np.asarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


_TABLE = None


def normal_table() -> np.ndarray:
    """65 536 bf16 bit patterns: inverse normal CDF at (k + 0.5) / 65536."""
    global _TABLE
    if _TABLE is None:
        from scipy.special import ndtri

        p = (np.arange(65536, dtype=np.float64) + 0.5) / 65536.0
        _TABLE = f32_to_bf16_bits(ndtri(p).astype(np.float32))
    return _TABLE


def normal_bf16(key: int, idx0: int, count: int) -> np.ndarray:
    """``count`` N(0,1) bf16 bit patterns of stream ``key`` from counter ``idx0``."""
    top = (raw_bits(key, idx0, count) >> U64(48)).astype(np.int64)
    return normal_table()[top]


def uniform_int(key: int, idx0: int, count: int, lo: int, hi: int) -> np.ndarray:
    """Integers uniform on [lo, hi] inclusive (multiply-shift on the top 32 bits)."""
    r = (raw_bits(key, idx0, count) >> U64(32)).astype(np.uint64)
    span = U64(hi - lo + 1)
    return (lo + ((r * span) >> U64(32)).astype(np.int64)).astype(np.int64)


def std_normal_f64(key: int, idx0: int, count: int) -> np.ndarray:
    """N(0,1) in float64 from the top 53 bits (lengths only, host side)."""
    from scipy.special import ndtri

    u = ((raw_bits(key, idx0, count) >> U64(11)).astype(np.float64) + 0.5) / float(1 << 53)
    return ndtri(u)


def permutation(key: int, n: int) -> np.ndarray:
    """Seeded permutation of range(n): stable argsort of n keyed draws."""
    return np.argsort(raw_bits(key, 0, n), kind="stable").astype(np.int64)


# ---------------------------------------------------------------------------
# tensors, addressed by logical coordinates
# ---------------------------------------------------------------------------

def gen_kv(seed: int, seq: int, tok0: int, tok1: int, n_kv_heads: int, head_dim: int):
    """K and V bit patterns of sequence ``seq`` for token positions [tok0, tok1).

    Returns two uint16 arrays of shape [tok1 - tok0, n_kv_heads, head_dim].
    """
    per_tok = n_kv_heads * head_dim
    n = (tok1 - tok0) * per_tok
    shape = (tok1 - tok0, n_kv_heads, head_dim)
    k = normal_bf16(stream_key(seed, TENSOR_K, seq), tok0 * per_tok, n).reshape(shape)
    v = normal_bf16(stream_key(seed, TENSOR_V, seq), tok0 * per_tok, n).reshape(shape)
    return k, v


def gen_q(seed: int, seq: int, pos0: int, pos1: int, n_q_heads: int, head_dim: int) -> np.ndarray:
    """Q bit patterns of sequence ``seq`` for absolute token positions [pos0, pos1)."""
    per_tok = n_q_heads * head_dim
    n = (pos1 - pos0) * per_tok
    return normal_bf16(stream_key(seed, TENSOR_Q, seq), pos0 * per_tok, n).reshape(
        pos1 - pos0, n_q_heads, head_dim
    )


# ---------------------------------------------------------------------------
# batches
# ---------------------------------------------------------------------------

@dataclasses.dataclass
class Shape:
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    page_size: int = 16

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def kv_token_bytes(self) -> int:
        """Bytes of K plus V of one token over all kv heads (bf16)."""
        return 2 * self.n_kv_heads * self.head_dim * 2


@dataclasses.dataclass
class Batch:
    """One serving iteration: request r has ``prior[r]`` cached tokens and
    ``q_len[r]`` new tokens; all ``prior + q_len`` tokens' K,V sit in pages
    ``block_table[r, :ceil(kv_len/page)]`` of a pool of ``num_pages`` pages."""

    shape: Shape
    seed: int
    prior: np.ndarray  # int32 [n]
    q_len: np.ndarray  # int32 [n]
    block_table: np.ndarray  # int32 [n, max_pages], unused entries -1
    num_pages: int

    @property
    def n(self) -> int:
        return int(self.prior.shape[0])

    @property
    def kv_len(self) -> np.ndarray:
        return (self.prior + self.q_len).astype(np.int32)

    @property
    def total_q(self) -> int:
        return int(self.q_len.sum())

    @property
    def max_pages(self) -> int:
        return int(self.block_table.shape[1])

    @property
    def q_start(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum(self.q_len)[:-1]]).astype(np.int64)

    def q_bits(self) -> np.ndarray:
        """Packed Q [total_q, Hq, d]: requests in batch order, tokens in order."""
        s = self.shape
        parts = [
            gen_q(self.seed, r, int(self.prior[r]), int(self.prior[r] + self.q_len[r]), s.n_q_heads, s.head_dim)
            for r in range(self.n)
        ]
        return np.concatenate(parts, axis=0)

    def kv_bits(self, r: int):
        """Logical K, V of request r: uint16 [kv_len[r], Hkv, d] each."""
        s = self.shape
        return gen_kv(self.seed, r, 0, int(self.kv_len[r]), s.n_kv_heads, s.head_dim)

    def decode_kv_tokens(self) -> int:
        return int(self.kv_len[self.q_len == 1].sum())

    def decode_bytes(self) -> int:
        """Algorithmic KV bytes streamed by the decode rows (kv_len x K+V bytes per token)."""
        return self.decode_kv_tokens() * self.shape.kv_token_bytes

    def prefill_flops(self) -> int:
        """Algorithmic flops of the prefill rows: 4 d Hq (c prior + c (c + 1) / 2) per chunk."""
        s = self.shape
        phi = 4 * s.head_dim * s.n_q_heads
        tot = 0
        for p, c in zip(self.prior.tolist(), self.q_len.tolist()):
            if c > 1:
                tot += phi * (c * p + c * (c + 1) // 2)
        return tot


def assign_pages(seed: int, kv_len: np.ndarray, page_size: int, spare: float = 0.25):
    """Block table from a seeded permutation of a pool with ``spare`` extra pages.

    Pool = ceil((1 + spare) * pages needed), at least 8 more than needed.
    Request r takes the next ceil(kv_len[r] / page_size) entries of the
    permutation.  Unused block-table entries are -1.
    """
    need = (np.asarray(kv_len, dtype=np.int64) + page_size - 1) // page_size
    total = int(need.sum())
    num_pages = max(int(math.ceil(total * (1.0 + spare))), total + 8)
    perm = permutation(stream_key(seed, STREAM_PERM), num_pages)
    max_pages = int(need.max()) if len(need) else 0
    bt = np.full((len(need), max_pages), -1, dtype=np.int32)
    off = 0
    for r, c in enumerate(need.tolist()):
        bt[r, :c] = perm[off : off + c]
        off += c
    return bt, num_pages


def make_batch(shape: Shape, seed: int, prior, q_len, spare: float = 0.25) -> Batch:
    prior = np.asarray(prior, dtype=np.int32)
    q_len = np.asarray(q_len, dtype=np.int32)
    bt, num_pages = assign_pages(seed, prior + q_len, shape.page_size, spare)
    return Batch(shape, seed, prior, q_len, bt, num_pages)


SHAPE_TINY = Shape(4, 2, 64, 16)
SHAPE_8B = Shape(32, 8, 128, 16)
SHAPE_LARGE = Shape(64, 8, 128, 16)

GRID_CHUNKS = (64, 128, 256, 512, 1024, 2048)
GRID_DECODES = (8, 32, 128, 256)
GRID_MEAN_CTX = (512, 2048, 8192)
GRID_SEEDS = 27


def config0(seed: int = 1000) -> Batch:
    """Tiny mixed batch: 4 decode rows with contexts {17,33,64,100} (context
    counts the current token) and one 32-token chunk on 48 prior tokens."""
    return make_batch(SHAPE_TINY, seed, [16, 32, 63, 99, 48], [1, 1, 1, 1, 32])


def config1(seed: int = 1001) -> Batch:
    """Decode-only, 8B-class GQA shape: 64 rows, context uniform on [512, 4096]."""
    ctx = uniform_int(stream_key(seed, STREAM_LEN), 0, 64, 512, 4096)
    return make_batch(SHAPE_8B, seed, ctx - 1, np.ones(64, dtype=np.int32))


def config2(seed: int = 1002) -> Batch:
    """Dynamic-chunking mixed batch under a 2048-token budget: 512 decode rows
    with lognormal contexts (median 1024, sigma 1, clipped to [16, 16384]) and
    one 1536-token chunk on a prior context uniform on [0, 8192]."""
    z = std_normal_f64(stream_key(seed, STREAM_LEN), 0, 512)
    ctx = np.clip(np.rint(np.exp(math.log(1024.0) + z)), 16, 16384).astype(np.int64)
    pr = int(uniform_int(stream_key(seed, STREAM_PRIOR), 0, 1, 0, 8192)[0])
    prior = np.concatenate([ctx - 1, [pr]])
    q_len = np.concatenate([np.ones(512, dtype=np.int64), [1536]])
    return make_batch(SHAPE_8B, seed, prior, q_len)


def grid_seed(cell: int, s: int) -> int:
    return 3000 + GRID_SEEDS * cell + s


def grid_cells():
    """(cell index, chunk, decode count, mean context) in sweep order."""
    out = []
    for chunk in GRID_CHUNKS:
        for nd in GRID_DECODES:
            for m in GRID_MEAN_CTX:
                out.append((len(out), chunk, nd, m))
    return out


def config3_cell(chunk: int, n_decode: int, mean_ctx: int, seed: int) -> Batch:
    """One cell of the latency-table sweep: decode contexts uniform on
    [mean/2, 3 mean/2]; the chunk's prior context is one more draw of that law."""
    lo, hi = mean_ctx // 2, (3 * mean_ctx) // 2
    ctx = uniform_int(stream_key(seed, STREAM_LEN), 0, n_decode, lo, hi)
    pr = int(uniform_int(stream_key(seed, STREAM_PRIOR), 0, 1, lo, hi)[0])
    prior = np.concatenate([ctx - 1, [pr]])
    q_len = np.concatenate([np.ones(n_decode, dtype=np.int64), [chunk]])
    return make_batch(SHAPE_8B, seed, prior, q_len)


def config4(seed: int = 1004) -> Batch:
    """Large-model long-context mixed batch: 256 decode rows with contexts
    uniform on [4096, 32768] and two 2048-token chunks on prior contexts
    uniform on [16384, 30000]."""
    ctx = uniform_int(stream_key(seed, STREAM_LEN), 0, 256, 4096, 32768)
    pr = uniform_int(stream_key(seed, STREAM_PRIOR), 0, 2, 16384, 30000)
    prior = np.concatenate([ctx - 1, pr])
    q_len = np.concatenate([np.ones(256, dtype=np.int64), [2048, 2048]])
    return make_batch(SHAPE_LARGE, seed, prior, q_len)


CONFIGS = {0: config0, 1: config1, 2: config2, 4: config4}
