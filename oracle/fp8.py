"""FP8 (e4m3) KV-cache quantisation for the oracle (test infrastructure).

The library's FP8 cache variant stores K and V as OCP FP8 E4M3 codes (1 sign,
4 exponent bits with bias 7, 3 mantissa bits; largest finite value 448; no
infinities; S.1111.111 is NaN) with one fp32 scale per (token, kv head) and
tensor:

    scale = amax / 448 rounded up to 8 significant bits (a bf16-representable fp32)
            amax = max |x| over the head_dim values (scale = 1 if amax = 0)
    code  = round_to_nearest_even_e4m3( x / scale ), saturating at +-448
    value = decode(code) * scale

(The scale keeps 8 significant bits so that a softmax weight of exactly 1 times
the scale is still exact in a 16-bit matrix operand; rounding up keeps
|x| / scale <= 448.)

The paper states no precision; this format is this repository's reading.  The
divisions are IEEE fp32 (both sides take the rounding decision in that
precision); decode(code) * scale is evaluated exactly (fp64 holds the 4 + 24
significant bits).  The attention arithmetic over the dequantised values stays
the plain fp64 definition (``attn_oracle.c``).

Pins (tests/test_oracle_fp8_pins.py): every code round-trips; the encoder equals a
brute-force nearest-value search with ties to the even code; saturation;
scale = amax / 448; lossless data gives the bf16 oracle's result.
"""
from __future__ import annotations

import numpy as np

E4M3_MAX = 448.0


def decode_table() -> np.ndarray:
    """The 256 values of the E4M3 codes as float64 (NaN for S.1111.111)."""
    out = np.empty(256, dtype=np.float64)
    for c in range(256):
        s = -1.0 if c & 0x80 else 1.0
        e = (c >> 3) & 0xF
        m = c & 0x7
        if e == 0xF and m == 0x7:
            out[c] = np.nan
        elif e == 0:
            out[c] = s * m * 2.0 ** -9          # subnormal: m / 8 * 2^-6
        else:
            out[c] = s * (1.0 + m / 8.0) * 2.0 ** (e - 7)
    return out


_TABLE = decode_table()


def encode(y) -> np.ndarray:
    """fp32 -> E4M3 code, round to nearest even, saturating to +-448 (NaN stays NaN)."""
    y = np.asarray(y, dtype=np.float32)
    a = np.abs(y).astype(np.float64)
    a = np.minimum(a, E4M3_MAX)
    code = np.zeros(y.shape, dtype=np.uint8)
    # spacing of the E4M3 grid at |y|: 2^-9 below 2^-6 (subnormals), else 2^(floor(log2 a) - 3)
    with np.errstate(divide="ignore"):
        ex = np.floor(np.log2(np.where(a > 0, a, 1.0)))
    ex = np.clip(ex, -6, 8)
    step = 2.0 ** (ex - 3)
    q = np.rint(a / step)  # numpy rounds half to even; a / step is exact (power-of-two divisor)
    v = q * step           # a grid value, possibly the next binade's first one
    # value -> code
    with np.errstate(divide="ignore"):
        ev = np.floor(np.log2(np.where(v > 0, v, 1.0)))
    sub = v < 2.0 ** -6
    e_field = np.where(sub, 0, ev + 7).astype(np.int64)
    m_field = np.where(sub, np.rint(v * 2.0 ** 9), np.rint((v / 2.0 ** ev - 1.0) * 8.0)).astype(np.int64)
    code = (e_field << 3 | m_field).astype(np.uint8)
    code = np.where(np.signbit(y), code | 0x80, code).astype(np.uint8)
    code = np.where(np.isnan(y), np.uint8(0x7F), code).astype(np.uint8)
    return code


def quantise(x_bits: np.ndarray):
    """bf16 bit patterns [..., d] -> (codes uint8 [..., d], scales float32 [...])."""
    u = np.asarray(x_bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    x = u.view(np.float32)
    amax = np.max(np.abs(x), axis=-1)
    scale = np.where(amax > 0, amax / np.float32(E4M3_MAX), np.float32(1.0)).astype(np.float32)
    u = scale.view(np.uint32)
    u = np.where((u & np.uint32(0xFFFF)) != 0, (u | np.uint32(0xFFFF)) + np.uint32(1), u).astype(np.uint32)  # round up to bf16 precision
    scale = u.view(np.float32)
    y = (x / scale[..., None]).astype(np.float32)  # IEEE fp32 division
    return encode(y), scale


def dequantise(codes: np.ndarray, scale: np.ndarray) -> np.ndarray:
    """codes [..., d], scales [...] -> float64 values, exact."""
    return _TABLE[np.asarray(codes, dtype=np.uint8)] * np.asarray(scale, dtype=np.float64)[..., None]
