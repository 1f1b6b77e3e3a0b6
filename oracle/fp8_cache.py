"""CPU oracle for the 8-bit K/V cache extension (NOT in the paper: a bandwidth extension of its decode path).

Test infrastructure only: imported by tests/, the smoke check and bench.py's CPU baseline, never by the product.

The cache holds K and V rows as 8-bit floating point in the OCP "E4M3" interchange format (1 sign bit, 4 exponent
bits with bias 7, 3 mantissa bits; no infinities; the all-ones exponent with all-ones mantissa is NaN; largest
finite value 448; subnormals are multiples of 2^-9), with one fp32 scale per head:  value = decode(byte) * scale[h].
A row enters the cache as  byte = encode(x / scale[h])  with the division in fp32, round to nearest (ties to the even
code), values beyond +-448 clamped to +-448.

Decode attention over such a cache is Eq. 6 of the paper on the DEQUANTISED rows: the current token is attended in
its own (unquantised) precision, kept or not, and, if kept, appended in quantised form.
Everything is written out from the format's definition in fp64; no blocking, no tables shared with the GPU code.
"""
from __future__ import annotations

import numpy as np

E4M3_MAX = 448.0
E4M3_NAN = 0x7F


def e4m3_decode(code) -> np.ndarray:
    """Value (float64) of each 8-bit code."""
    c = np.asarray(code, dtype=np.uint8).astype(np.int64)
    sign = np.where((c >> 7) & 1, -1.0, 1.0)
    e = (c >> 3) & 0xF
    m = (c & 0x7).astype(np.float64)
    normal = (1.0 + m / 8.0) * np.exp2((e - 7).astype(np.float64))
    subnormal = (m / 8.0) * 2.0 ** -6
    val = np.where(e == 0, subnormal, normal)
    val = np.where((e == 15) & (m == 7), np.nan, val)
    return sign * val


def _magnitudes() -> np.ndarray:
    """The 127 finite non-negative values, in code order 0x00 .. 0x7E (strictly increasing)."""
    return e4m3_decode(np.arange(0x7F, dtype=np.uint8))


def e4m3_encode(x) -> np.ndarray:
    """Code of each float32 value: nearest representable magnitude, a tie goes to the code whose last mantissa bit
    is 0 (the even code), magnitudes beyond 448 give 448; the sign bit is the input's; NaN gives 0x7F."""
    x = np.asarray(x, dtype=np.float32)
    a = np.abs(x).astype(np.float64)
    mags = _magnitudes()
    hi = np.clip(np.searchsorted(mags, a, side="left"), 1, 126)     # first code with magnitude >= a (at least 1)
    lo = hi - 1
    d_lo, d_hi = a - mags[lo], mags[hi] - a
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi % 2 == 0))
    code = np.where(pick_hi, hi, lo)
    code = np.where(a >= E4M3_MAX, 126, code)
    code = code.astype(np.uint8) | (np.signbit(x).astype(np.uint8) << 7)
    return np.where(np.isnan(x), np.uint8(E4M3_NAN), code).astype(np.uint8)


def quantize_rows(x, scale) -> np.ndarray:
    """Bytes of rows x (any float array whose values are exact in float32) under `scale` (broadcastable, fp32):
    the quotient is taken in float32, as the conversion's input is."""
    t = np.asarray(x, dtype=np.float32) / np.asarray(scale, dtype=np.float32)
    return e4m3_encode(t.astype(np.float32))


def dequantize_rows(code, scale) -> np.ndarray:
    """float64 values of cached bytes under `scale` (fp32, broadcastable)."""
    return e4m3_decode(code) * np.asarray(scale, dtype=np.float32).astype(np.float64)


def attention_decode_fp8(q, k_t, v_t, k_code, v_code, k_scale: float, v_scale: float, n: int, scale: float) -> np.ndarray:
    """Eq. 6, second line, for one (sequence, head): the current token attends the n cached rows, read as
    decode(byte) * scale, and itself (k_t, v_t as given).  q, k_t, v_t [D]; k_code, v_code [>= n][D] uint8."""
    q = np.asarray(q, dtype=np.float64)
    d = q.shape[0]
    k = np.vstack([dequantize_rows(np.asarray(k_code)[:n].reshape(n, d), k_scale),
                   np.asarray(k_t, dtype=np.float64)[None, :]])
    v = np.vstack([dequantize_rows(np.asarray(v_code)[:n].reshape(n, d), v_scale),
                   np.asarray(v_t, dtype=np.float64)[None, :]])
    z = (k @ q) * scale
    e = np.exp(z - z.max())
    return (e / e.sum()) @ v


def append_row_fp8(k_t, v_t, k_scale: float, v_scale: float, k_code, v_code, n: int, cap: int, keep: bool) -> int:
    """Eq. 6, third line, on the 8-bit cache of one (sequence, head): a kept token's row goes to position n in
    quantised form (a full cache is left untouched).  Returns the new length."""
    if not keep or n >= cap:
        return n
    k_code[n] = quantize_rows(k_t, k_scale)
    v_code[n] = quantize_rows(v_t, v_scale)
    return n + 1
