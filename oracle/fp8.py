"""The e4m3 8-bit floating-point encoding, for the tests of the 8-bit LM head -- TEST INFRASTRUCTURE.

Written from the format's published definition (OCP 8-bit floating point, E4M3): 1 sign bit, 4
exponent bits with bias 7, 3 mantissa bits; exponent field 0 holds subnormals m * 2^-9; there are no
infinities, the all-ones pattern is NaN, the largest finite value is 448 (code 0x7E).  The tests use
it to build, on the CPU, the dequantised LM head a context with 8-bit weights computes with:
``W8[v, :] = scale[v] * e4m3(W[v, :] / scale[v])`` with ``scale[v] = 2^E``, E the smallest integer with
``max|W[v, :]| <= 448 * 2^E``, rounding to nearest with ties to the even code.  The oracle then runs
unchanged on W8.  Shares nothing with the CUDA path.
"""
from __future__ import annotations

import numpy as np


def code_values() -> np.ndarray:
    """Values of the non-negative finite codes 0x00 .. 0x7E (float64, ascending)."""
    v = np.empty(127, np.float64)
    for c in range(127):
        e, m = c >> 3, c & 7
        v[c] = m * 2.0 ** -9 if e == 0 else 2.0 ** (e - 7) * (1.0 + m / 8.0)
    return v


_VALS = code_values()


def encode(y: np.ndarray) -> np.ndarray:
    """uint8 e4m3 codes of float values: nearest code, ties to the even code, saturating at 448."""
    y = np.asarray(y, np.float64)
    a = np.abs(y)
    hi = np.searchsorted(_VALS, a, side="left")            # first code whose value is >= a
    hi = np.minimum(hi, 126)
    lo = np.maximum(hi - 1, 0)
    d_lo, d_hi = a - _VALS[lo], _VALS[hi] - a
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi % 2 == 0))
    code = np.where(a >= 448.0, 126, np.where(pick_hi, hi, lo)).astype(np.uint8)
    return code | np.where(np.signbit(y), 0x80, 0).astype(np.uint8)


def decode(code: np.ndarray) -> np.ndarray:
    code = np.asarray(code, np.uint8)
    mag = _VALS[np.minimum(code & 0x7F, 126)]
    return np.where(code & 0x80, -mag, mag)


def row_scales(w: np.ndarray) -> np.ndarray:
    """2^E per row, E the smallest integer with max|row| <= 448 * 2^E (1 for an all-zero row)."""
    amax = np.abs(np.asarray(w, np.float64)).max(axis=1)
    f, e = np.frexp(amax)                                   # amax = f * 2^e, f in [0.5, 1); 448 = 0.875 * 2^9
    E = e - 9 + (f > 0.875)
    return np.where(amax > 0, np.ldexp(1.0, E), 1.0)


def quantise_rows(w: np.ndarray):
    """(codes uint8 [V, d], scales float32 [V], dequantised float32 [V, d]) of a weight matrix."""
    w = np.asarray(w, np.float32)
    s = row_scales(w)
    codes = encode(w.astype(np.float64) / s[:, None])
    deq = (decode(codes) * s[:, None]).astype(np.float32)
    return codes, s.astype(np.float32), deq
