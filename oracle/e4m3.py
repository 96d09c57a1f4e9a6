"""TEST INFRASTRUCTURE — CPU oracle, part 0: the FP8 E4M3 number format.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA path shares no code with it.

The paper compresses cached K/V "into FP8 format" (Section 3.1, Opt-KV) and restores
them with ``dequant`` (Eq. 6) without fixing the format.  The reading taken here is the
OCP 8-bit float E4M3 ("fn" variant): 1 sign bit, 4 exponent bits with bias 7, 3 mantissa
bits, no infinities, codes 0x7F / 0xFF are NaN, largest finite value 448 (code 0x7E),
smallest normal 2**-6, subnormals m * 2**-9.  Encoding rounds to nearest, ties to the
even code, and saturates to +-448 ("satfinite").

Everything is written as the definition: decode is the closed form of the format,
encode is "the nearest representable value, ties to even", found by search in the sorted
list of representable values.  No bit tricks.
"""
from __future__ import annotations

import numpy as np

E4M3_MAX = 448.0
MAX = E4M3_MAX          # the names the cache oracle uses for whichever format it is given
NAME = "e4m3"


def decode_code(code: int) -> float:
    """Value of one E4M3 code (closed form of the format)."""
    sign = -1.0 if (code >> 7) & 1 else 1.0
    e = (code >> 3) & 0xF
    m = code & 0x7
    if e == 0xF and m == 0x7:
        return float("nan")
    if e == 0:
        return sign * m * 2.0 ** -9
    return sign * 2.0 ** (e - 7) * (1.0 + m / 8.0)


#: value of every code, float64 (exact); NaN at 0x7F and 0xFF
DECODE_TABLE = np.array([decode_code(c) for c in range(256)], dtype=np.float64)

#: the 127 non-negative finite values in increasing order; index == code
_POSITIVE = DECODE_TABLE[:0x7F].copy()


def decode(codes: np.ndarray) -> np.ndarray:
    """uint8 codes -> float64 values (Eq. 6's ``dequant`` without the scale)."""
    return DECODE_TABLE[np.asarray(codes, dtype=np.uint8)]


def encode(x: np.ndarray) -> np.ndarray:
    """float values -> uint8 E4M3 codes: nearest value, ties to even code, saturating.

    The sign of the input is kept even when the magnitude rounds to zero.  NaN maps
    to the NaN code 0x7F (inputs are required to be finite; this is for completeness).
    """
    x = np.asarray(x)
    a = np.abs(x.astype(np.float64))
    neg = np.signbit(x)
    nan = np.isnan(a)
    a = np.where(nan, 0.0, a)
    # hi = first representable value >= a (or past the end when a > 448)
    hi = np.searchsorted(_POSITIVE, a, side="left")
    hi_c = np.minimum(hi, 0x7E)
    lo_c = np.maximum(hi_c - 1, 0)
    d_hi = np.abs(_POSITIVE[hi_c] - a)
    d_lo = np.abs(a - _POSITIVE[lo_c])
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi_c % 2 == 0))
    code = np.where(pick_hi, hi_c, lo_c)
    code = np.where(hi > 0x7E, 0x7E, code)          # beyond 448: saturate
    code = np.where(nan, 0x7F, code)
    code = code.astype(np.uint8)
    return np.where(neg & ~nan, code | np.uint8(0x80), code).astype(np.uint8)
