"""TEST INFRASTRUCTURE — CPU oracle: the FP8 E5M2 number format (an ablation of the cache format).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA path shares no code with it.

The paper says "FP8" (Section 3.1, Eq. 6) and nothing more.  E4M3 is the reading the build
takes; E5M2, the other OCP 8-bit float, is offered as an ablation: 1 sign bit, 5 exponent
bits with bias 15, 2 mantissa bits, infinities at S.11111.00 and NaN at S.11111.{01,10,11},
largest finite value 57344 (code 0x7B), smallest normal 2**-14, subnormals m * 2**-16.
Encoding rounds to nearest, ties to the even code, and saturates to +-57344: an infinity
is never produced.

As in ``e4m3``: decode is the closed form of the format, encode is the nearest
representable value found by search in the sorted list of finite values.
"""
from __future__ import annotations

import numpy as np

MAX = 57344.0
NAME = "e5m2"
MAX_CODE = 0x7B
NAN_CODE = 0x7F


def decode_code(code: int) -> float:
    """Value of one E5M2 code (closed form of the format)."""
    sign = -1.0 if (code >> 7) & 1 else 1.0
    e = (code >> 2) & 0x1F
    m = code & 0x3
    if e == 0x1F:
        return sign * float("inf") if m == 0 else float("nan")
    if e == 0:
        return sign * m * 2.0 ** -16
    return sign * 2.0 ** (e - 15) * (1.0 + m / 4.0)


#: value of every code, float64 (exact); +-inf at 0x7C / 0xFC, NaN behind them
DECODE_TABLE = np.array([decode_code(c) for c in range(256)], dtype=np.float64)

#: the 124 non-negative finite values in increasing order; index == code
_POSITIVE = DECODE_TABLE[:MAX_CODE + 1].copy()


def decode(codes: np.ndarray) -> np.ndarray:
    """uint8 codes -> float64 values."""
    return DECODE_TABLE[np.asarray(codes, dtype=np.uint8)]


def encode(x: np.ndarray) -> np.ndarray:
    """float values -> uint8 E5M2 codes: nearest finite value, ties to even code, saturating.

    The sign of the input is kept even when the magnitude rounds to zero.  NaN maps to a
    NaN code (inputs are required to be finite; this is for completeness).
    """
    x = np.asarray(x)
    a = np.abs(x.astype(np.float64))
    neg = np.signbit(x)
    nan = np.isnan(a)
    a = np.where(nan, 0.0, a)
    hi = np.searchsorted(_POSITIVE, a, side="left")          # first finite value >= a, or past the end
    hi_c = np.minimum(hi, MAX_CODE)
    lo_c = np.maximum(hi_c - 1, 0)
    d_hi = np.abs(_POSITIVE[hi_c] - a)
    d_lo = np.abs(a - _POSITIVE[lo_c])
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi_c % 2 == 0))
    code = np.where(pick_hi, hi_c, lo_c)
    code = np.where(hi > MAX_CODE, MAX_CODE, code)            # beyond 57344: saturate
    code = np.where(nan, NAN_CODE, code).astype(np.uint8)
    return np.where(neg & ~nan, code | np.uint8(0x80), code).astype(np.uint8)
