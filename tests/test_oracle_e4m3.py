"""Pins for the oracle's E4M3 encode / decode (CPU only).

The oracle encodes by searching the sorted list of representable values.  It is pinned
here against things that are not that search: the format's published constants, an
independently written bit-level rounding routine, exact rational arithmetic, and the
``torch.float8_e4m3fn`` cast inside its non-saturating range.
"""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import e4m3

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "e4m3_format.txt")


def test_decode_matches_published_format_constants():
    rows = [ln.split() for ln in open(GOLDEN) if ln.strip() and not ln.startswith("#")]
    assert len(rows) >= 12
    for code_s, value_s in rows:
        code, want = int(code_s, 16), float(value_s)
        got = e4m3.decode(np.array([code], dtype=np.uint8))[0]
        if np.isnan(want):
            assert np.isnan(got)
        else:
            assert got == want and np.signbit(got) == np.signbit(want), (code_s, got, want)


def test_decode_is_monotone_and_has_254_finite_codes():
    pos = e4m3.DECODE_TABLE[:0x7F]
    assert np.all(np.diff(pos) > 0)
    assert np.isfinite(e4m3.DECODE_TABLE).sum() == 254
    assert np.array_equal(e4m3.DECODE_TABLE[0x80:0xFF], -pos)


def test_round_trip_every_code():
    codes = np.arange(256, dtype=np.uint8)
    finite = np.isfinite(e4m3.DECODE_TABLE)
    back = e4m3.encode(e4m3.DECODE_TABLE[finite].astype(np.float32))
    assert np.array_equal(back, codes[finite])


def test_midpoints_tie_to_even_and_neighbours_round_to_nearest():
    pos = e4m3.DECODE_TABLE[:0x7F]
    for c in range(0x7E):
        lo, hi = pos[c], pos[c + 1]
        mid = np.float32((lo + hi) / 2)                 # exact: both are short dyadics
        assert float(mid) == (lo + hi) / 2
        even = c if c % 2 == 0 else c + 1
        assert e4m3.encode(np.array([mid]))[0] == even
        assert e4m3.encode(np.array([-mid]))[0] == (even | 0x80)
        below = np.nextafter(mid, np.float32(0), dtype=np.float32)
        above = np.nextafter(mid, np.float32(1e9), dtype=np.float32)
        assert e4m3.encode(np.array([below]))[0] == c
        assert e4m3.encode(np.array([above]))[0] == c + 1


def test_saturation_and_tiny_values():
    x = np.array([448.0, 449.0, 464.0, 464.0001, 1e6, 3.0e38, -500.0], dtype=np.float32)
    assert list(e4m3.encode(x)) == [0x7E] * 6 + [0xFE]
    tiny = np.array([2.0 ** -10, np.nextafter(np.float32(2.0 ** -10), np.float32(1)), 2.0 ** -11,
                     1e-30, -1e-30, 0.0, -0.0], dtype=np.float32)
    # 2^-10 is the midpoint of 0 and 2^-9: ties to the even code 0
    assert list(e4m3.encode(tiny)) == [0x00, 0x01, 0x00, 0x00, 0x80, 0x00, 0x80]


def _encode_bits(x: np.ndarray) -> np.ndarray:
    """Independent encoder: integer rounding on the fp32 bit pattern (round-half-even by
    adding a bias), written separately from the oracle's search."""
    bits = x.astype(np.float32).view(np.uint32).astype(np.int64)
    sign = (bits >> 31) & 1
    mag = bits & 0x7FFFFFFF
    out = np.zeros(x.shape, dtype=np.int64)
    normal = mag >= ((127 - 6) << 23)                       # |x| >= 2^-6
    lsb = (mag >> 20) & 1
    r = (mag + 0x7FFFF + lsb) >> 20                         # keep 3 mantissa bits
    out_n = r - ((127 - 7) << 3)
    out_n = np.minimum(out_n, 0x7E)
    # subnormal range: code = round_half_even(|x| * 2^9), computed on the exact value
    a = np.where(normal, 0.0, np.abs(x.astype(np.float64))) * 512.0
    out_s = np.rint(a).astype(np.int64)                     # numpy rint is half-to-even
    out = np.where(normal, out_n, out_s)
    out = np.where(mag > 0x7F800000, 0x7F, out)
    return (out | np.where(mag > 0x7F800000, 0, sign << 7)).astype(np.uint8)


def test_against_independent_bit_level_encoder_all_bf16_and_random_fp32():
    hi16 = np.arange(1 << 16, dtype=np.uint32) << 16        # every bf16 value as fp32
    x = hi16.view(np.float32)
    x = x[np.isfinite(x)]
    assert np.array_equal(e4m3.encode(x), _encode_bits(x))
    rng = np.random.default_rng(0)
    y = (rng.standard_normal(400_000) * np.exp(rng.uniform(-12, 7, 400_000))).astype(np.float32)
    assert np.array_equal(e4m3.encode(y), _encode_bits(y))
    z = rng.integers(0, 1 << 32, 400_000, dtype=np.uint64).astype(np.uint32).view(np.float32)
    z = z[np.isfinite(z)]
    assert np.array_equal(e4m3.encode(z), _encode_bits(z))


def test_against_exact_rational_nearest_on_a_sample():
    vals = [Fraction(float(v)) for v in e4m3.DECODE_TABLE[:0x7F]]
    rng = np.random.default_rng(1)
    xs = (rng.standard_normal(300) * np.exp(rng.uniform(-9, 6.5, 300))).astype(np.float32)
    for x in xs:
        a = abs(Fraction(float(x)))
        best = min(range(0x7F), key=lambda c: (abs(vals[c] - a), c % 2))
        want = best | (0x80 if x < 0 else 0)
        assert e4m3.encode(np.array([x]))[0] == want


def test_against_torch_float8_cast_inside_its_finite_range():
    rng = np.random.default_rng(2)
    x = (rng.standard_normal(500_000) * np.exp(rng.uniform(-12, 5.5, 500_000))).astype(np.float32)
    x = x[np.abs(x) <= 464.0]                                # torch returns NaN beyond, by design
    want = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(e4m3.encode(x), want)
    back = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).double().numpy()
    finite = np.isfinite(back)
    assert np.array_equal(back[finite], e4m3.DECODE_TABLE[finite])


def test_half_ulp_error_bound():
    rng = np.random.default_rng(3)
    y = rng.uniform(-448, 448, 200_000).astype(np.float32)
    err = np.abs(e4m3.decode(e4m3.encode(y)) - y.astype(np.float64))
    e = np.maximum(np.floor(np.log2(np.maximum(np.abs(y.astype(np.float64)), 1e-300))), -6)
    assert np.all(err <= 2.0 ** (e - 4))


def test_planted_mistakes_are_caught():
    """The pins above must fail for plausible wrong encoders (truncation, ties away)."""
    pos = e4m3.DECODE_TABLE[:0x7F]

    def truncating(x):
        return np.maximum(np.searchsorted(pos, np.abs(x), side="right") - 1, 0).astype(np.uint8)

    mids = ((pos[:-1] + pos[1:]) / 2).astype(np.float32)
    assert not np.array_equal(truncating(mids), e4m3.encode(mids))
    ties_away = np.arange(1, 0x7F)                         # always the upper neighbour
    assert not np.array_equal(ties_away, e4m3.encode(mids))
