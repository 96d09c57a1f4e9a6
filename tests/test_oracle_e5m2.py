"""Pins for the oracle's E5M2 encode / decode and for the cache write in that format (CPU only).

As for E4M3, the encoder (a search in the sorted list of finite values) is pinned against things that
are not that search: the format's published constants, the fact that an E5M2 code is the upper byte of
the IEEE half-precision number of the same value, exact rational arithmetic, the ``torch.float8_e5m2``
cast inside its finite range, and planted mistakes.
"""
import os
from fractions import Fraction

import numpy as np
import torch

from oracle import e4m3, e5m2, kv_cache

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "e5m2_format.txt")


def test_decode_matches_published_format_constants():
    rows = [ln.split() for ln in open(GOLDEN) if ln.strip() and not ln.startswith("#")]
    assert len(rows) >= 14
    for code_s, value_s in rows:
        got, want = e5m2.decode(np.array([int(code_s, 16)], dtype=np.uint8))[0], float(value_s)
        if np.isnan(want):
            assert np.isnan(got)
        else:
            assert got == want and np.signbit(got) == np.signbit(want), (code_s, got, want)


def test_a_code_is_the_upper_byte_of_the_half_precision_number():
    codes = np.arange(256, dtype=np.uint16)
    halves = (codes << 8).astype(np.uint16).view(np.float16).astype(np.float64)
    table = e5m2.DECODE_TABLE
    same = (halves == table) | (np.isnan(halves) & np.isnan(table))
    assert same.all()
    assert np.isfinite(table).sum() == 248 and np.all(np.diff(table[:0x7C]) > 0)


def test_round_trip_and_saturation():
    finite = np.array([c for c in range(256) if np.isfinite(e5m2.DECODE_TABLE[c])], dtype=np.uint8)
    assert np.array_equal(e5m2.encode(e5m2.decode(finite)), finite)
    big = np.array([57344.0, 60000.0, 65504.0, 1e9, -61440.1, -1e30])
    assert e5m2.encode(big).tolist() == [0x7B, 0x7B, 0x7B, 0x7B, 0xFB, 0xFB]
    tiny = np.array([2.0 ** -17, -2.0 ** -17, 2.0 ** -17 * 1.0001, 0.0, -0.0])
    assert e5m2.encode(tiny).tolist() == [0x00, 0x80, 0x01, 0x00, 0x80]       # the midpoint below the first code ties to even (zero)


def test_every_midpoint_ties_to_the_even_code_and_its_neighbours_round_away():
    pos = e5m2.DECODE_TABLE[:0x7C]
    for c in range(0x7B):
        mid = (Fraction(pos[c]) + Fraction(pos[c + 1])) / 2
        assert float(mid) == mid                                             # midpoints are exact in float64
        even = c if c % 2 == 0 else c + 1
        assert e5m2.encode(np.array([float(mid)]))[0] == even
        assert e5m2.encode(np.array([np.nextafter(float(mid), 0.0)]))[0] == c
        assert e5m2.encode(np.array([np.nextafter(float(mid), np.inf)]))[0] == c + 1


def test_encode_is_the_exact_nearest_value_on_random_inputs():
    rng = np.random.default_rng(3)
    x = np.concatenate([rng.normal(0, 1, 3000), rng.normal(0, 300, 3000), rng.uniform(-6e4, 6e4, 2000),
                        rng.normal(0, 1e-4, 2000)]).astype(np.float32)
    got = e5m2.decode(e5m2.encode(x))
    finite = [Fraction(v) for v in e5m2.DECODE_TABLE[:0x7C]]
    for xi, gi in zip(x[::7], got[::7]):
        a = abs(Fraction(float(xi)))
        best = min(abs(a - f) for f in finite)
        assert abs(abs(Fraction(float(gi))) - a) == best


def test_matches_the_torch_cast_inside_the_finite_range():
    rng = np.random.default_rng(4)
    x = np.concatenate([rng.normal(0, 1, 20000), rng.normal(0, 2000, 20000), rng.normal(0, 1e-3, 20000)]).astype(np.float32)
    x = x[np.abs(x) <= 57344.0]
    want = torch.from_numpy(x).to(torch.float8_e5m2).view(torch.uint8).numpy()
    assert np.array_equal(e5m2.encode(x), want)


def test_planted_mistakes_are_caught():
    # midpoints between neighbouring codes: 1.0|1.25, 1.25|1.5, 2.0|2.5, -(0.4375|0.5)
    x = np.array([1.125, 1.375, 2.25, -0.46875], dtype=np.float32)
    good = e5m2.encode(x)
    truncating = (x.astype(np.float16).view(np.uint16) >> 8).astype(np.uint8)  # drops the low byte instead of rounding
    away = np.array([0x3D, 0x3E, 0x41, 0xB8], dtype=np.uint8)                  # ties away from zero
    assert good.tolist() == [0x3C, 0x3E, 0x40, 0xB8]                           # ties to the even code
    assert truncating.tolist() == [0x3C, 0x3D, 0x40, 0xB7]
    assert not np.array_equal(good, truncating) and not np.array_equal(good, away)


def test_cache_write_in_e5m2_follows_the_same_scale_rule():
    """scale = amax / 57344, the largest value lands on the top code, resident codes are re-expressed when
    the scale grows, and the E4M3 write is unchanged by the format parameter's existence."""
    rng = np.random.default_rng(5)
    k = rng.normal(0, 1, (20, 2, 8)).astype(np.float32)
    v = rng.normal(0, 3, (20, 2, 8)).astype(np.float32)
    slots = np.arange(20, dtype=np.int64) + 16                                 # blocks 1 and 2
    codes, scales = kv_cache.new_cache(4, 2, 8)
    kv_cache.kv_write(codes, scales, k[:10], v[:10], slots[:10], fmt=e5m2)
    amax = np.abs(k[:10, 0]).max()
    assert scales[1, 0, 0] == np.float32(amax / np.float32(57344.0))
    assert (codes[1, 0, 0, :10] & 0x7F).max() == 0x7B
    before = e5m2.decode(codes[1, 0, 0, :10]) * float(scales[1, 0, 0])
    k2 = k[10:16].copy()
    k2[0, 0, 0] = 4 * amax                                                    # grows the scale of block 1, head 0, K
    kv_cache.kv_write(codes, scales, k2, v[10:16], slots[10:16], fmt=e5m2)
    assert scales[1, 0, 0] == np.float32(np.float32(4 * amax) / np.float32(57344.0))
    after = e5m2.decode(codes[1, 0, 0, :10]) * float(scales[1, 0, 0])
    assert np.all(np.abs(after - before) <= 0.125 * np.abs(before) + 2.0 ** -16 * float(scales[1, 0, 0]))   # half an ulp of two mantissa bits
    c4, s4 = kv_cache.new_cache(4, 2, 8)
    kv_cache.kv_write(c4, s4, k, v, slots)
    c4b, s4b = kv_cache.new_cache(4, 2, 8)
    kv_cache.kv_write(c4b, s4b, k, v, slots, fmt=e4m3)
    assert np.array_equal(c4, c4b) and np.array_equal(s4, s4b)
