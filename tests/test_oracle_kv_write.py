"""Pins for the oracle's Opt-KV write (CPU only): exact rational brute force on tiny
inputs, closed-form special cases and the invariants the method must keep."""
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import e4m3, kv_cache


def _bf16(x: np.ndarray) -> np.ndarray:
    return torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16).float().numpy()


def _inputs(rng, T, H, D, outliers=True):
    k = rng.standard_normal((T, H, D))
    v = rng.standard_normal((T, H, D))
    if outliers:
        k[:, :, 1] *= 20.0
        v[:, :, D - 1] *= 20.0
    return _bf16(k), _bf16(v)


# ---- exact rational re-derivation ----------------------------------------------------------

def _round_to_fp32(fr: Fraction) -> Fraction:
    """Round a rational to the nearest fp32 value (ties to even), normal or subnormal."""
    if fr == 0:
        return fr
    sign = -1 if fr < 0 else 1
    a = abs(fr)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    e = max(e, -126)
    q = a / Fraction(2) ** (e - 23)                      # significand as a multiple of one ulp
    n = q.numerator // q.denominator
    rem = q - n
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and n % 2 == 1):
        n += 1
    return sign * n * Fraction(2) ** (e - 23)


_CODE_VALUES = [Fraction(float(v)) for v in e4m3.DECODE_TABLE[:0x7F]]


def _enc_exact(y: Fraction, negative: bool) -> int:
    a = abs(y)
    if a > 448:
        c = 0x7E
    else:
        c = min(range(0x7F), key=lambda i: (abs(_CODE_VALUES[i] - a), i % 2))
    return c | (0x80 if negative else 0)


def _brute_force_write(codes, scales, k, v, slots):
    """The write, token group by token group, in exact rational arithmetic with explicit
    fp32 roundings.  codes: dict[(blk,h,w,off,d)] -> int, scales: dict[(blk,h,w)] -> Fraction."""
    T, H, D = k.shape
    groups = {}
    for i, s in enumerate(slots):
        if s >= 0:
            groups.setdefault(s // 16, []).append(i)
    for blk, toks in groups.items():
        offs = [slots[i] % 16 for i in toks]
        fresh = 0 in offs
        for h in range(H):
            for w, src in enumerate((k, v)):
                amax = max(abs(Fraction(float(src[i, h, d]))) for i in toks for d in range(D))
                s_old = Fraction(0) if fresh else scales.get((blk, h, w), Fraction(0))
                s_new = max(s_old, _round_to_fp32(amax / 448))
                for off in range(16):
                    if off in offs:
                        continue
                    for d in range(D):
                        key = (blk, h, w, off, d)
                        if fresh:
                            codes[key] = 0
                        elif s_new > s_old and s_old > 0:
                            c = codes.get(key, 0)
                            val = _round_to_fp32(Fraction(float(e4m3.DECODE_TABLE[c])) * s_old)
                            y = _round_to_fp32(val / s_new)
                            codes[key] = _enc_exact(y, bool(c & 0x80))
                for i, off in zip(toks, offs):
                    for d in range(D):
                        x = float(src[i, h, d])
                        neg = bool(np.signbit(np.float32(x)))
                        if s_new == 0:
                            codes[(blk, h, w, off, d)] = 0x80 if neg else 0
                        else:
                            y = _round_to_fp32(Fraction(x) / s_new)
                            codes[(blk, h, w, off, d)] = _enc_exact(y, neg)
                scales[(blk, h, w)] = s_new


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_brute_force_tiny_with_appends_skips_and_block_reuse(seed):
    rng = np.random.default_rng(seed)
    NB, H, D = 3, 2, 4
    codes, scales = kv_cache.new_cache(NB, H, D)
    ref_codes, ref_scales = {}, {}
    calls = [
        list(range(16, 16 + 5)) + [-1] + list(range(32, 32 + 16)) + list(range(0, 3)),   # bulk + skip
        [21], [22], [-1], [23, 24, 25],                                                 # appends to block 1
        [3], [4, 5],                                                                    # appends to block 0
        list(range(16, 16 + 2)),                                                        # block 1 reused: fresh
    ]
    for call_no, slots in enumerate(calls):
        k, v = _inputs(rng, len(slots), H, D)
        if call_no in (1, 5):                 # force scale growth and an all-zero token
            k *= 3.0
            v[:] = 0.0
            k, v = _bf16(k), _bf16(v)
        kv_cache.kv_write(codes, scales, k, v, np.array(slots))
        _brute_force_write(ref_codes, ref_scales, k, v, slots)
        for (blk, h, w), s in ref_scales.items():
            assert Fraction(float(scales[blk, h, w])) == s
        for (blk, h, w, off, d), c in ref_codes.items():
            assert codes[blk, h, w, off, d] == c, (call_no, blk, h, w, off, d)
    untouched = set(range(NB)) - {b for (b, _, _) in ref_scales}
    for blk in untouched:
        assert not codes[blk].any() and not scales[blk].any()


# ---- closed forms and invariants ---------------------------------------------------------------

def test_scale_is_amax_over_448_and_top_value_hits_max_code():
    rng = np.random.default_rng(5)
    k, v = _inputs(rng, 16, 2, 8)
    codes, scales = kv_cache.new_cache(2, 2, 8)
    kv_cache.kv_write(codes, scales, k, v, np.arange(16, 32))
    for h in range(2):
        for w, x in enumerate((k, v)):
            amax = np.abs(x[:, h]).max()
            assert scales[1, h, w] == np.float32(amax) / np.float32(448.0)
            assert (codes[1, h, w] & 0x7F).max() == 0x7E
    assert not codes[0].any() and not scales[0].any()


def test_dequant_error_within_half_ulp_of_the_block_scale():
    rng = np.random.default_rng(6)
    T, H, D = 64, 3, 32
    k, v = _inputs(rng, T, H, D)
    codes, scales = kv_cache.new_cache(4, H, D)
    kv_cache.kv_write(codes, scales, k, v, np.arange(T))
    deq = kv_cache.dequantise(codes, scales)
    for w, x in enumerate((k, v)):
        x = x.reshape(4, 16, H, D).transpose(0, 2, 1, 3).astype(np.float64)     # [blk, h, off, d]
        s = scales[:, :, w].astype(np.float64)[:, :, None, None]
        y = np.abs(x) / s
        e = np.maximum(np.floor(np.log2(np.maximum(y, 1e-300))), -6)
        bound = 2.0 ** (e - 4) * s * (1 + 2.0 ** -20)
        assert np.all(np.abs(deq[:, :, w] - x) <= bound)
        assert np.all(bound <= np.abs(x).max(axis=(2, 3), keepdims=True) / 28 * (1 + 1e-6))


def test_doubling_the_scale_halves_resident_values_exactly():
    """Special case with a closed form: a new token whose amax is exactly twice the
    block's makes s_new = 2 * s_old, and every resident normal code loses one exponent."""
    D = 8
    codes, scales = kv_cache.new_cache(1, 1, D)
    first = np.zeros((1, 1, D), dtype=np.float32)
    first[0, 0] = [448, 224, 1.0, 2 ** -3, 0.5, -3.5, 96, 0]        # scale becomes exactly 1
    kv_cache.kv_write(codes, scales, first, first, np.array([0]))
    assert scales[0, 0, 0] == 1.0
    before = codes[0, 0, 0, 0].copy()
    second = np.zeros((1, 1, D), dtype=np.float32)
    second[0, 0, 0] = 896.0
    kv_cache.kv_write(codes, scales, second, second, np.array([1]))
    assert scales[0, 0, 0] == 2.0
    after = codes[0, 0, 0, 0]
    assert np.array_equal(e4m3.decode(after), e4m3.decode(before) / 2)
    assert np.array_equal(after[:7] & 0x78, (before[:7] & 0x78) - 8)  # exponent field minus one
    assert codes[0, 0, 0, 1, 0] == 0x7E


def test_scale_is_monotone_under_appends_and_token_by_token_stays_bounded():
    rng = np.random.default_rng(7)
    H, D = 2, 16
    k, v = _inputs(rng, 16, H, D)
    one_c, one_s = kv_cache.new_cache(1, H, D)
    kv_cache.kv_write(one_c, one_s, k, v, np.arange(16))
    inc_c, inc_s = kv_cache.new_cache(1, H, D)
    prev = inc_s.copy()
    growth = np.zeros_like(inc_s)
    for t in range(16):
        kv_cache.kv_write(inc_c, inc_s, k[t:t + 1], v[t:t + 1], np.array([t]))
        assert np.all(inc_s >= prev)
        growth += (inc_s > prev) & (prev > 0)
        prev = inc_s.copy()
    assert np.array_equal(inc_s, one_s)                       # the final scale is the same amax/448
    deq = kv_cache.dequantise(inc_c, inc_s)
    for w, x in enumerate((k, v)):
        x = x.transpose(1, 0, 2).astype(np.float64)           # [h, off, d]
        s = inc_s[0, :, w].astype(np.float64)[:, None, None]
        half_ulp_top = 16 * s                                 # half an ulp in the top binade
        assert np.all(np.abs(deq[0, :, w] - x) <= (1 + growth[0, :, w][:, None, None]) * half_ulp_top)


def test_permuting_physical_blocks_permutes_the_cache_and_nothing_else():
    rng = np.random.default_rng(8)
    T, H, D, NB = 40, 2, 8, 5
    k, v = _inputs(rng, T, H, D)
    logical = np.arange(T)
    results = []
    for perm in (np.arange(NB), rng.permutation(NB)):
        codes, scales = kv_cache.new_cache(NB, H, D)
        slots = perm[logical // 16] * 16 + logical % 16
        kv_cache.kv_write(codes, scales, k, v, slots)
        results.append((perm, codes, scales))
    (p0, c0, s0), (p1, c1, s1) = results
    for j in range(3):
        assert np.array_equal(c0[p0[j]], c1[p1[j]]) and np.array_equal(s0[p0[j]], s1[p1[j]])
    used = set(p1[:3].tolist())
    for blk in range(NB):
        if blk not in used:
            assert not c1[blk].any() and not s1[blk].any()


def test_negative_slots_are_skipped_and_heads_subset_matches():
    rng = np.random.default_rng(9)
    T, H, D = 20, 3, 8
    k, v = _inputs(rng, T, H, D)
    slots = np.arange(T)
    slots_skip = slots.copy()
    slots_skip[[3, 17]] = -1
    a_c, a_s = kv_cache.new_cache(2, H, D)
    kv_cache.kv_write(a_c, a_s, k, v, slots_skip)
    keep = slots_skip >= 0
    b_c, b_s = kv_cache.new_cache(2, H, D)
    kv_cache.kv_write(b_c, b_s, k[keep], v[keep], slots[keep])
    assert np.array_equal(a_c, b_c) and np.array_equal(a_s, b_s)
    assert not a_c[0, :, :, 3].any() and not a_c[1, :, :, 1].any()
    c_c, c_s = kv_cache.new_cache(2, H, D)
    kv_cache.kv_write(c_c, c_s, k, v, slots_skip, heads=[1])
    assert np.array_equal(c_c[:, 1], a_c[:, 1]) and np.array_equal(c_s[:, 1], a_s[:, 1])
    assert not c_c[:, 0].any() and not c_c[:, 2].any()


def test_all_zero_block_and_signed_zero():
    codes, scales = kv_cache.new_cache(1, 1, 4)
    z = np.zeros((2, 1, 4), dtype=np.float32)
    z[1, 0, 2] = -0.0
    kv_cache.kv_write(codes, scales, z, z, np.array([0, 1]))
    assert scales[0, 0, 0] == 0 and codes[0, 0, 0, 1, 2] == 0x80
    assert np.count_nonzero(codes) == 2
    assert not kv_cache.dequantise(codes, scales).any()


def test_bf16_ablation_write_stores_values_unchanged():
    rng = np.random.default_rng(10)
    k, v = _inputs(rng, 20, 2, 8)
    vals = kv_cache.new_cache_bf16(3, 2, 8)
    slots = np.concatenate([np.arange(32, 48), [-1], np.arange(3, 6)])
    kv_cache.kv_write_bf16(vals, k, v, slots)
    assert np.array_equal(vals[2, :, 0], k[:16].transpose(1, 0, 2))
    assert np.array_equal(vals[0, :, 1, 3:6], v[17:].transpose(1, 0, 2))
    assert not vals[1].any() and not vals[0, :, :, :3].any()
