"""CPU-side checks of the C-ABI library: it loads, exports every symbol the public header
declares, and its host-only arithmetic (layout, sizes, argument checks) behaves."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2602_09323_b200 import binding, build

HEADER = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include", "coopt.h")


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def _declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(coopt_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(lib):
    names = _declared_functions()
    assert {"coopt_kv_write", "coopt_paged_decode", "coopt_paged_chunked"} <= set(names)
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in coopt.h but not exported"
        assert name in binding._SIGNATURES, f"{name} has no ctypes signature"
    assert lib.coopt_version() >= 100
    assert binding.status_string(0) == "ok" and "timed out" in binding.status_string(-5)


class _FakeCache:
    """A descriptor without device memory, for the host-only layout functions."""

    def __init__(self, head_dim, dtype, num_blocks=3, num_kv_heads=2):
        self.head_dim, self.dtype, self.num_blocks, self.num_kv_heads = head_dim, dtype, num_blocks, num_kv_heads
        self.desc = binding.coopt_cache(0x1000, num_blocks, num_kv_heads, head_dim, 16, dtype)

    def ref(self):
        return ctypes.byref(self.desc)


@pytest.mark.parametrize("head_dim", [64, 128])
@pytest.mark.parametrize("dtype", [binding.KV_FP8_E4M3, binding.KV_BF16])
def test_layout_is_a_bijection_inside_each_granule(lib, head_dim, dtype):
    c = _FakeCache(head_dim, dtype)
    gran = lib.coopt_granule_bytes(head_dim, dtype)
    esize = 1 if dtype == binding.KV_FP8_E4M3 else 2
    header = 0                                   # the FP8 header sits behind the codes
    assert gran == (128 if dtype == binding.KV_FP8_E4M3 else 0) + 2 * 16 * head_dim * esize
    assert lib.coopt_cache_bytes(3, 2, head_dim, dtype) == 3 * 2 * gran
    for blk, h in [(0, 0), (2, 1)]:
        base = (blk * 2 + h) * gran
        seen = set()
        for w in range(2):
            for t in range(16):
                for d in range(head_dim):
                    off = binding.cache_offset(c, blk, h, w, t, d)
                    assert base + header + w * 16 * head_dim * esize <= off < base + header + (w + 1) * 16 * head_dim * esize
                    assert off % esize == 0
                    seen.add(off)
        assert len(seen) == 2 * 16 * head_dim
        if dtype == binding.KV_FP8_E4M3:
            assert binding.scale_offset(c, blk, h, 0) == base + 32 * head_dim and binding.scale_offset(c, blk, h, 1) == base + 32 * head_dim + 4
    assert binding.cache_offset(c, 3, 0, 0, 0, 0) == -1 and binding.cache_offset(c, 0, 0, 0, 16, 0) == -1
    assert binding.cache_offset(c, 0, 0, 2, 0, 0) == -1 and binding.cache_offset(c, 0, 0, 0, 0, head_dim) == -1


def test_fp8_parts_are_tensor_core_operands_in_place(lib):
    """FP8 granule: both parts are K-major operands made of 8-row x 16-byte core matrices, K with tokens
    as rows (contraction over dims), V transposed with dims as rows (contraction over tokens)."""
    for D in (64, 128):
        c = _FakeCache(D, binding.KV_FP8_E4M3)
        k0 = binding.cache_offset(c, 0, 0, 0, 0, 0)
        v0 = binding.cache_offset(c, 0, 0, 1, 0, 0)
        assert k0 == 0 and v0 == 16 * D and binding.scale_offset(c, 0, 0, 0) == 32 * D
        for t in (0, 5, 8, 15):
            for d in (0, 1, 15, 16, 37, D - 1):
                assert binding.cache_offset(c, 0, 0, 0, t, d) - k0 == (t // 8) * 8 * D + (d // 16) * 128 + (t % 8) * 16 + d % 16
                assert binding.cache_offset(c, 0, 0, 1, t, d) - v0 == (d // 8) * 128 + (d % 8) * 16 + t


def test_bf16_fragment_order_serves_16_byte_loads(lib):
    """bf16 granule: a lane's operands for two k-steps (K) or two n-tiles (V) share one 16-byte chunk."""
    c = _FakeCache(128, binding.KV_BF16)
    for token in (0, 5, 11):
        for quad in range(4):
            dims = [16 * s + 2 * quad + e for s in range(2) for e in (0, 1, 8, 9)]
            offs = [binding.cache_offset(c, 0, 0, 0, token, d) for d in dims]
            assert offs == list(range(offs[0], offs[0] + 16, 2)) and offs[0] % 16 == 0


def test_sizes_and_host_side_argument_checks(lib):
    assert lib.coopt_granule_bytes(96, 0) == 0 and lib.coopt_granule_bytes(128, 7) == 0
    n0 = lib.coopt_workspace_bytes(32, 40, 8, 128, 128, 0, 32)
    n1 = lib.coopt_workspace_bytes(4, 40, 8, 128, 8192, 2048, 4)
    assert n0 > 64 * 1024 and n1 > 4 * 40 * 64 * 130 * 4
    o, m, l, mc = ctypes.c_size_t(), ctypes.c_size_t(), ctypes.c_size_t(), ctypes.c_int32()
    assert lib.coopt_chunk_partials(4, 40, 128, 8192, 2048, ctypes.byref(o), ctypes.byref(m), ctypes.byref(l),
                                    ctypes.byref(mc)) == 0
    assert mc.value == 64 and o.value < m.value < l.value and l.value + 4 * 4 * 40 * 64 <= n1
    assert lib.coopt_chunk_partials(4, 40, 128, 8192, 100, ctypes.byref(o), ctypes.byref(m), ctypes.byref(l),
                                    ctypes.byref(mc)) == -1
    # calls that must be rejected before anything touches a device
    good = binding.coopt_cache(0x1000, 4, 2, 128, 16, 0)
    assert lib.coopt_kv_write(None, None, None, 0, None, 1, None) == -1
    assert lib.coopt_kv_write(ctypes.byref(good), None, None, 256, None, 0, None) == 0      # empty call
    assert lib.coopt_kv_write(ctypes.byref(good), None, None, 256, None, 1, None) == -1
    assert lib.coopt_kv_write(ctypes.byref(good), 0x100, 0x100, 8, 0x100, 1, None) == -1    # stride too small
    bad_dim = binding.coopt_cache(0x1000, 4, 2, 96, 16, 0)
    assert lib.coopt_kv_write(ctypes.byref(bad_dim), 0x100, 0x100, 256, 0x100, 1, None) == -2
    bad_bs = binding.coopt_cache(0x1000, 4, 2, 128, 32, 0)
    assert lib.coopt_kv_write(ctypes.byref(bad_bs), 0x100, 0x100, 256, 0x100, 1, None) == -2
    misaligned = binding.coopt_cache(0x1004, 4, 2, 128, 16, 0)
    assert lib.coopt_kv_write(ctypes.byref(misaligned), 0x100, 0x100, 256, 0x100, 1, None) == -1
    args = (0x100, 0x100, 0x100, 8, 0x100)
    assert lib.coopt_paged_decode(ctypes.byref(good), *args, 2, 7, 0.1, 0x100, 1 << 30, None) == -2    # 7 % 2
    assert lib.coopt_paged_decode(ctypes.byref(good), *args, 2, 32, 0.1, 0x100, 1 << 30, None) == -2   # group 16
    assert lib.coopt_paged_decode(ctypes.byref(good), *args, 2000, 4, 0.1, 0x100, 1 << 30, None) == -2  # batch
    assert lib.coopt_paged_decode(ctypes.byref(good), *args, 2, 4, 0.1, None, 0, None) == -3
    assert lib.coopt_paged_decode(ctypes.byref(good), *args, 2, 4, 0.1, 0x100, 16, None) == -3
    assert lib.coopt_paged_decode(ctypes.byref(good), None, 0x100, 0x100, 8, 0x100, 2, 4, 0.1, 0x100, 1 << 30, None) == -1
    assert lib.coopt_paged_chunked(ctypes.byref(good), 0x100, 0x100, 0x100, 0x100, 8, 0x100, 2, 4, 2, 100, 1, 0.1,
                                   0x100, 1 << 30, None) == -1                                           # chunk % 16
    assert lib.coopt_workspace_init(None, 0, None) == -1 and lib.coopt_workspace_init(0x100, 8, None) == -3
