"""GPU parity: coopt_kv_write against the oracle, bit for bit (codes, scales, untouched bytes)."""
import numpy as np
import pytest
import torch

from oracle import e4m3, kv_cache
from paper_2602_09323_b200 import binding, workloads
from tests import helpers

pytestmark = pytest.mark.gpu


def _compare_fp8(cache, codes, scales, what=""):
    g_codes, g_scales, rest = helpers.cache_to_logical(cache)
    assert np.array_equal(g_scales.view(np.uint32), scales.view(np.uint32)), f"{what}: scales differ"
    bad = np.argwhere(g_codes != codes)
    assert bad.size == 0, f"{what}: {len(bad)} codes differ, first at {bad[0]}: gpu {g_codes[tuple(bad[0])]:#x} oracle {codes[tuple(bad[0])]:#x}"
    assert not rest.any(), f"{what}: header padding not zero"


def test_hardware_encode_matches_oracle_on_every_boundary():
    """Blocks whose scale is exactly 1 (they contain 448): the stored code is the hardware's
    rounding of the value itself.  Values: every representable magnitude, every midpoint and
    its two fp32 neighbours... restricted to what bf16 can express, plus all bf16 values in
    a sweep of exponents."""
    pos = e4m3.DECODE_TABLE[:0x7F]
    mids = (pos[:-1] + pos[1:]) / 2
    vals = np.concatenate([pos, mids, [2.0 ** -10, 2.0 ** -11, 3e-5, 460.0, 464.0, 0.0]])
    hi16 = (np.arange(0x3000, 0x4400, dtype=np.uint32) << 16).view(np.float32)   # bf16 sweep 2^-31 .. 512
    vals = np.concatenate([vals, hi16.astype(np.float64)])
    vals = torch.tensor(vals, dtype=torch.float32).to(torch.bfloat16).float().numpy()
    vals = vals[np.abs(vals) <= 448.0]
    vals = np.concatenate([vals, -vals])
    D, H = 128, 1
    per_block = 16 * D - 1
    nblk = (len(vals) + per_block - 1) // per_block
    flat = np.zeros(nblk * 16 * D, dtype=np.float32)
    for b in range(nblk):
        chunk = vals[b * per_block:(b + 1) * per_block]
        flat[b * 16 * D] = 448.0
        flat[b * 16 * D + 1:b * 16 * D + 1 + len(chunk)] = chunk
    k = torch.from_numpy(flat.reshape(nblk * 16, H, D)).to(torch.bfloat16)
    v = -k
    slots = torch.arange(nblk * 16, dtype=torch.int64)
    cache = binding.Cache(nblk, H, D)
    binding.kv_write(cache, k.cuda(), v.cuda(), slots.cuda())
    codes, scales = kv_cache.new_cache(nblk, H, D)
    kv_cache.kv_write(codes, scales, k.float().numpy(), v.float().numpy(), slots.numpy())
    assert np.all(scales == 1.0)
    _compare_fp8(cache, codes, scales, "encode sweep")


@pytest.mark.parametrize("mode", ["single_shot", "token_by_token", "mixed_calls"])
def test_tiny_config_cache_is_bit_exact(mode):
    w = workloads.config_tiny()
    T = w.k.shape[0]
    calls = {"single_shot": None, "token_by_token": [(i, i + 1) for i in range(T)],
             "mixed_calls": [(0, 5), (5, 17), (17, 30), (30, 31), (31, 200), (200, T)]}[mode]
    cache = helpers.gpu_fill(w, calls=calls)
    codes, scales = helpers.oracle_fp8_cache(w, calls=calls)
    _compare_fp8(cache, codes, scales, mode)


@pytest.mark.parametrize("head_dim,heads", [(64, 3), (128, 8), (128, 5)])
def test_skips_growth_and_block_reuse(head_dim, heads):
    rng = np.random.default_rng(head_dim + heads)
    NB = 6
    cache = binding.Cache(NB, heads, head_dim)
    codes, scales = kv_cache.new_cache(NB, heads, head_dim)
    call_slots = [
        list(range(16, 16 + 5)) + [-1, -1] + list(range(32, 48)) + [-7] + list(range(80, 83)),
        [21], [-1], [22, 23], [83, -1, 84], [85],
        list(range(16, 19)),                       # block 1 again from offset 0: opened anew
        [19, 20], list(range(48, 64)) + list(range(0, 9)),
    ]
    for n, slots in enumerate(call_slots):
        T = len(slots)
        scale_up = 4.0 if n in (1, 4) else (0.05 if n == 5 else 1.0)
        k = torch.from_numpy(rng.standard_normal((T, heads, head_dim)) * scale_up).to(torch.bfloat16)
        v = torch.from_numpy(rng.standard_normal((T, heads, head_dim)) * scale_up).to(torch.bfloat16)
        k[:, :, 3] *= 20
        if n == 3:
            v[:] = 0
        s = torch.tensor(slots, dtype=torch.int64)
        binding.kv_write(cache, k.cuda(), v.cuda(), s.cuda())
        kv_cache.kv_write(codes, scales, k.float().numpy(), v.float().numpy(), s.numpy())
        _compare_fp8(cache, codes, scales, f"call {n}")
    assert not codes[4].any()                       # a block nobody wrote stays zero on both sides


@pytest.mark.parametrize("head_dim", [64, 128])
def test_extreme_magnitudes_divide_exactly(head_dim):
    """Scales from 2^-110 to 2^80 and values down to bf16's subnormals inside one group: the stored
    code is the encoding of the IEEE fp32 quotient x / s whatever route the kernel takes to it.
    Whole blocks and partial groups, first writes and growth with re-expression."""
    rng = np.random.default_rng(7 + head_dim)
    H, NB = 2, 24
    cache = binding.Cache(NB, H, head_dim)
    codes, scales = kv_cache.new_cache(NB, H, head_dim)
    exps = [-118, -60, -41, -40, -39, -12, 0, 9, 30, 31, 32, 70]          # amax of block b is about 2^exps[b % 12]
    for call in range(3):
        slots, ks, vs = [], [], []
        for b in range(NB):
            whole = b % 2 == 0
            offs = list(range(16)) if (whole and call == 0) else ([] if whole else list(range(5 * call, 5 * call + 5)))
            for o in offs:
                slots.append(b * 16 + o)
                mag = 2.0 ** (exps[b % 12] + 2 * call)
                x = rng.standard_normal((2, H, head_dim)) * mag
                spread = 2.0 ** rng.integers(-100, 1, size=x.shape)           # mostly far below the block's amax
                x = np.where(rng.random(x.shape) < 0.5, x * spread, x)
                x.flat[rng.integers(0, x.size, 4)] = 2.0 ** -133              # bf16 subnormal
                x.flat[rng.integers(0, x.size, 2)] = -0.0
                ks.append(x[0]); vs.append(x[1])
        k = torch.from_numpy(np.stack(ks)).to(torch.bfloat16)
        v = torch.from_numpy(np.stack(vs)).to(torch.bfloat16)
        s = torch.tensor(slots, dtype=torch.int64)
        assert torch.isfinite(k.float()).all() and torch.isfinite(v.float()).all()
        binding.kv_write(cache, k.cuda(), v.cuda(), s.cuda())
        kv_cache.kv_write(codes, scales, k.float().numpy(), v.float().numpy(), s.numpy())
        _compare_fp8(cache, codes, scales, f"call {call}")
    assert scales.min() < 2.0 ** -100 and scales.max() > 2.0 ** 60


def test_long_call_of_scattered_and_contiguous_tokens():
    """More tokens than the per-token launch takes: runs of a whole block, runs that straddle the
    tokens one CTA looks at, single tokens in blocks of their own, and skipped tokens between."""
    rng = np.random.default_rng(11)
    H, D, NB = 5, 128, 400
    order = rng.permutation(NB)
    slots = []
    for i, b in enumerate(order):
        kind = i % 4
        if kind == 0: slots += [b * 16 + o for o in range(16)]
        elif kind == 1: slots += [b * 16 + o for o in range(3, 14)] + [-1]
        elif kind == 2: slots += [b * 16 + 7]
        else: slots += [-1, -1] + [b * 16 + o for o in (0, 1, 2)] + [-5] + [b * 16 + o for o in (9, 4)]
    T = len(slots)
    assert T > 512
    k = torch.from_numpy(rng.standard_normal((T, H, D))).to(torch.bfloat16)
    v = torch.from_numpy(rng.standard_normal((T, H, D)) * 3).to(torch.bfloat16)
    s = torch.tensor(slots, dtype=torch.int64)
    cache = binding.Cache(NB, H, D)
    codes, scales = kv_cache.new_cache(NB, H, D)
    for rep in range(2):                       # the second pass meets resident codes and old scales
        kk = k if rep == 0 else (k * 1.5).to(torch.bfloat16)
        binding.kv_write(cache, kk.cuda(), v.cuda(), s.cuda())
        kv_cache.kv_write(codes, scales, kk.float().numpy(), v.float().numpy(), s.numpy())
        _compare_fp8(cache, codes, scales, f"pass {rep}")


def test_strided_token_rows_and_out_of_range_blocks_are_ignored():
    w = workloads.make_workload("strided", [40], 4, 2, 128, seed=3)
    kv = torch.zeros(40, 3, 2, 128, dtype=torch.bfloat16)     # k and v interleaved with padding
    kv[:, 0], kv[:, 2] = w.k, w.v
    kv = kv.cuda()
    cache = binding.Cache(w.num_blocks, 2, 128)
    slots = w.slot_mapping.clone()
    binding.kv_write(cache, kv[:, 0], kv[:, 2], slots.cuda())
    codes, scales = helpers.oracle_fp8_cache(w)
    _compare_fp8(cache, codes, scales, "strided")
    before = cache.data.clone()
    far = torch.tensor([w.num_blocks * 16 + 3], dtype=torch.int64).cuda()
    binding.kv_write(cache, kv[:1, 0], kv[:1, 2], far)
    torch.cuda.synchronize()
    assert torch.equal(before, cache.data)


def test_bf16_ablation_cache_matches_oracle():
    w = workloads.make_workload("bf16", [17, 300], 8, 8, 64, seed=1)
    cache = helpers.gpu_fill(w, dtype=binding.KV_BF16)
    vals = kv_cache.new_cache_bf16(w.num_blocks, 8, 64)
    kv_cache.kv_write_bf16(vals, w.k.float().numpy(), w.v.float().numpy(), w.slot_mapping.numpy())
    got = helpers.cache_to_logical(cache)
    assert np.array_equal(got.view(np.uint32), vals.view(np.uint32))


def test_llama13b_shape_bulk_fill_sampled_blocks():
    """Full-size cache of the LLaMA-13B decode configuration; the oracle recomputes a sample of
    (sequence, kv head) pairs in full and those granules must match bit for bit."""
    w = workloads.config_llama13b_decode(batch=32, context=2048)
    cache = helpers.gpu_fill(w)
    g_codes, g_scales, _ = helpers.cache_to_logical(cache)
    rng = np.random.default_rng(0)
    k, v, slots = w.k.float().numpy(), w.v.float().numpy(), w.slot_mapping.numpy()
    for b, h in zip(rng.integers(0, 32, 6), rng.integers(0, 8, 6)):
        rows = slice(w.kv_offsets[b], w.kv_offsets[b] + 2048)
        codes, scales = kv_cache.new_cache(w.num_blocks, 8, 128)
        kv_cache.kv_write(codes, scales, k[rows], v[rows], slots[rows], heads=[h])
        blks = w.block_table[b, :128].numpy()
        assert np.array_equal(g_codes[blks, h], codes[blks, h]) and np.array_equal(g_scales[blks, h], scales[blks, h])
