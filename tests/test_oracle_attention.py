"""Pins for the oracle's float64 attention (CPU only): a pure-Python triple loop, the
library routine it must reduce to, closed-form special cases and the method's invariants."""
import math

import numpy as np
import pytest
import torch

from oracle import attention, kv_cache
from paper_2602_09323_b200 import workloads


def _fp8_cache(w):
    codes, scales = kv_cache.new_cache(w.num_blocks, w.num_kv_heads, w.head_dim)
    kv_cache.kv_write(codes, scales, w.k.float().numpy(), w.v.float().numpy(), w.slot_mapping.numpy())
    return codes, scales


def _small(seed=0, lens=(5, 37), hq=4, hkv=2, d=8, q_lens=None):
    return workloads.make_workload("small", list(lens), hq, hkv, d, seed=seed, q_lens=q_lens)


def _brute_force(w, deq, causal=True):
    """Triple loop in plain Python floats: no numpy reductions, no shared helper."""
    q = w.q.float().numpy().astype(float)
    table = w.block_table.numpy()
    cu = w.cu_q_lens.numpy()
    G = w.num_q_heads // w.num_kv_heads
    out = np.zeros(q.shape)
    scale = 1.0 / math.sqrt(w.head_dim)
    for b, L in enumerate(w.context_lens):
        n = cu[b + 1] - cu[b]
        for i in range(n):
            r = cu[b] + i
            last = L - n + i if causal else L - 1
            for h in range(w.num_q_heads):
                g = h // G
                logits = []
                for j in range(last + 1):
                    blk, off = int(table[b, j // 16]), j % 16
                    s = 0.0
                    for d in range(w.head_dim):
                        s += q[r, h, d] * float(deq[blk, g, 0, off, d])
                    logits.append(s * scale)
                top = max(logits)
                weights = [math.exp(s - top) for s in logits]
                total = sum(weights)
                for d in range(w.head_dim):
                    acc = 0.0
                    for j in range(last + 1):
                        blk, off = int(table[b, j // 16]), j % 16
                        acc += weights[j] * float(deq[blk, g, 1, off, d])
                    out[r, h, d] = acc / total
    return out


def test_decode_matches_pure_python_triple_loop():
    w = _small()
    codes, scales = _fp8_cache(w)
    deq = kv_cache.dequantise(codes, scales)
    got = attention.paged_attention(w.q.float().numpy(), (codes, scales), w.block_table.numpy(), w.context_lens)
    assert np.allclose(got, _brute_force(w, deq), rtol=0, atol=1e-11)
    also = attention.paged_attention(w.q.float().numpy(), deq, w.block_table.numpy(), w.context_lens)
    assert np.array_equal(got, also)


def test_causal_prefill_matches_pure_python_triple_loop():
    w = _small(seed=1, lens=(9, 30), q_lens=(4, 7))
    codes, scales = _fp8_cache(w)
    deq = kv_cache.dequantise(codes, scales)
    got = attention.paged_attention(w.q.float().numpy(), deq, w.block_table.numpy(), w.context_lens,
                                    cu_q_lens=w.cu_q_lens.numpy(), causal=True)
    assert np.allclose(got, _brute_force(w, deq, causal=True), rtol=0, atol=1e-11)
    full = attention.paged_attention(w.q.float().numpy(), deq, w.block_table.numpy(), w.context_lens,
                                     cu_q_lens=w.cu_q_lens.numpy(), causal=False)
    assert np.allclose(full, _brute_force(w, deq, causal=False), rtol=0, atol=1e-11)


def test_mha_case_equals_torch_sdpa_float64_on_gathered_tensors():
    w = workloads.make_workload("mha", [50, 33], 4, 4, 16, seed=2)
    codes, scales = _fp8_cache(w)
    deq = kv_cache.dequantise(codes, scales)
    got = attention.paged_attention(w.q.float().numpy(), deq, w.block_table.numpy(), w.context_lens)
    for b, L in enumerate(w.context_lens):
        pos = np.arange(L)
        blk = w.block_table[b].numpy()[pos // 16]
        K = torch.from_numpy(deq[blk, :, 0, pos % 16, :]).permute(1, 0, 2)      # [H, L, D]
        V = torch.from_numpy(deq[blk, :, 1, pos % 16, :]).permute(1, 0, 2)
        Q = w.q[b].double().unsqueeze(1)                                         # [H, 1, D]
        want = torch.nn.functional.scaled_dot_product_attention(Q, K, V).squeeze(1).numpy()
        assert np.allclose(got[b], want, rtol=0, atol=1e-11)


def test_gqa_equals_mha_over_a_cache_with_repeated_kv_heads():
    w = _small(seed=3, lens=(20, 70), hq=6, hkv=2, d=8)
    codes, scales = _fp8_cache(w)
    deq = kv_cache.dequantise(codes, scales)
    G = 3
    expanded = np.repeat(deq, G, axis=1)                       # kv head g serves query heads g*G..g*G+G-1
    a = attention.paged_attention(w.q.float().numpy(), deq, w.block_table.numpy(), w.context_lens)
    b = attention.paged_attention(w.q.float().numpy(), expanded, w.block_table.numpy(), w.context_lens)
    assert np.array_equal(a, b)
    wrong = np.repeat(deq, G, axis=1)[:, ::-1]                 # a wrong head mapping must differ
    c = attention.paged_attention(w.q.float().numpy(), wrong, w.block_table.numpy(), w.context_lens)
    assert np.abs(a - c).max() > 1e-3


def test_block_table_permutation_invariance():
    w = _small(seed=4, lens=(33, 64, 100))
    codes, scales = _fp8_cache(w)
    base = attention.paged_attention(w.q.float().numpy(), (codes, scales), w.block_table.numpy(), w.context_lens)
    rng = np.random.default_rng(0)
    perm = rng.permutation(w.num_blocks)                        # new id of old block i is perm[i]
    codes2, scales2 = np.empty_like(codes), np.empty_like(scales)
    codes2[perm], scales2[perm] = codes, scales
    table2 = w.block_table.numpy().copy()
    valid = table2 >= 0
    table2[valid] = perm[table2[valid]]
    moved = attention.paged_attention(w.q.float().numpy(), (codes2, scales2), table2, w.context_lens)
    assert np.array_equal(base, moved)


@pytest.mark.parametrize("chunk", [16, 48, 64, 4096])
def test_chunked_equals_unchunked(chunk):
    w = _small(seed=5, lens=(1, 17, 200, 333))
    codes, scales = _fp8_cache(w)
    q = w.q.float().numpy()
    base = attention.paged_attention(q, (codes, scales), w.block_table.numpy(), w.context_lens)
    got, partials = attention.paged_attention_chunked(q, (codes, scales), w.block_table.numpy(),
                                                      w.context_lens, chunk)
    assert np.allclose(got, base, rtol=0, atol=1e-12)
    m, l, o = partials[(3, 0)]
    assert len(m) == (333 + chunk - 1) // chunk and np.all(l >= 1.0)


def test_merge_ignores_empty_chunks_and_is_shift_invariant():
    rng = np.random.default_rng(6)
    m = rng.standard_normal(5) * 30
    l = rng.uniform(1, 9, 5)
    o = rng.standard_normal((5, 4))
    base = attention.merge_partials(m, l, o)
    m2 = np.concatenate([m, [-np.inf]])
    l2 = np.concatenate([l, [0.0]])
    o2 = np.concatenate([o, np.full((1, 4), 7.0)])
    assert np.allclose(attention.merge_partials(m2, l2, o2), base, atol=1e-14)
    assert np.allclose(attention.merge_partials(m + 100.0, l, o), base, atol=1e-13)
    w = l * np.exp(m)
    assert np.allclose(base, (w / w.sum()) @ o, atol=1e-12)     # the unshifted definition


def test_closed_form_special_cases():
    # one cached token: the output is that token's V
    w = _small(seed=7, lens=(1,), hq=2, hkv=1, d=8)
    codes, scales = _fp8_cache(w)
    deq = kv_cache.dequantise(codes, scales)
    out = attention.paged_attention(w.q.float().numpy(), deq, w.block_table.numpy(), w.context_lens)
    blk = int(w.block_table[0, 0])
    assert np.allclose(out[0, 0], deq[blk, 0, 1, 0]) and np.allclose(out[0, 1], deq[blk, 0, 1, 0])
    # identical keys: the output is the mean of V
    w = _small(seed=8, lens=(40,), hq=2, hkv=1, d=8)
    w.k[:] = w.k[0:1]
    codes, scales = _fp8_cache(w)
    deq = kv_cache.dequantise(codes, scales)
    out = attention.paged_attention(w.q.float().numpy(), deq, w.block_table.numpy(), w.context_lens)
    pos = np.arange(40)
    V = deq[w.block_table[0].numpy()[pos // 16], 0, 1, pos % 16]
    assert np.allclose(out[0, 0], V.mean(axis=0), atol=1e-12)
    # empty context: zeros
    w = _small(seed=9, lens=(0, 5))
    codes, scales = _fp8_cache(w)
    out = attention.paged_attention(w.q.float().numpy(), (codes, scales), w.block_table.numpy(), w.context_lens)
    assert not out[0].any() and np.isfinite(out[1]).all()


def test_causal_row_equals_decode_with_truncated_context():
    w = _small(seed=10, lens=(45,), q_lens=(6,))
    codes, scales = _fp8_cache(w)
    q = w.q.float().numpy()
    full = attention.paged_attention(q, (codes, scales), w.block_table.numpy(), w.context_lens,
                                     cu_q_lens=w.cu_q_lens.numpy(), causal=True)
    for i in range(6):
        dec = attention.paged_attention(q[i:i + 1], (codes, scales), w.block_table.numpy(), [45 - 6 + i + 1])
        assert np.array_equal(full[i], dec[0])


def test_sm_scale_and_tail_masking_matter():
    """Planted-mistake check: dropping 1/sqrt(d) or reading past the context must change
    the result by far more than the parity tolerance."""
    w = _small(seed=11, lens=(21,))
    codes, scales = _fp8_cache(w)
    q = w.q.float().numpy()
    good = attention.paged_attention(q, (codes, scales), w.block_table.numpy(), w.context_lens)
    no_scale = attention.paged_attention(q, (codes, scales), w.block_table.numpy(), w.context_lens, sm_scale=1.0)
    assert np.abs(good - no_scale).max() > 0.05
    shorter = attention.paged_attention(q, (codes, scales), w.block_table.numpy(), [20])
    assert np.abs(good - shorter).max() > 1e-4


def test_sample_pairs_only():
    w = _small(seed=12, lens=(30, 31))
    codes, scales = _fp8_cache(w)
    q = w.q.float().numpy()
    full = attention.paged_attention(q, (codes, scales), w.block_table.numpy(), w.context_lens)
    part = attention.paged_attention(q, (codes, scales), w.block_table.numpy(), w.context_lens,
                                     pairs=[(1, 3)])
    assert np.array_equal(part[1, 3], full[1, 3]) and np.isnan(part[0]).all()
