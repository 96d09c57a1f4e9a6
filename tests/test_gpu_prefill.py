"""GPU parity: coopt_paged_chunked with runs of several query tokens per sequence (chunked prefill on
tensor cores) against the float64 oracle evaluated on the oracle's own cache."""
import numpy as np
import pytest
import torch

from oracle import attention, kv_cache
from paper_2602_09323_b200 import binding, workloads
from tests import helpers

pytestmark = pytest.mark.gpu


def _gpu_prefill(w, cache, causal=True):
    ws = binding.new_workspace(w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.block_table.shape[1], 2048,
                               sum(w.q_lens))
    out = binding.paged_chunked(cache, w.q.cuda(), w.cu_q_lens.cuda(), w.block_table.cuda(),
                                w.context_lens_tensor.cuda(), 2048, causal, w.sm_scale, ws)
    torch.cuda.synchronize()
    assert binding.workspace_status(ws) == 0
    return out


def _oracle(w, causal=True, pairs=None):
    codes, scales = helpers.oracle_fp8_cache(w)
    return attention.paged_attention(w.q.float().numpy(), (codes, scales), w.block_table.numpy(), w.context_lens,
                                     cu_q_lens=w.cu_q_lens.numpy(), causal=causal, pairs=pairs)


@pytest.mark.parametrize("hq,hkv,d", [(8, 2, 64), (10, 2, 128), (8, 8, 128), (16, 2, 64), (3, 1, 128)])
@pytest.mark.parametrize("causal", [True, False])
def test_ragged_query_runs_group_sizes_and_head_dims(hq, hkv, d, causal):
    lens = [70, 333, 16, 129, 1, 200]
    q_lens = [70, 40, 3, 129, 1, 7]          # whole-sequence prefill, partial runs, single tokens
    w = workloads.make_workload("prefill", lens, hq, hkv, d, seed=hq + d, q_lens=q_lens)
    out = _gpu_prefill(w, helpers.gpu_fill(w), causal)
    helpers.check_attention(out, _oracle(w, causal), what=f"prefill hq{hq} hkv{hkv} d{d} causal={causal}")


def test_rows_past_the_tile_and_tail_positions_are_left_alone():
    w = workloads.make_workload("guard", [500, 77], 10, 2, 128, seed=4, q_lens=[130, 77])
    cache = helpers.gpu_fill(w)
    want = _gpu_prefill(w, cache)
    total = sum(w.q_lens)
    padded = torch.full((total + 2, 10, 128), 7.0, dtype=torch.bfloat16, device="cuda")
    ws = binding.new_workspace(w.batch, 10, 2, 128, w.block_table.shape[1], 2048, total)
    binding.paged_chunked(cache, w.q.cuda(), w.cu_q_lens.cuda(), w.block_table.cuda(), w.context_lens_tensor.cuda(),
                          2048, True, w.sm_scale, ws, out=padded[1:-1])
    torch.cuda.synchronize()
    assert torch.equal(padded[1:-1], want) and (padded[0] == 7).all() and (padded[-1] == 7).all()


def test_causal_row_equals_decode_over_the_truncated_context():
    """Row i of a causal run sees exactly what a decode call with context L - n + i + 1 sees."""
    L, n = 300, 37
    w = workloads.make_workload("rowdec", [L], 8, 2, 128, seed=11, q_lens=[n])
    cache = helpers.gpu_fill(w)
    out = _gpu_prefill(w, cache)
    ws = binding.new_workspace(1, 8, 2, 128, w.block_table.shape[1])
    for i in (0, 5, n - 1):
        lens = torch.tensor([L - n + i + 1], dtype=torch.int32).cuda()
        dec = binding.paged_decode(cache, w.q[i:i + 1].cuda(), w.block_table.cuda(), lens, w.sm_scale, ws)
        torch.cuda.synchronize()
        diff = (dec[0].float() - out[i].float()).abs()
        assert float((diff - 2.0 ** -7 * out[i].float().abs()).max()) <= 5e-3


@pytest.mark.parametrize("plain", [False, True])
def test_chunked_prefill_full_size(plain):
    """The chunked-prefill configuration at full size: 8 sequences, 4096 cached + 512 new tokens, causal.  The whole
    device cache against the oracle's bit for bit; every query row and head of one (sequence, kv head) group,
    and for every sequence and kv head the rows on both sides of every boundary between the kernel's tiles of
    25 query tokens (plus the first and the last row), for one query head of the group."""
    w = workloads.config_chunked_prefill(v_outliers=not plain)
    cache = helpers.gpu_fill(w)
    out = _gpu_prefill(w, cache)
    assert torch.isfinite(out.float()).all()
    heads = [0, 5] if plain else None
    codes, scales = helpers.oracle_fp8_cache(w, heads=heads)
    helpers.check_cache_bit_exact(cache, codes, scales, heads=heads, what="chunked prefill")
    kv_heads = heads or range(8)
    full_b, full_g = 3, 5
    pairs = {(full_b * 512 + i, h) for i in range(512) for h in range(full_g * 5, full_g * 5 + 5)}
    edge_rows = sorted({0, 511} | {i for i in range(512) if i % 25 in (0, 24)})
    for b in range(8):
        for g in kv_heads:
            pairs |= {(b * 512 + i, g * 5 + (b + g) % 5) for i in edge_rows}
    ref = attention.paged_attention(w.q.float().numpy(), (codes, scales), w.block_table.numpy(), w.context_lens,
                                    cu_q_lens=w.cu_q_lens.numpy(), causal=True, pairs=sorted(pairs))
    helpers.check_attention(out, ref, plain=plain, what="chunked prefill full size")


@pytest.mark.parametrize("hq,hkv", [(16, 2), (12, 2), (4, 4)])
def test_group_sizes_up_to_eight_on_the_tensor_memory_kernel(hq, hkv):
    """head_dim 128 with G = 8, 6 and 1: 16, 21 and 128 query tokens per 128-row tile, tiles that end in the
    middle of a cache block, a sequence that is all new tokens and one with a single new token."""
    lens = [513, 300, 129, 47, 1024]
    q_lens = [200, 300, 1, 20, 33]
    w = workloads.make_workload("prefill_g", lens, hq, hkv, 128, seed=3 * hq + hkv, q_lens=q_lens)
    out = _gpu_prefill(w, helpers.gpu_fill(w))
    helpers.check_attention(out, _oracle(w), what=f"prefill hq{hq} hkv{hkv}")


def test_long_context_prefill_many_tiles_and_block_batches():
    """A 40,000-token context (2,500 blocks, 313 tiles of 128 keys, 79 batches of block ids) behind 96 new
    tokens: the copy ring wraps many times in both walks; sampled rows against the oracle."""
    L, n = 40000, 96
    w = workloads.make_workload("prefill_long", [L, 700], 10, 2, 128, seed=29, q_lens=[n, 50])
    out = _gpu_prefill(w, helpers.gpu_fill(w))
    assert torch.isfinite(out.float()).all()
    pairs = [(r, h) for r in (0, 1, 50, n - 1, n, n + 49) for h in (0, 4, 5, 9)]
    ref = _oracle(w, pairs=pairs)
    helpers.check_attention(out, ref, what="long prefill")


def test_prefill_twice_is_bitwise_identical_and_all_zero_v_blocks_are_handled():
    """Blocks whose V values are all zero (scale 0) still take part in the softmax; two runs give the same bits."""
    w = workloads.make_workload("prefill_zero_v", [400, 90], 10, 2, 128, seed=31, q_lens=[60, 90])
    w.v[16:48] = 0                      # two whole blocks of the first sequence
    w.v[400 + 32:400 + 48] = 0          # one block of the second
    cache = helpers.gpu_fill(w)
    out1 = _gpu_prefill(w, cache)
    out2 = _gpu_prefill(w, cache)
    assert torch.equal(out1, out2)
    helpers.check_attention(out1, _oracle(w), what="prefill zero v")
