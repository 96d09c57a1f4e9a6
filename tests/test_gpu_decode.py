"""GPU parity: coopt_paged_decode / coopt_paged_chunked (one query token per sequence) against
the float64 oracle evaluated on the oracle's own cache."""
import numpy as np
import pytest
import torch

from oracle import attention, kv_cache
from paper_2602_09323_b200 import binding, workloads
from tests import helpers

pytestmark = pytest.mark.gpu


def _oracle_out(w, calls=None, pairs=None):
    codes, scales = helpers.oracle_fp8_cache(w, calls=calls)
    return attention.paged_attention(w.q.float().numpy(), (codes, scales), w.block_table.numpy(),
                                     w.context_lens, pairs=pairs)


@pytest.mark.parametrize("mode", ["single_shot", "token_by_token"])
def test_tiny_config(mode):
    w = workloads.config_tiny()
    calls = None if mode == "single_shot" else [(i, i + 1) for i in range(w.k.shape[0])]
    cache = helpers.gpu_fill(w, calls=calls)
    out, _ = helpers.gpu_decode(w, cache)
    helpers.check_attention(out, _oracle_out(w, calls), what=f"tiny/{mode}")


def test_tiny_config_without_v_outliers_meets_the_plain_bound():
    w = workloads.config_tiny(v_outliers=False)
    out, _ = helpers.gpu_decode(w, helpers.gpu_fill(w))
    helpers.check_attention(out, _oracle_out(w), plain=True, what="tiny/plain")


@pytest.mark.parametrize("hq,hkv,d", [(8, 8, 64), (4, 2, 128), (8, 2, 128), (10, 2, 128), (16, 2, 64), (5, 1, 128)])
@pytest.mark.parametrize("lens", [(1, 16, 17, 0, 333), (700, 15, 2000)])
def test_group_sizes_head_dims_and_ragged_lengths(hq, hkv, d, lens):
    w = workloads.make_workload("shapes", list(lens), hq, hkv, d, seed=hq * 100 + d)
    out, _ = helpers.gpu_decode(w, helpers.gpu_fill(w))
    ref = _oracle_out(w)
    helpers.check_attention(out, ref, what=f"hq{hq} hkv{hkv} d{d}")
    for b, L in enumerate(lens):
        if L == 0:
            assert not out[b].any()


def test_many_short_sequences_cross_segment_and_round_limits():
    lens = [int(x) for x in np.random.default_rng(0).integers(1, 80, 200)]
    w = workloads.make_workload("short", lens, 8, 2, 64, seed=5)
    out, _ = helpers.gpu_decode(w, helpers.gpu_fill(w))
    helpers.check_attention(out, _oracle_out(w), what="short")


def test_one_long_sequence_is_split_across_the_whole_gpu():
    w = workloads.make_workload("long", [40000], 8, 1, 128, seed=6)
    out, _ = helpers.gpu_decode(w, helpers.gpu_fill(w))
    helpers.check_attention(out, _oracle_out(w), what="long")


def test_bf16_cache_mha_ablation_small():
    w = workloads.make_workload("mha", [300, 17, 1025], 8, 8, 128, seed=7)
    cache = helpers.gpu_fill(w, dtype=binding.KV_BF16)
    vals = kv_cache.new_cache_bf16(w.num_blocks, 8, 128)
    kv_cache.kv_write_bf16(vals, w.k.float().numpy(), w.v.float().numpy(), w.slot_mapping.numpy())
    ref = attention.paged_attention(w.q.float().numpy(), vals, w.block_table.numpy(), w.context_lens)
    out, _ = helpers.gpu_decode(w, cache)
    helpers.check_attention(out, ref, what="bf16 mha")


def test_block_permutation_invariance_determinism_and_guard_bytes():
    w = workloads.make_workload("perm", [257, 90], 10, 2, 128, seed=8)
    cache = helpers.gpu_fill(w)
    out1, ws = helpers.gpu_decode(w, cache)
    out2, _ = helpers.gpu_decode(w, cache)
    assert torch.equal(out1, out2)                         # run-to-run bitwise determinism
    # move every physical block somewhere else: same logical content, same result
    perm = torch.randperm(w.num_blocks, generator=torch.Generator().manual_seed(1))
    moved = binding.Cache(w.num_blocks, 2, 128)
    gran = cache.granule_bytes * 2
    moved.data.view(w.num_blocks, gran)[perm.cuda()] = cache.data.view(w.num_blocks, gran)
    table = w.block_table.clone()
    table[table >= 0] = perm[table[table >= 0].long()].int()
    w2 = workloads.Workload(**{**w.__dict__, "block_table": table})
    out3, _ = helpers.gpu_decode(w2, moved)
    assert torch.equal(out1, out3)
    # guard bytes around the output are left alone
    padded = torch.full((w.batch + 2, 10, 128), 7.0, dtype=torch.bfloat16, device="cuda")
    binding.paged_decode(cache, w.q.cuda(), w.block_table.cuda(), w.context_lens_tensor.cuda(), w.sm_scale, ws,
                         out=padded[1:-1])
    torch.cuda.synchronize()
    assert torch.equal(padded[1:-1], out1) and (padded[0] == 7).all() and (padded[-1] == 7).all()


def test_cold_l2_and_poisoned_workspace_do_not_change_the_result():
    """Timing must not matter: evict L2 before the call (all loads come from HBM, so the copy ring runs
    dry and the roles of the kernel meet in a different order) and fill the partials area of the
    workspace with NaN patterns (a piece that is merged before it was written would show)."""
    w = workloads.make_workload("cold", [700, 15, 2000], 8, 8, 64, seed=0)
    cache = helpers.gpu_fill(w)
    ref = _oracle_out(w)
    q, table, lens = w.q.cuda(), w.block_table.cuda(), w.context_lens_tensor.cuda()
    outs = []
    for rep in range(3):
        n = binding.workspace_bytes(w.batch, 8, 8, 64, w.block_table.shape[1])
        ws = torch.empty(n, dtype=torch.uint8, device="cuda")
        ws.view(torch.int32)[:] = 0x7FC00000
        binding.workspace_init(ws)
        junk = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
        junk.fill_(rep)                                    # larger than L2: evicts the cache and the queries
        del junk
        out = binding.paged_decode(cache, q, table, lens, w.sm_scale, ws)
        torch.cuda.synchronize()
        assert binding.workspace_status(ws) == 0
        helpers.check_attention(out, ref, what=f"cold rep {rep}")
        outs.append(out)
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2])


PLAIN_HEADS = [0, 5]      # kv heads of the outlier-free runs (all sequences, all query heads of these groups)


def _pairs_of_heads(batch, group, kv_heads):
    return [(b, h) for b in range(batch) for g in kv_heads for h in range(g * group, (g + 1) * group)]


def test_llama13b_decode_full_size_every_output():
    """The LLaMA-13B-shaped decode configuration at full size, in the launch configuration the benchmark times: the whole
    device cache against the oracle's bit for bit, and every (sequence, query head) output."""
    w = workloads.config_llama13b_decode()
    cache = helpers.gpu_fill(w)
    out, _ = helpers.gpu_decode(w, cache)
    codes, scales = helpers.oracle_fp8_cache(w)
    helpers.check_cache_bit_exact(cache, codes, scales, what="llama13b decode")
    ref = attention.paged_attention(w.q.float().numpy(), (codes, scales), w.block_table.numpy(), w.context_lens)
    helpers.check_attention(out, ref, what="llama13b decode")


def test_llama13b_decode_full_size_without_v_outliers_meets_the_plain_bound():
    w = workloads.config_llama13b_decode(v_outliers=False)
    cache = helpers.gpu_fill(w)
    out, _ = helpers.gpu_decode(w, cache)
    codes, scales = helpers.oracle_fp8_cache(w, heads=PLAIN_HEADS)
    helpers.check_cache_bit_exact(cache, codes, scales, heads=PLAIN_HEADS, what="llama13b decode / plain")
    ref = attention.paged_attention(w.q.float().numpy(), (codes, scales), w.block_table.numpy(), w.context_lens,
                                    pairs=_pairs_of_heads(w.batch, 5, PLAIN_HEADS))
    helpers.check_attention(out, ref, plain=True, what="llama13b decode / plain")
    assert torch.isfinite(out.float()).all()


def test_llama13b_mha_ablation_full_size_every_output():
    """The ablation of the LLaMA-13B-shaped decode configuration at full size: 40 KV heads (one per query head) and a bf16 cache.
    The oracle's un-quantised write and float64 attention, eight heads at a time to bound host memory."""
    w = workloads.config_llama13b_mha_ablation()
    cache = helpers.gpu_fill(w, dtype=binding.KV_BF16)
    out, _ = helpers.gpu_decode(w, cache)
    k, v, q = w.k.float().numpy(), w.v.float().numpy(), w.q.float().numpy()
    slots, table = w.slot_mapping.numpy(), w.block_table.numpy()
    ref = np.empty((w.batch, 40, 128))
    for h0 in range(0, 40, 8):
        vals = kv_cache.new_cache_bf16(w.num_blocks, 8, 128)
        kv_cache.kv_write_bf16(vals, k[:, h0:h0 + 8], v[:, h0:h0 + 8], slots)
        g_vals = helpers.cache_to_logical(cache, heads=slice(h0, h0 + 8))
        assert np.array_equal(g_vals.view(np.uint32), vals.view(np.uint32)), "bf16 cache differs"
        ref[:, h0:h0 + 8] = attention.paged_attention(q[:, h0:h0 + 8], vals, table, w.context_lens)
    helpers.check_attention(out, ref, what="llama13b mha ablation")


@pytest.mark.parametrize("chunk", [16, 64, 2048])
def test_chunked_decode_partials_and_merge(chunk):
    w = workloads.make_workload("chunked", [1, 100, 777, 2049], 10, 2, 128, seed=9)
    cache = helpers.gpu_fill(w)
    out, ws = helpers.gpu_decode(w, cache, chunk_size=chunk)
    codes, scales = helpers.oracle_fp8_cache(w)
    ref, partials = attention.paged_attention_chunked(w.q.float().numpy(), (codes, scales), w.block_table.numpy(),
                                                      w.context_lens, chunk)
    helpers.check_attention(out, ref, what=f"chunk {chunk}")
    o_c, m_c, l_c = binding.chunk_partials(ws, w.batch, 10, 128, w.block_table.shape[1], chunk)
    for (b, h), (m, l, o) in partials.items():
        n = len(m)
        assert np.allclose(m_c[b, h, :n].cpu().numpy(), m, rtol=1e-4, atol=1e-3)
        assert np.allclose(l_c[b, h, :n].cpu().numpy(), l, rtol=5e-3, atol=1e-4)
        assert np.allclose(o_c[b, h, :n].cpu().numpy(), o, rtol=5e-3, atol=2e-2)


@pytest.mark.parametrize("lens,hq,hkv", [([100000], 2, 1), ([640] * 220 + [37, 1300], 2, 1), ([3000] * 70, 4, 2)])
def test_chunked_decode_runs_that_span_planning_rounds(lens, hq, hkv):
    """Chunks of one block: a CTA holds more chunks of one (sequence, kv head) than one planning round
    lists, so the run it merges on chip is parked in the workspace between rounds, both for runs that
    are one piece of their sequence and for runs that cover their sequence whole.  Run twice on the same
    workspace: the piece counters must have been left ready."""
    w = workloads.make_workload("rounds", lens, hq, hkv, 64, seed=21)
    cache = helpers.gpu_fill(w)
    ref = _oracle_out(w)
    ws = binding.new_workspace(w.batch, hq, hkv, 64, w.block_table.shape[1], 16, w.batch)
    q, table, lens_t, cu = w.q.cuda(), w.block_table.cuda(), w.context_lens_tensor.cuda(), w.cu_q_lens.cuda()
    for rep in range(2):
        out = binding.paged_chunked(cache, q, cu, table, lens_t, 16, True, w.sm_scale, ws)
        torch.cuda.synchronize()
        assert binding.workspace_status(ws) == 0
        helpers.check_attention(out, ref, what=f"rounds rep {rep}")


def test_decode_step_equals_write_then_decode_bit_for_bit():
    """Token by token over the last 40 positions of every sequence, the one-call step and the two
    separate calls must leave identical cache bytes and identical outputs, and the outputs must match
    the oracle at the end."""
    w = workloads.make_workload("step", [300, 64, 2048, 1500, 47, 900], 10, 2, 128, seed=17)
    rows = np.concatenate([np.arange(w.kv_offsets[b], w.kv_offsets[b] + L - 40) for b, L in enumerate(w.context_lens)])
    rows_t = torch.from_numpy(rows).cuda()
    k, v, slots = w.k.cuda(), w.v.cuda(), w.slot_mapping.cuda()
    table, q = w.block_table.cuda(), w.q.cuda()
    caches = []
    for _ in range(2):
        c = binding.Cache(w.num_blocks, 2, 128)
        binding.kv_write(c, k[rows_t], v[rows_t], slots[rows_t])
        caches.append(c)
    ws = [binding.new_workspace(w.batch, 10, 2, 128, w.block_table.shape[1]) for _ in range(2)]
    outs = [None, None]
    for step in range(40):
        new = torch.tensor([w.kv_offsets[b] + L - 40 + step for b, L in enumerate(w.context_lens)]).cuda()
        lens = torch.tensor([L - 40 + step + 1 for L in w.context_lens], dtype=torch.int32).cuda()
        k_new, v_new, s_new = k[new].contiguous(), v[new].contiguous(), slots[new].contiguous()
        outs[0] = binding.decode_step(caches[0], k_new, v_new, s_new, q, table, lens, w.sm_scale, ws[0])
        binding.kv_write(caches[1], k_new, v_new, s_new)
        outs[1] = binding.paged_decode(caches[1], q, table, lens, w.sm_scale, ws[1])
        torch.cuda.synchronize()
        assert binding.workspace_status(ws[0]) == 0 and binding.workspace_status(ws[1]) == 0
        assert torch.equal(outs[0], outs[1]), f"step {step}: outputs differ"
        assert torch.equal(caches[0].data, caches[1].data), f"step {step}: cache bytes differ"
    # the oracle fills the same way: the history of every sequence in one call, then 40 single-token calls
    codes, scales = kv_cache.new_cache(w.num_blocks, 2, 128)
    kf, vf, sf = w.k.float().numpy(), w.v.float().numpy(), w.slot_mapping.numpy()
    kv_cache.kv_write(codes, scales, kf[rows], vf[rows], sf[rows])
    for step in range(40):
        new = np.array([w.kv_offsets[b] + L - 40 + step for b, L in enumerate(w.context_lens)])
        kv_cache.kv_write(codes, scales, kf[new], vf[new], sf[new])
    ref = attention.paged_attention(w.q.float().numpy(), (codes, scales), w.block_table.numpy(), w.context_lens)
    helpers.check_attention(outs[0], ref, what="decode step")


def _serving_step_calls(w):
    """Row indices of the two writes of a serving step: the history of every sequence, then its last token."""
    last = np.array([w.kv_offsets[b] + L - 1 for b, L in enumerate(w.context_lens)])
    hist = np.ones(w.k.shape[0], dtype=bool)
    hist[last] = False
    return [np.nonzero(hist)[0], last]


@pytest.mark.parametrize("plain", [False, True])
def test_mixed_length_serving_step_full_size_every_output(plain):
    """The mixed-length serving configuration at full size: 64 sequences with contexts uniform in [128, 8192]; the history is
    filled in bulk, then one token per sequence is appended with coopt_kv_write (which may grow a block's
    scale and re-express its resident codes) and the decode runs over the updated cache.  The oracle replays
    the same two writes; the whole cache is compared bit for bit and every output within the tolerance
    (the outlier-free variant, on two kv heads, against the plain bound)."""
    w = workloads.config_mixed_serving(v_outliers=not plain)
    calls = _serving_step_calls(w)
    heads = PLAIN_HEADS if plain else None
    cache = helpers.gpu_fill(w, calls=calls)
    out, _ = helpers.gpu_decode(w, cache)
    assert torch.isfinite(out.float()).all()
    codes, scales = helpers.oracle_fp8_cache(w, calls=calls, heads=heads)
    helpers.check_cache_bit_exact(cache, codes, scales, heads=heads, what="mixed serving step")
    pairs = _pairs_of_heads(w.batch, 5, PLAIN_HEADS) if plain else None
    ref = attention.paged_attention(w.q.float().numpy(), (codes, scales), w.block_table.numpy(), w.context_lens, pairs=pairs)
    helpers.check_attention(out, ref, plain=plain, what="mixed serving step")


@pytest.mark.parametrize("plain", [False, True])
def test_long_context_chunked_full_size_every_output(plain):
    """The long-context configuration at full size: contexts of 32768 .. 131072 tokens, chunk size 2048; every
    per-chunk (m, l, o) and every merged output against the oracle's chunk-and-merge path."""
    w = workloads.config_long_context(v_outliers=not plain)
    heads = PLAIN_HEADS if plain else None
    cache = helpers.gpu_fill(w)
    out, ws = helpers.gpu_decode(w, cache, chunk_size=2048)
    assert torch.isfinite(out.float()).all()
    codes, scales = helpers.oracle_fp8_cache(w, heads=heads)
    helpers.check_cache_bit_exact(cache, codes, scales, heads=heads, what="long context")
    pairs = _pairs_of_heads(w.batch, 5, PLAIN_HEADS) if plain else None
    ref, partials = attention.paged_attention_chunked(w.q.float().numpy(), (codes, scales), w.block_table.numpy(),
                                                      w.context_lens, 2048, pairs=pairs)
    o_c, m_c, l_c = (t.cpu().numpy() for t in binding.chunk_partials(ws, w.batch, 40, 128, w.block_table.shape[1], 2048))
    for (b, h), (m, l, o) in partials.items():
        n = len(m)
        assert n == w.context_lens[b] // 2048
        assert np.allclose(m_c[b, h, :n], m, rtol=1e-4, atol=1e-3)
        assert np.allclose(l_c[b, h, :n], l, rtol=5e-3, atol=1e-4)
        assert np.allclose(o_c[b, h, :n], o, rtol=5e-3, atol=2e-2)
    helpers.check_attention(out, ref, plain=plain, what="long context chunked")
