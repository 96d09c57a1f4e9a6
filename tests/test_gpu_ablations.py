"""GPU parity of the ablations the paper gestures at but does not define: the E5M2 code format (Section 3.1
says "FP8" and nothing more) and two SkipSet policies of Eq. 5 (padding tokens, duplicate prefix tokens),
against the oracle run the same way."""
import numpy as np
import pytest
import torch

from oracle import attention, e5m2, kv_cache
from paper_2602_09323_b200 import binding, workloads
from tests import helpers

pytestmark = pytest.mark.gpu


def _bf16_reference(w):
    """Float64 attention over the un-quantised values (what a cache without compression would give)."""
    vals = kv_cache.new_cache_bf16(w.num_blocks, w.num_kv_heads, w.head_dim)
    keep = w.slot_mapping.numpy() >= 0
    kv_cache.kv_write_bf16(vals, w.k.float().numpy()[keep], w.v.float().numpy()[keep], w.slot_mapping.numpy()[keep])
    return vals


@pytest.mark.parametrize("hq,hkv,d", [(10, 2, 128), (8, 2, 64), (16, 2, 128)])
def test_e5m2_cache_write_decode_and_fused_step(hq, hkv, d):
    """The same write rule with E5M2 codes (scale = amax / 57344): cache bytes bit for bit against the oracle for a
    bulk fill followed by token-by-token appends (scales grow, residents are re-expressed), through the separate
    write call and through the one-launch step; attention within the usual tolerance of the oracle's result on
    the oracle's E5M2 cache."""
    w = workloads.make_workload("e5m2", [300, 64, 2048, 47, 900], hq, hkv, d, seed=91)
    steps = 20
    hist = np.concatenate([np.arange(w.kv_offsets[b], w.kv_offsets[b] + L - steps) for b, L in enumerate(w.context_lens)])
    table, q = w.block_table.cuda(), w.q.cuda()
    k, v, slots = w.k.cuda(), w.v.cuda(), w.slot_mapping.cuda()
    caches = [helpers.gpu_fill(w, dtype=binding.KV_FP8_E5M2, calls=[hist]) for _ in range(2)]
    codes, scales = helpers.oracle_fp8_cache(w, calls=[hist], fmt=e5m2)
    ws = binding.new_workspace(w.batch, hq, hkv, d, table.shape[1])
    plan = torch.empty(binding.plan_bytes(w.batch, hkv, table.shape[1]), dtype=torch.uint8, device="cuda")
    kf, vf, sf = w.k.float().numpy(), w.v.float().numpy(), w.slot_mapping.numpy()
    for step in range(steps):
        new = np.array([w.kv_offsets[b] + L - steps + step for b, L in enumerate(w.context_lens)])
        new_t = torch.from_numpy(new).cuda()
        lens = torch.tensor([L - steps + step + 1 for L in w.context_lens], dtype=torch.int32).cuda()
        k_new, v_new, s_new = k[new_t].contiguous(), v[new_t].contiguous(), slots[new_t].contiguous()
        binding.kv_write(caches[0], k_new, v_new, s_new)
        out_a = binding.paged_decode(caches[0], q, table, lens, w.sm_scale, ws)
        binding.decode_plan(table, lens, hkv, w.num_blocks, plan=plan)
        out_b = binding.decode_step_planned(caches[1], plan, q, table.shape[1], w.sm_scale, ws, k_new, v_new, s_new)
        kv_cache.kv_write(codes, scales, kf[new], vf[new], sf[new], fmt=e5m2)
    torch.cuda.synchronize()
    assert binding.workspace_status(ws) == 0
    for c in caches:
        helpers.check_cache_bit_exact(c, codes, scales, what="e5m2")
    assert torch.equal(out_a, out_b)
    ref = attention.paged_attention(w.q.float().numpy(), (codes, scales, e5m2), w.block_table.numpy(), w.context_lens)
    helpers.check_attention(out_a, ref, what="e5m2 decode")


def test_e5m2_chunked_prefill_and_what_the_format_costs():
    """Chunked prefill over an E5M2 cache against the oracle; and, for the record, how far either format's
    attention is from attention over the un-quantised values (two mantissa bits against three)."""
    w = workloads.make_workload("e5m2_prefill", [700, 333, 129], 10, 2, 128, seed=92, q_lens=[200, 40, 129])
    ws = binding.new_workspace(w.batch, 10, 2, 128, w.block_table.shape[1], 2048, sum(w.q_lens))
    errs = {}
    exact = attention.paged_attention(w.q.float().numpy(), _bf16_reference(w), w.block_table.numpy(), w.context_lens,
                                      cu_q_lens=w.cu_q_lens.numpy(), causal=True)
    for name, dtype, fmt in (("e4m3", binding.KV_FP8_E4M3, None), ("e5m2", binding.KV_FP8_E5M2, e5m2)):
        cache = helpers.gpu_fill(w, dtype=dtype)
        out = binding.paged_chunked(cache, w.q.cuda(), w.cu_q_lens.cuda(), w.block_table.cuda(), w.context_lens_tensor.cuda(),
                                    2048, True, w.sm_scale, ws)
        torch.cuda.synchronize()
        assert binding.workspace_status(ws) == 0
        codes, scales = helpers.oracle_fp8_cache(w, fmt=fmt)
        helpers.check_cache_bit_exact(cache, codes, scales, what=name)
        kv = (codes, scales) if fmt is None else (codes, scales, fmt)
        ref = attention.paged_attention(w.q.float().numpy(), kv, w.block_table.numpy(), w.context_lens,
                                        cu_q_lens=w.cu_q_lens.numpy(), causal=True)
        helpers.check_attention(out, ref, what=f"{name} prefill")
        errs[name] = float(np.abs(out.double().cpu().numpy() - exact).mean())
    print("mean |attention - attention over un-quantised K/V|:", errs)
    assert errs["e5m2"] > errs["e4m3"]                     # one mantissa bit less shows


def test_skipset_padding_tokens():
    """A padded batch of write rows: every sequence's rows are padded to the longest with junk that must never
    reach the cache (Eq. 5: the caller gives those rows a negative slot)."""
    w = workloads.make_workload("padding", [70, 333, 16, 129], 8, 2, 128, seed=93)
    padded = max(w.context_lens)
    k = torch.full((w.batch * padded, 2, 128), 777.0, dtype=torch.bfloat16)       # junk that would wreck the scales
    v = torch.full_like(k, -555.0)
    slots = torch.zeros(w.batch * padded, dtype=torch.int64)                      # junk rows point at slot 0
    for b, L in enumerate(w.context_lens):
        rows = slice(w.kv_offsets[b], w.kv_offsets[b] + L)
        k[b * padded:b * padded + L], v[b * padded:b * padded + L] = w.k[rows], w.v[rows]
        slots[b * padded:b * padded + L] = w.slot_mapping[rows]
    slots = workloads.skip_padding(slots, w.context_lens, padded)
    cache = binding.Cache(w.num_blocks, 2, 128)
    binding.kv_write(cache, k.cuda(), v.cuda(), slots.cuda())
    codes, scales = kv_cache.new_cache(w.num_blocks, 2, 128)
    kv_cache.kv_write(codes, scales, k.float().numpy(), v.float().numpy(), slots.numpy())
    helpers.check_cache_bit_exact(cache, codes, scales, what="padding")
    plain_codes, plain_scales = helpers.oracle_fp8_cache(w)                      # the un-padded write gives the same cache
    assert np.array_equal(codes, plain_codes) and np.array_equal(scales, plain_scales)
    out, _ = helpers.gpu_decode(w, cache)
    ref = attention.paged_attention(w.q.float().numpy(), (codes, scales), w.block_table.numpy(), w.context_lens)
    helpers.check_attention(out, ref, what="padding")


def test_skipset_duplicate_prefix_tokens():
    """Two sequences share a 160-token prefix: the second one's block table points at the first one's blocks and
    its prefix rows are skipped.  The cache holds the prefix once, and both sequences attend over it."""
    base = workloads.make_workload("prefix", [500, 300, 90], 10, 2, 128, seed=94)
    w = workloads.share_prefix(base, donor=0, taker=1, prefix_tokens=160)
    assert (w.slot_mapping[w.kv_offsets[1]:w.kv_offsets[1] + 160] < 0).all()
    cache = helpers.gpu_fill(w)
    codes, scales = helpers.oracle_fp8_cache(w)
    helpers.check_cache_bit_exact(cache, codes, scales, what="prefix")
    own = base.block_table[1, :10].long()                                       # the taker's own prefix blocks stay empty
    assert not codes[own].any() and not scales[own].any()
    out, _ = helpers.gpu_decode(w, cache)
    ref = attention.paged_attention(w.q.float().numpy(), (codes, scales), w.block_table.numpy(), w.context_lens)
    helpers.check_attention(out, ref, what="prefix")
    # the same answer as writing the duplicate rows into blocks of their own, up to the prefix blocks' scales
    # having been set by the donor's rows alone (identical rows, identical scales): bit-identical outputs
    dup = dataclasses_replace_prefix(base)
    cache2 = helpers.gpu_fill(dup)
    out2, _ = helpers.gpu_decode(dup, cache2)
    assert torch.equal(out[1], out2[1])


def dataclasses_replace_prefix(base):
    """The taker's prefix rows equal to the donor's, but written into the taker's own blocks (nothing skipped)."""
    import dataclasses
    k, v = base.k.clone(), base.v.clone()
    d0, t0 = base.kv_offsets[0], base.kv_offsets[1]
    k[t0:t0 + 160], v[t0:t0 + 160] = k[d0:d0 + 160], v[d0:d0 + 160]
    return dataclasses.replace(base, k=k, v=v)
