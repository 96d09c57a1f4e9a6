"""The SkipSet policies (Eq. 5: tokens whose slot is negative are not written) as slot-mapping generators, checked on
the CPU with the oracle: what they skip must be redundant, i.e. leave the cache and the attention unchanged."""
import dataclasses

import numpy as np
import torch

from oracle import attention, kv_cache
from paper_2602_09323_b200 import workloads


def _write(w, k=None, v=None, slots=None):
    codes, scales = kv_cache.new_cache(w.num_blocks, w.num_kv_heads, w.head_dim)
    k = w.k if k is None else k
    v = w.v if v is None else v
    slots = w.slot_mapping if slots is None else slots
    kv_cache.kv_write(codes, scales, k.float().numpy(), v.float().numpy(), slots.numpy())
    return codes, scales


def test_padding_rows_are_skipped_and_the_cache_equals_the_unpadded_write():
    w = workloads.make_workload("padding", [37, 90, 16, 5], 4, 2, 64, seed=3)
    padded = max(w.context_lens)
    k = torch.full((w.batch * padded, 2, 64), 777.0, dtype=torch.bfloat16)        # junk that would wreck the scales
    v = torch.full_like(k, -555.0)
    slots = torch.zeros(w.batch * padded, dtype=torch.int64)                       # junk rows point at slot 0
    for b, L in enumerate(w.context_lens):
        rows = slice(w.kv_offsets[b], w.kv_offsets[b] + L)
        k[b * padded:b * padded + L], v[b * padded:b * padded + L] = w.k[rows], w.v[rows]
        slots[b * padded:b * padded + L] = w.slot_mapping[rows]
    skipped = workloads.skip_padding(slots, w.context_lens, padded)
    assert int((skipped < 0).sum()) == w.batch * padded - sum(w.context_lens)
    assert torch.equal(skipped[skipped >= 0], w.slot_mapping)
    codes, scales = _write(w, k, v, skipped)
    plain_codes, plain_scales = _write(w)
    assert np.array_equal(codes, plain_codes) and np.array_equal(scales, plain_scales)
    # without the policy the junk rows do reach the cache
    bad_codes, bad_scales = _write(w, k, v, slots)
    assert not (np.array_equal(bad_codes, plain_codes) and np.array_equal(bad_scales, plain_scales))


def test_shared_prefix_is_held_once_and_attention_is_unchanged():
    base = workloads.make_workload("prefix", [200, 130, 40], 4, 2, 64, seed=4)
    w = workloads.share_prefix(base, donor=0, taker=1, prefix_tokens=96)
    t0 = w.kv_offsets[1]
    assert (w.slot_mapping[t0:t0 + 96] < 0).all() and (w.slot_mapping[t0 + 96:t0 + 130] >= 0).all()
    assert torch.equal(w.block_table[1, :6], w.block_table[0, :6])
    codes, scales = _write(w)
    own = base.block_table[1, :6].long().numpy()                                   # the taker's own prefix blocks stay empty
    assert not codes[own].any() and not scales[own].any()
    out = attention.paged_attention(w.q.float().numpy(), (codes, scales), w.block_table.numpy(), w.context_lens)
    # the same tokens written into blocks of the taker's own: identical rows give identical codes and scales, so
    # the attention is the same to the last bit
    dup = dataclasses.replace(w, block_table=base.block_table, slot_mapping=base.slot_mapping)
    codes2, scales2 = _write(dup)
    out2 = attention.paged_attention(dup.q.float().numpy(), (codes2, scales2), dup.block_table.numpy(), dup.context_lens)
    assert np.array_equal(out, out2)
    # and it differs from the taker's attention before its prefix was replaced by the donor's
    codes3, scales3 = _write(base)
    out3 = attention.paged_attention(base.q.float().numpy(), (codes3, scales3), base.block_table.numpy(), base.context_lens)
    assert not np.array_equal(out[1], out3[1]) and np.array_equal(out[0], out3[0]) and np.array_equal(out[2], out3[2])
