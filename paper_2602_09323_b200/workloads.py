"""Seeded synthetic workloads for the paged FP8 GQA attention path.

This module only draws random inputs and builds index structures (block tables,
slot mappings).  It holds none of the method's arithmetic: no quantisation, no
softmax, no cache layout.  Both the tests' CPU oracle and the CUDA path are fed
from here so that they see identical inputs.

Value recipe (all configurations): q, k, v ~ N(0, 1) rounded to bf16; for every
head two channels, drawn once per head from the seed, are multiplied by 20 (the
"outlier channels" that make a per-block dynamic scale necessary).  Physical
blocks are a seeded random permutation of ``range(num_blocks)`` where
``num_blocks`` is the number of needed blocks plus about 10 % unused spares.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Sequence

import torch

BLOCK_SIZE = 16


@dataclasses.dataclass
class Workload:
    """One synthetic attention-layer problem.

    Shapes: ``q`` bf16 [sum(q_lens), Hq, D]; ``k``/``v`` bf16 [sum(context_lens), Hkv, D]
    hold the K/V of *every* logical token, sequence after sequence;
    ``slot_mapping`` int64 [sum(context_lens)] gives each of those tokens its
    physical slot (block * 16 + offset); ``block_table`` int32 [B, max_blocks].
    ``kv_offsets[b]`` is the row in ``k``/``v`` where sequence ``b`` starts.
    """

    name: str
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    context_lens: List[int]
    q_lens: List[int]
    num_blocks: int
    q: torch.Tensor
    k: torch.Tensor
    v: torch.Tensor
    slot_mapping: torch.Tensor
    block_table: torch.Tensor
    kv_offsets: List[int]
    seed: int

    @property
    def batch(self) -> int:
        return len(self.context_lens)

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads

    @property
    def sm_scale(self) -> float:
        return 1.0 / math.sqrt(self.head_dim)

    @property
    def cu_q_lens(self) -> torch.Tensor:
        cu = [0]
        for n in self.q_lens:
            cu.append(cu[-1] + n)
        return torch.tensor(cu, dtype=torch.int32)

    @property
    def context_lens_tensor(self) -> torch.Tensor:
        return torch.tensor(self.context_lens, dtype=torch.int32)


def _randn_bf16_with_outliers(gen: torch.Generator, rows: int, heads: int, dim: int,
                              outliers: bool) -> torch.Tensor:
    """N(0,1) values with two x20 channels per head, rounded to bf16."""
    x = torch.randn(rows, heads, dim, generator=gen, dtype=torch.float32)
    if outliers:
        for h in range(heads):
            ch = torch.randperm(dim, generator=gen)[:2]
            x[:, h, ch] *= 20.0
    return x.to(torch.bfloat16)


def make_block_table(gen: torch.Generator, context_lens: Sequence[int],
                     spare_fraction: float = 0.10, max_blocks: Optional[int] = None):
    """Randomly placed physical blocks for each sequence.

    Returns ``(block_table int32 [B, max_blocks], num_blocks)``; unused table
    entries hold -1 so that reading one is an obvious error.
    """
    need = [(L + BLOCK_SIZE - 1) // BLOCK_SIZE for L in context_lens]
    total = sum(need)
    num_blocks = total + max(1, int(math.ceil(total * spare_fraction)))
    perm = torch.randperm(num_blocks, generator=gen)
    width = max(need) if need else 1
    width = max(width, 1)
    if max_blocks is not None:
        width = max(width, max_blocks)
    table = torch.full((len(context_lens), width), -1, dtype=torch.int32)
    pos = 0
    for b, n in enumerate(need):
        table[b, :n] = perm[pos:pos + n].to(torch.int32)
        pos += n
    return table, num_blocks


def slots_for(block_table: torch.Tensor, b: int, start: int, stop: int) -> torch.Tensor:
    """Physical slots of logical tokens ``start..stop-1`` of sequence ``b``."""
    pos = torch.arange(start, stop, dtype=torch.int64)
    blk = block_table[b, pos // BLOCK_SIZE].to(torch.int64)
    return blk * BLOCK_SIZE + pos % BLOCK_SIZE


def make_workload(name: str, context_lens: Sequence[int], num_q_heads: int, num_kv_heads: int,
                  head_dim: int, seed: int = 0, q_lens: Optional[Sequence[int]] = None,
                  outliers: bool = True, v_outliers: Optional[bool] = None,
                  extra_table_blocks: int = 0) -> Workload:
    """Draw q/k/v and a shuffled block table for the given length mix.

    ``q_lens[b]`` new query tokens per sequence (default 1 = decode); they are the
    *last* ``q_lens[b]`` positions of the sequence, so ``context_lens`` counts them.
    ``extra_table_blocks`` reserves that many further blocks per sequence in the
    block table (room to append tokens later).
    """
    context_lens = [int(x) for x in context_lens]
    q_lens = [1] * len(context_lens) if q_lens is None else [int(x) for x in q_lens]
    if v_outliers is None:
        v_outliers = outliers
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    table_lens = [L + extra_table_blocks * BLOCK_SIZE for L in context_lens]
    block_table, num_blocks = make_block_table(gen, table_lens)
    total_kv = sum(context_lens)
    q = _randn_bf16_with_outliers(gen, sum(q_lens), num_q_heads, head_dim, outliers)
    k = _randn_bf16_with_outliers(gen, total_kv, num_kv_heads, head_dim, outliers)
    v = _randn_bf16_with_outliers(gen, total_kv, num_kv_heads, head_dim, v_outliers)
    kv_offsets, slots, off = [], [], 0
    for b, L in enumerate(context_lens):
        kv_offsets.append(off)
        slots.append(slots_for(block_table, b, 0, L))
        off += L
    slot_mapping = torch.cat(slots) if slots else torch.zeros(0, dtype=torch.int64)
    return Workload(name, num_q_heads, num_kv_heads, head_dim, context_lens, q_lens, num_blocks,
                    q, k, v, slot_mapping, block_table, kv_offsets, seed)


def relayout(w: Workload, seed: int) -> Workload:
    """The same tokens placed in a different random set of physical blocks (another layer's
    cache has its own placement); q, k, v are shared, not copied."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    width = w.block_table.shape[1]
    table, num_blocks = make_block_table(gen, [width * BLOCK_SIZE] * w.batch)
    need = torch.tensor([(L + BLOCK_SIZE - 1) // BLOCK_SIZE for L in w.context_lens])
    table[torch.arange(width)[None, :] >= need[:, None]] = -1
    slots = [slots_for(table, b, 0, L) for b, L in enumerate(w.context_lens)]
    slot_mapping = torch.cat(slots) if slots else torch.zeros(0, dtype=torch.int64)
    return dataclasses.replace(w, block_table=table, slot_mapping=slot_mapping, num_blocks=num_blocks)


def uniform_lengths(batch: int, lo: int, hi: int, seed: int) -> List[int]:
    """``batch`` context lengths uniform in [lo, hi] (inclusive), seeded."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed + 7919)
    return [int(x) for x in torch.randint(lo, hi + 1, (batch,), generator=gen)]


# --- SkipSet policies (Eq. 5): which tokens of a write call the caller marks as skipped ---------------------
# The paper filters tokens whose slot is negative or in a SkipSet of "redundant" slots and never says how
# the set is built.  Two policies that a serving stack meets are given here as slot-mapping generators; a
# skipped token is a negative slot, which is all the library ever tests.

def skip_padding(slot_mapping: torch.Tensor, row_lens: Sequence[int], padded_len: int) -> torch.Tensor:
    """Padding tokens: a batch of write rows laid out as ``len(row_lens)`` sequences of ``padded_len`` rows
    each, of which only the first ``row_lens[b]`` are real.  The padding rows get slot -1."""
    out = slot_mapping.clone()
    for b, n in enumerate(row_lens):
        out[b * padded_len + n:(b + 1) * padded_len] = -1
    return out


def share_prefix(w: Workload, donor: int, taker: int, prefix_tokens: int) -> Workload:
    """Duplicate prefix tokens: sequence ``taker`` starts with the same ``prefix_tokens`` tokens (a multiple of the
    block size) as sequence ``donor``, whose blocks already hold them.  The taker's block table points at the
    donor's blocks for the prefix, its own K/V rows of the prefix are made equal to the donor's, and their
    slots become -1: writing them again would be redundant."""
    assert prefix_tokens % BLOCK_SIZE == 0 and prefix_tokens <= min(w.context_lens[donor], w.context_lens[taker])
    nb = prefix_tokens // BLOCK_SIZE
    table = w.block_table.clone()
    table[taker, :nb] = table[donor, :nb]
    k, v, slots = w.k.clone(), w.v.clone(), w.slot_mapping.clone()
    d0, t0 = w.kv_offsets[donor], w.kv_offsets[taker]
    k[t0:t0 + prefix_tokens] = k[d0:d0 + prefix_tokens]
    v[t0:t0 + prefix_tokens] = v[d0:d0 + prefix_tokens]
    slots[t0:t0 + prefix_tokens] = -1
    return dataclasses.replace(w, block_table=table, k=k, v=v, slot_mapping=slots)


# --- the five named configurations -------------------------------------------------------------

def config_tiny(seed: int = 0, **kw) -> Workload:
    """Two sequences (17 and 300 tokens), 8 query heads, 2 KV heads, head_dim 64."""
    return make_workload("tiny_decode", [17, 300], 8, 2, 64, seed=seed, **kw)


def config_llama13b_decode(seed: int = 0, batch: int = 32, context: int = 2048, **kw) -> Workload:
    """LLaMA-13B-shaped decode: 40 query heads over 8 KV heads, head_dim 128."""
    return make_workload("llama13b_decode", [context] * batch, 40, 8, 128, seed=seed, **kw)


def config_llama13b_mha_ablation(seed: int = 0, batch: int = 32, context: int = 2048, **kw) -> Workload:
    """The un-optimised layout: one KV head per query head (bf16 cache is chosen at write time)."""
    return make_workload("llama13b_mha_ablation", [context] * batch, 40, 40, 128, seed=seed, **kw)


def config_mixed_serving(seed: int = 0, batch: int = 64, lo: int = 128, hi: int = 8192, **kw) -> Workload:
    """Mixed-length serving step; lengths count the token appended in this step."""
    lens = uniform_lengths(batch, lo, hi, seed)
    return make_workload("mixed_serving", lens, 40, 8, 128, seed=seed, **kw)


def config_long_context(seed: int = 0, lens: Sequence[int] = (32768, 65536, 98304, 131072), **kw) -> Workload:
    """Long-context chunked decode (chunk size is an argument of the call, 2048 by default)."""
    return make_workload("long_context", list(lens), 40, 8, 128, seed=seed, **kw)


def config_chunked_prefill(seed: int = 0, batch: int = 8, prior: int = 4096, new: int = 512, **kw) -> Workload:
    """Each sequence has ``prior`` cached tokens and ``new`` query tokens (causal)."""
    return make_workload("chunked_prefill", [prior + new] * batch, 40, 8, 128, seed=seed,
                         q_lens=[new] * batch, **kw)
