"""TEST INFRASTRUCTURE — CPU oracle, part 1: the Opt-KV write (Algorithm 1, phase 1).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA path shares no code with it.

The cache is held in its *logical* order, one array per kind:

    codes  uint8   [num_blocks, num_kv_heads, 2 (0 = K, 1 = V), 16, head_dim]
    scales float32 [num_blocks, num_kv_heads, 2]

What a write call does, token group by token group (a group = the call's non-skipped
tokens that land in one physical block):

  * Eq. 5 / Algorithm 1 "filtering condition": a token whose slot index is negative is
    skipped (membership in the paper's SkipSet is expressed by the caller as a negative
    slot).
  * "reshape and store K_i, V_i into block_wise cache structure": slot = block * 16 +
    offset.
  * "compressing valid blocks into FP8" (Section 3.1) with dynamic scales, read as: one
    fp32 scale per (block, kv head, K|V), scale = max(previous scale, amax / 448), where
    amax is the largest magnitude among the group's values for that head.  A group that
    writes offset 0 opens the block anew: the previous scale counts as 0 and every slot
    the group does not write is cleared to code 0.  When the scale of a block that
    already holds tokens grows, the resident codes are re-expressed in the new scale:
    code <- enc((dec(code) * s_old) / s_new), every operation rounded to fp32.
  * new values: code = enc(x / s_new) in fp32; if s_new == 0 the code is a signed zero.

All arithmetic that decides a code is IEEE fp32 (numpy float32), as stated above.
"""
from __future__ import annotations

import numpy as np

from . import e4m3

BLOCK_SIZE = 16
_F32 = np.float32


def new_cache(num_blocks: int, num_kv_heads: int, head_dim: int):
    """An empty FP8 cache: all codes 0, all scales 0."""
    codes = np.zeros((num_blocks, num_kv_heads, 2, BLOCK_SIZE, head_dim), dtype=np.uint8)
    scales = np.zeros((num_blocks, num_kv_heads, 2), dtype=np.float32)
    return codes, scales


def _quantise(x: np.ndarray, scale: np.float32, fmt=e4m3) -> np.ndarray:
    """enc(x / scale) with an fp32 division; a zero scale gives signed zeros."""
    x = x.astype(_F32)
    if not scale > 0:
        return fmt.encode(np.copysign(_F32(0.0), x))
    return fmt.encode((x / _F32(scale)).astype(_F32))


def kv_write(codes: np.ndarray, scales: np.ndarray, k: np.ndarray, v: np.ndarray,
             slot_mapping: np.ndarray, heads=None, fmt=e4m3) -> None:
    """Apply one write call in place.

    ``fmt`` is the 8-bit format of the codes: ``e4m3`` (the reading the build takes), or ``e5m2``
    as an ablation of the format the paper leaves open; the scale is amax / fmt.MAX either way.

    ``k``, ``v``: float32 [T, Hkv, D] holding bf16-representable values; ``slot_mapping``
    int64 [T].  ``heads`` restricts the work to some kv heads (used to check samples of a
    large cache); the result for those heads does not depend on the others.
    """
    slot_mapping = np.asarray(slot_mapping, dtype=np.int64)
    kv = (np.asarray(k, dtype=_F32), np.asarray(v, dtype=_F32))
    heads = range(codes.shape[1]) if heads is None else heads
    keep = np.nonzero(slot_mapping >= 0)[0]                       # Eq. 5
    blocks = slot_mapping[keep] // BLOCK_SIZE
    for blk in np.unique(blocks):
        tok = keep[blocks == blk]                                 # token rows of this group
        off = slot_mapping[tok] % BLOCK_SIZE
        fresh = bool(np.any(off == 0))
        others = np.setdiff1d(np.arange(BLOCK_SIZE), off)         # slots the group leaves alone
        for h in heads:
            for w in (0, 1):
                x = kv[w][tok, h, :]                              # [n, D]
                amax = _F32(np.max(np.abs(x)))
                s_old = _F32(0.0) if fresh else _F32(scales[blk, h, w])
                s_new = max(s_old, _F32(amax / _F32(fmt.MAX)))
                if fresh:
                    codes[blk, h, w, others, :] = 0
                elif s_new > s_old and s_old > 0:
                    resident = fmt.decode(codes[blk, h, w, others, :]).astype(_F32)
                    resident = (resident * s_old).astype(_F32)
                    codes[blk, h, w, others, :] = _quantise(resident, s_new, fmt)
                codes[blk, h, w, off, :] = _quantise(x, s_new, fmt)
                scales[blk, h, w] = s_new


def new_cache_bf16(num_blocks: int, num_kv_heads: int, head_dim: int) -> np.ndarray:
    """The un-quantised ablation cache: float32 array holding bf16-representable values."""
    return np.zeros((num_blocks, num_kv_heads, 2, BLOCK_SIZE, head_dim), dtype=np.float32)


def kv_write_bf16(values: np.ndarray, k: np.ndarray, v: np.ndarray, slot_mapping: np.ndarray) -> None:
    """Un-quantised write: skip negative slots (Eq. 5), store the rest unchanged."""
    slot_mapping = np.asarray(slot_mapping, dtype=np.int64)
    keep = np.nonzero(slot_mapping >= 0)[0]
    blk = slot_mapping[keep] // BLOCK_SIZE
    off = slot_mapping[keep] % BLOCK_SIZE
    for w, x in enumerate((k, v)):
        values[blk, :, w, off, :] = np.asarray(x, dtype=np.float32)[keep]


def dequantise(codes: np.ndarray, scales: np.ndarray, fmt=e4m3) -> np.ndarray:
    """Eq. 6: float64 values of a whole FP8 cache, dec(code) * scale (exact in float64)."""
    return fmt.decode(codes) * scales.astype(np.float64)[..., None, None]
