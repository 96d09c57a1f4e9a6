"""TEST INFRASTRUCTURE — CPU oracle, part 2: attention over the paged cache, in float64.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA path shares no code with it.

Inputs are the cache in logical order plus the block table.  The cache ``kv`` is either
an array of values [num_blocks, Hkv, 2, 16, D] (the bf16 ablation cache, or an FP8 cache
already passed through ``kv_cache.dequantise``) or the pair ``(codes, scales)`` of an FP8
cache (a third entry names the format module when it is not ``e4m3``), which is dequantised
(Eq. 6: dec(code) * scale, exact in float64) as it is read.
The computation is the definition, written out per (sequence, query head):

  * Eq. 9 / Algorithm 3 phase 1: only blocks 0 .. ceil(t/B)-1 of the sequence are read,
    and within the last block only the first t - B*(ceil(t/B)-1) tokens.
  * Eq. 7 / Algorithm 2 phase 1: query head i reads kv head floor(i / H_g), H_g = H_q / H_k.
  * Eq. 1, Eq. 8, Eq. 10: o = softmax(q K^T * sm_scale) V with the maximum subtracted.
  * Opt-Pa's long-sequence path (abstract, conclusion): the context is cut into chunks of
    a fixed number of tokens; each chunk yields (m_c, l_c, o_c) = (max logit, sum of
    exp(logit - m_c), softmax-weighted V within the chunk); the chunks are merged with
    weights l_c * exp(m_c - max_c m_c).  Logits are in natural-log units after sm_scale.
"""
from __future__ import annotations

import numpy as np

from . import e4m3

BLOCK_SIZE = 16


def gather_kv(kv: np.ndarray, table_row: np.ndarray, length: int, kv_head: int):
    """Logical K and V of one sequence and kv head: two float64 arrays [length, D]."""
    pos = np.arange(length)
    blk = np.asarray(table_row)[pos // BLOCK_SIZE].astype(np.int64)     # Eq. 9: valid blocks only
    off = pos % BLOCK_SIZE
    if isinstance(kv, tuple):                                           # FP8: Eq. 6 on the fly
        codes, scales = kv[0], kv[1]
        fmt = kv[2] if len(kv) > 2 else e4m3                            # (codes, scales[, format module])
        return tuple(fmt.decode(codes[blk, kv_head, w, off, :])
                     * scales[blk, kv_head, w].astype(np.float64)[:, None] for w in (0, 1))
    return (kv[blk, kv_head, 0, off, :].astype(np.float64),
            kv[blk, kv_head, 1, off, :].astype(np.float64))


def softmax_attention(q: np.ndarray, K: np.ndarray, V: np.ndarray, sm_scale: float) -> np.ndarray:
    """Eq. 1 for one query vector: softmax(q K^T * sm_scale) V; zeros for an empty context."""
    if K.shape[0] == 0:
        return np.zeros(V.shape[1], dtype=np.float64)
    s = (K @ q.astype(np.float64)) * sm_scale
    p = np.exp(s - np.max(s))                                           # Eq. 10
    return (p / np.sum(p)) @ V


def paged_attention(q: np.ndarray, kv: np.ndarray, block_table: np.ndarray, context_lens,
                    cu_q_lens=None, causal: bool = True, sm_scale: float | None = None,
                    pairs=None) -> np.ndarray:
    """Attention for every query token and head: float64 [total_q, Hq, D].

    ``q`` [total_q, Hq, D]; sequence b owns query rows cu_q_lens[b] .. cu_q_lens[b+1]-1
    (default: one row per sequence = decode).  The n query rows of a sequence are its last
    n positions; with ``causal`` row i sees positions 0 .. L-n+i (Eq. 1's K_{<=t}).
    ``pairs`` (iterable of (query row, query head)) limits the work to a sample; other
    rows of the result stay NaN.
    """
    total_q, num_q_heads, head_dim = q.shape
    num_kv_heads = (kv[0] if isinstance(kv, tuple) else kv).shape[1]
    group = num_q_heads // num_kv_heads                                 # H_g of Eq. 7
    batch = len(context_lens)
    if cu_q_lens is None:
        cu_q_lens = np.arange(batch + 1)
    if sm_scale is None:
        sm_scale = 1.0 / np.sqrt(head_dim)
    out = np.full((total_q, num_q_heads, head_dim), np.nan, dtype=np.float64)
    wanted = None if pairs is None else set((int(r), int(h)) for r, h in pairs)
    for b in range(batch):
        L = int(context_lens[b])
        r0, r1 = int(cu_q_lens[b]), int(cu_q_lens[b + 1])
        n = r1 - r0
        for g in range(num_kv_heads):
            rows = [(r, h) for r in range(r0, r1) for h in range(g * group, (g + 1) * group)
                    if wanted is None or (r, h) in wanted]
            if not rows:
                continue
            K, V = gather_kv(kv, block_table[b], L, g)
            for r, h in rows:
                visible = L - n + (r - r0) + 1 if causal else L
                visible = max(0, min(L, visible))
                out[r, h] = softmax_attention(q[r, h], K[:visible], V[:visible], sm_scale)
    return out


def chunk_partials(q_vec: np.ndarray, K: np.ndarray, V: np.ndarray, sm_scale: float, chunk: int):
    """Per-chunk (m_c, l_c, o_c) for one query vector over K, V [L, D]."""
    L = K.shape[0]
    n_chunks = (L + chunk - 1) // chunk
    m = np.full(n_chunks, -np.inf)
    l = np.zeros(n_chunks)
    o = np.zeros((n_chunks, V.shape[1]))
    for c in range(n_chunks):
        Kc, Vc = K[c * chunk:(c + 1) * chunk], V[c * chunk:(c + 1) * chunk]
        s = (Kc @ q_vec.astype(np.float64)) * sm_scale
        m[c] = np.max(s)
        p = np.exp(s - m[c])
        l[c] = np.sum(p)
        o[c] = (p / l[c]) @ Vc
    return m, l, o


def merge_partials(m: np.ndarray, l: np.ndarray, o: np.ndarray) -> np.ndarray:
    """Log-sum-exp merge of chunk partials; chunks with l == 0 carry no weight."""
    if m.size == 0 or not np.any(l > 0):
        return np.zeros(o.shape[1] if o.ndim == 2 else 0)
    M = np.max(m[l > 0])
    w = np.where(l > 0, l * np.exp(np.where(l > 0, m, M) - M), 0.0)
    return (w / np.sum(w)) @ o


def paged_attention_chunked(q: np.ndarray, kv: np.ndarray, block_table: np.ndarray, context_lens,
                            chunk: int, sm_scale: float | None = None, pairs=None):
    """Decode (one query row per sequence) through the chunk-and-merge path.

    Returns ``(out float64 [B, Hq, D], partials)`` where ``partials[(b, h)] = (m, l, o)``.
    """
    batch, num_q_heads, head_dim = q.shape
    num_kv_heads = (kv[0] if isinstance(kv, tuple) else kv).shape[1]
    group = num_q_heads // num_kv_heads
    if sm_scale is None:
        sm_scale = 1.0 / np.sqrt(head_dim)
    out = np.full((batch, num_q_heads, head_dim), np.nan, dtype=np.float64)
    partials = {}
    wanted = None if pairs is None else set((int(r), int(h)) for r, h in pairs)
    for b in range(batch):
        for g in range(num_kv_heads):
            hs = [h for h in range(g * group, (g + 1) * group) if wanted is None or (b, h) in wanted]
            if not hs:
                continue
            K, V = gather_kv(kv, block_table[b], int(context_lens[b]), g)
            for h in hs:
                m, l, o = chunk_partials(q[b, h], K, V, sm_scale, chunk)
                partials[(b, h)] = (m, l, o)
                out[b, h] = merge_partials(m, l, o)
    return out, partials
