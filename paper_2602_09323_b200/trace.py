"""Where the time of one launch goes: ``python -m paper_2602_09323_b200.trace [--workload ...]``.

Builds ``libcoopt_trace.so`` (the library's sources with ``-DCOOPT_TRACE``), runs the fused decode step of a
workload a few times and prints, for the last launch, when each role of the tcgen05 kernel reached its
milestones: per milestone the median, the earliest and the latest CTA, in microseconds from that CTA's own
first instruction, and the span of the whole launch on the global timer.  The stamps cost a few stores per
tile; the launch is a few per cent slower than in the ordinary library, so this is a breakdown, not a
benchmark.  ``--workload chunked_prefill`` prints instead, for the tcgen05 prefill kernel, the cycles that the
first thread of softmax team 0 and the two instruction-issuing lanes spend in each phase of a tile.
"""
from __future__ import annotations

import argparse
import ctypes

import numpy as np
import torch

from . import binding, build, workloads

SLOTS = 256
MAX_CTAS = 1024
NAMES = ["entry", "entry_ns", "setup_done", "plan_in_smem", "first_copy", "first_landed", "first_probs", "last_copy",
         "last_landed", "last_pv", "teams_done", "last_hand_off", "piece_stored", "counted", "epilogue_done", "exit",
         "exit_ns", "write_done", "num_seg", "num_tiles", "sm_id", "producer_plan", "prev_exit_ns", "first_copy_ready"]
SEG_BASE, TEAM_SEG_BASE = 24, 44


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="llama13b_decode", choices=["llama13b_decode", "mixed_serving", "long_context", "chunked_prefill"])
    ap.add_argument("--no-append", action="store_true", help="attention only (no new token written in the launch)")
    ap.add_argument("--launches", type=int, default=12)
    ap.add_argument("--timeline", type=int, nargs="*", default=None, help="CTAs whose tile-by-tile timeline is printed")
    ap.add_argument("--rotate", type=int, default=0, help="with --per-cta: the second listed launch gives CTA i the plan "
                    "region i + ROTATE, to tell slow shares of the plan from slow SMs")
    ap.add_argument("--per-cta", action="store_true", help="also list every CTA: SM, segments, streaming time")
    ap.add_argument("--sm-mhz", type=float, default=1965.0, help="SM clock used to turn cycles into microseconds")
    args = ap.parse_args()
    binding.use_library(build.build(trace=True))
    lib = binding.load_library()
    lib.coopt_trace_set_buffer.restype, lib.coopt_trace_set_buffer.argtypes = ctypes.c_int, [ctypes.c_void_p, ctypes.c_size_t]
    torch.cuda.set_device(0)
    if args.workload == "chunked_prefill":
        return prefill_trace(lib)
    chunk = 0
    if args.workload == "llama13b_decode":
        w = workloads.config_llama13b_decode()
    elif args.workload == "mixed_serving":
        w = workloads.config_mixed_serving()
    else:
        w, chunk = workloads.config_long_context(), 2048
    B, Hq, Hkv, D = w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim
    k, v, slots = w.k.cuda(), w.v.cuda(), w.slot_mapping.cuda()
    last = torch.tensor([w.kv_offsets[b] + L - 1 for b, L in enumerate(w.context_lens)])
    hist = torch.ones(k.shape[0], dtype=torch.bool)
    hist[last] = False
    hist_idx, new_idx = hist.nonzero().squeeze(1).cuda(), last.cuda()
    k_new, v_new, s_new = k[new_idx].contiguous(), v[new_idx].contiguous(), slots[new_idx].contiguous()
    caches = []
    for _ in range(2):                      # two caches visited in turn: more than L2 between two visits of one
        c = binding.Cache(w.num_blocks, Hkv, D)
        binding.kv_write(c, k[hist_idx], v[hist_idx], slots[hist_idx])
        caches.append(c)
    table, lens, q = w.block_table.clamp(min=0).cuda(), w.context_lens_tensor.cuda(), w.q.cuda()
    plan = binding.decode_plan(table, lens, Hkv, w.num_blocks, chunk)
    ws = binding.new_workspace(B, Hq, Hkv, D, table.shape[1], chunk, B)
    buf = torch.zeros(MAX_CTAS * SLOTS, dtype=torch.int64, device="cuda")
    assert lib.coopt_trace_set_buffer(ctypes.c_void_p(buf.data_ptr()), buf.numel() * 8) == 0
    out = torch.empty_like(q)
    lib.coopt_trace_set_rotate.restype, lib.coopt_trace_set_rotate.argtypes = ctypes.c_int, [ctypes.c_int]
    for i in range(args.launches):
        if i != args.launches - 1:
            buf.zero_()                     # (the last launch follows its predecessor directly and keeps its exit times)
        lib.coopt_trace_set_rotate(args.rotate if i == args.launches - 1 else 0)
        if args.no_append:
            binding.decode_step_planned(caches[i % 2], plan, q, table.shape[1], w.sm_scale, ws, chunk_size=chunk, out=out)
        else:
            binding.decode_step_planned(caches[i % 2], plan, q, table.shape[1], w.sm_scale, ws, k_new, v_new, s_new,
                                        chunk_size=chunk, out=out)
        if i == args.launches - 3:
            torch.cuda.synchronize()
            prev = buf.cpu().numpy().reshape(MAX_CTAS, SLOTS).copy()
    torch.cuda.synchronize()
    assert binding.workspace_status(ws) == 0
    t = buf.cpu().numpy().reshape(MAX_CTAS, SLOTS)
    if args.per_cta:
        # streaming time (first copy requested to last tile landed) of every CTA in the last two launches, by SM
        us_ = 1.0 / args.sm_mhz
        rows = []
        for rec in (prev, t):
            r = rec[rec[:, 0] != 0]
            rows.append({int(x[20]) - 1: ((x[8] - x[4]) * us_, int(x[18]), (x[15] - x[0]) * us_) for x in r})
        print("sm  launch A: stream_us nseg life_us | launch B: stream_us nseg life_us")
        for sm in sorted(set(rows[0]) & set(rows[1])):
            a, b = rows[0][sm], rows[1][sm]
            print(f"{sm:3d}  {a[0]:6.2f} {a[1]} {a[2]:6.2f} | {b[0]:6.2f} {b[1]} {b[2]:6.2f}")
    if args.timeline is not None:
        us_ = 1.0 / args.sm_mhz
        for cta in (args.timeline or [0, 1, 2, 3]):
            x = t[cta]
            seg_first = [int(v) - 1 for v in x[128:148] if v]
            print(f"CTA {cta}: {int(x[18])} segments starting at tiles {seg_first}; epilogue got them at "
                  f"{[round(float((v - x[0]) * us_), 2) for v in x[24:44] if v]}")
            print(" tile   requested  logits_issued  probs_written  pv_issued   (us)")
            for i in range(32):
                if x[64 + i]:
                    f = lambda v: f"{(v - x[0]) * us_:10.2f}" if v else "         -"
                    print(f"{i:5d} {f(x[64 + i])}    {f(x[148 + i])}     {f(x[96 + i])}  {f(x[180 + i])}{'   <- segment starts' if i in seg_first else ''}")
    t = t[t[:, 0] != 0]
    us = 1.0 / args.sm_mhz
    print(f"workload {args.workload}{' (no append)' if args.no_append else ''}: {t.shape[0]} CTAs, "
          f"segments per CTA median {np.median(t[:, 18]):.0f} max {t[:, 18].max()}, tiles per CTA median {np.median(t[:, 19]):.0f} "
          f"max {t[:, 19].max()}")
    span = (t[:, 16].max() - t[:, 1].min()) / 1e3
    print(f"launch span on the global timer: {span:.1f} us (first entry to last exit); entries spread over "
          f"{(t[:, 1].max() - t[:, 1].min()) / 1e3:.1f} us, exits over {(t[:, 16].max() - t[:, 16].min()) / 1e3:.1f} us")
    if t[:, 22].min() > 0:
        print(f"gap to the launch before (its last exit to this one's first entry): {(t[:, 1].min() - t[:, 22].max()) / 1e3:.2f} us")
    print(f"{'milestone':<16}{'median':>9}{'earliest':>10}{'latest':>9}   (us after the CTA's first instruction, {args.sm_mhz:.0f} MHz)")
    for i, name in enumerate(NAMES):
        if name in ("entry", "entry_ns", "exit_ns", "num_seg", "num_tiles", "sm_id", "prev_exit_ns"):
            continue
        col = t[:, i]
        ok = col != 0
        if not ok.any():
            continue
        rel = (col[ok] - t[ok, 0]) * us
        print(f"{name:<16}{np.median(rel):9.2f}{rel.min():10.2f}{rel.max():9.2f}   ({int(ok.sum())} CTAs)")
    for base, label in ((TEAM_SEG_BASE, "team 0 begins segment"), (SEG_BASE, "epilogue gets segment")):
        for i in range(6):
            col = t[:, base + i]
            ok = col != 0
            if ok.any():
                rel = (col[ok] - t[ok, 0]) * us
                print(f"{label + ' ' + str(i):<26}{np.median(rel):9.2f}{rel.min():10.2f}{rel.max():9.2f}   ({int(ok.sum())} CTAs)")


PREFILL_PHASES = (
    (1, "team: waits for the tile's V part and scales"), (7, "team: V widened to f16"),
    (3, "team: waits for the tile's logits"), (2, "team: first pass (maximum of the thread's half row), halves meet"),
    (4, "team: references, rescale, second pass (probabilities to tensor memory)"),
    (13, "team: first thread done -> whole team arrived"), (5, "team: whole loop"),
    (8, "logits lane: waits for the K tile"), (9, "logits lane: waits for the team's previous P V product"),
    (10, "P V lane: waits for the probabilities"), (11, "P V lane: issues 8 instructions + commit"),
    (12, "P V lane: commit -> completion"))


def prefill_trace(lib):
    """Cycles per tile of team 0 in the phases of the tcgen05 prefill kernel (configuration: 8 sequences of 4096
    cached + 512 new tokens).  The lanes' figures are sums over both teams' tiles, divided by team 0's tile count."""
    w = workloads.config_chunked_prefill()
    cache = binding.Cache(w.num_blocks, w.num_kv_heads, w.head_dim)
    binding.kv_write(cache, w.k.cuda(), w.v.cuda(), w.slot_mapping.cuda())
    ws = binding.new_workspace(w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.block_table.shape[1], 2048, sum(w.q_lens))
    buf = torch.zeros(MAX_CTAS * SLOTS, dtype=torch.int64, device="cuda")
    assert lib.coopt_trace_set_buffer(ctypes.c_void_p(buf.data_ptr()), buf.numel() * 8) == 0
    q, cu, table, lens = w.q.cuda(), w.cu_q_lens.cuda(), w.block_table.cuda(), w.context_lens_tensor.cuda()
    for _ in range(3):
        buf.zero_()
        binding.paged_chunked(cache, q, cu, table, lens, 2048, True, w.sm_scale, ws)
    torch.cuda.synchronize()
    assert binding.workspace_status(ws) == 0
    t = buf.cpu().numpy().reshape(MAX_CTAS, SLOTS)
    t = t[t[:, 0] > 0]
    own = t[:, 0].astype(float) / 2                      # team 0's tiles of the CTA
    print(f"workload chunked_prefill: {len(t)} CTAs recorded (the first {MAX_CTAS} of the grid), tiles per CTA median {np.median(t[:, 0]):.0f}")
    print(f"{'phase':<62}{'median':>8}{'min':>8}{'max':>8}   (cycles per tile of team 0)")
    for i, name in PREFILL_PHASES:
        per = t[:, i] / own
        print(f"{name:<62}{np.median(per):8.0f}{per.min():8.0f}{per.max():8.0f}")


if __name__ == "__main__":
    main()
