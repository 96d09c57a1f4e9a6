"""Thin ctypes binding of ``libcoopt.so``: argument marshalling only.

Every function has the name of the C entry point it wraps (without the ``coopt_`` prefix is
also exported for convenience).  Tensors are torch CUDA tensors; their ``data_ptr()`` and the
current torch stream are passed through.  Nothing is computed here, and there is no fallback:
if the shared library is missing or a call returns an error status, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

KV_FP8_E4M3 = 0
KV_BF16 = 1
KV_FP8_E5M2 = 2
BLOCK_SIZE = 16

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libcoopt.so")
_lib: Optional[ctypes.CDLL] = None


class CooptError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: status {status} ({status_string(status)})")


class coopt_cache(ctypes.Structure):
    _fields_ = [("data", ctypes.c_void_p), ("num_blocks", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("block_size", ctypes.c_int32), ("dtype", ctypes.c_int32)]


class coopt_step_layout(ctypes.Structure):
    _fields_ = [(n, ctypes.c_size_t) for n in ("q", "k_new", "v_new", "slot_mapping", "block_table", "context_lens",
                                               "in_bytes", "out", "out_bytes", "total_bytes")]


class coopt_layer_io(ctypes.Structure):
    _fields_ = [("cache", ctypes.POINTER(coopt_cache)), ("k_new", ctypes.c_void_p), ("v_new", ctypes.c_void_p),
                ("slot_mapping", ctypes.c_void_p), ("q", ctypes.c_void_p), ("out", ctypes.c_void_p)]


FLAG_OVERLAP_PREVIOUS = 1

_SIGNATURES = {
    "coopt_granule_bytes": (ctypes.c_size_t, [ctypes.c_int32, ctypes.c_int32]),
    "coopt_cache_bytes": (ctypes.c_size_t, [ctypes.c_int32] * 4),
    "coopt_cache_offset": (ctypes.c_int64, [ctypes.POINTER(coopt_cache)] + [ctypes.c_int32] * 5),
    "coopt_scale_offset": (ctypes.c_int64, [ctypes.POINTER(coopt_cache)] + [ctypes.c_int32] * 3),
    "coopt_kv_write": (ctypes.c_int, [ctypes.POINTER(coopt_cache), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64,
                                      ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p]),
    "coopt_paged_decode": (ctypes.c_int, [ctypes.POINTER(coopt_cache), ctypes.c_void_p, ctypes.c_void_p,
                                          ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p, ctypes.c_int32,
                                          ctypes.c_int32, ctypes.c_float, ctypes.c_void_p, ctypes.c_size_t,
                                          ctypes.c_void_p]),
    "coopt_paged_decode_static": (ctypes.c_int, [ctypes.POINTER(coopt_cache), ctypes.c_void_p, ctypes.c_void_p,
                                                 ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p, ctypes.c_int32,
                                                 ctypes.c_int32, ctypes.c_float, ctypes.c_void_p]),
    "coopt_paged_chunked": (ctypes.c_int, [ctypes.POINTER(coopt_cache), ctypes.c_void_p, ctypes.c_void_p,
                                           ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p,
                                           ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                           ctypes.c_int32, ctypes.c_float, ctypes.c_void_p, ctypes.c_size_t,
                                           ctypes.c_void_p]),
    "coopt_workspace_bytes": (ctypes.c_size_t, [ctypes.c_int32] * 7),
    "coopt_workspace_init": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]),
    "coopt_chunk_partials": (ctypes.c_int, [ctypes.c_int32] * 5 + [ctypes.POINTER(ctypes.c_size_t)] * 3
                             + [ctypes.POINTER(ctypes.c_int32)]),
    "coopt_decode_step_host": (ctypes.c_int, [ctypes.POINTER(coopt_cache), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32,
                                              ctypes.c_int32, ctypes.c_int32, ctypes.c_float, ctypes.c_void_p, ctypes.c_size_t,
                                              ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]),
    "coopt_step_staging_layout": (ctypes.c_int, [ctypes.c_int32] * 5 + [ctypes.c_void_p]),
    "coopt_decode_step": (ctypes.c_int, [ctypes.POINTER(coopt_cache), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64,
                                         ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32,
                                         ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_float, ctypes.c_void_p,
                                         ctypes.c_size_t, ctypes.c_void_p]),
    "coopt_plan_bytes": (ctypes.c_size_t, [ctypes.c_int32] * 4),
    "coopt_decode_plan": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32,
                                         ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]),
    "coopt_decode_step_planned": (ctypes.c_int, [ctypes.POINTER(coopt_cache), ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p,
                                                 ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                                 ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_float,
                                                 ctypes.c_void_p, ctypes.c_size_t, ctypes.c_uint32, ctypes.c_void_p]),
    "coopt_decode_layers": (ctypes.c_int, [ctypes.POINTER(coopt_layer_io), ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p,
                                           ctypes.c_int32, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_float,
                                           ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_uint32,
                                           ctypes.c_void_p]),
    "coopt_selftest_bounded_wait": (ctypes.c_int, [ctypes.c_uint64, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]),
    "coopt_status_string": (ctypes.c_char_p, [ctypes.c_int]),
    "coopt_version": (ctypes.c_int, []),
}


def library_path() -> str:
    return _LIB_PATH


def use_library(path: str) -> None:
    """Bind to another build of the library (the trace build) instead of ``libcoopt.so``; call before any other use."""
    global _lib, _LIB_PATH
    _lib, _LIB_PATH = None, path


def load_library() -> ctypes.CDLL:
    """dlopen ``libcoopt.so`` (built by ``paper_2602_09323_b200.build``) and type its symbols."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: run `python -m paper_2602_09323_b200.build` "
                               "(there is no CPU fallback)")
        lib = ctypes.CDLL(_LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return load_library().coopt_status_string(int(status)).decode()


def _check(status: int, what: str) -> None:
    if status != 0:
        raise CooptError(status, what)


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr(t: torch.Tensor) -> ctypes.c_void_p:
    return ctypes.c_void_p(t.data_ptr())


class Cache:
    """A paged KV cache in device memory plus the C descriptor that names it."""

    def __init__(self, num_blocks: int, num_kv_heads: int, head_dim: int, dtype: int = KV_FP8_E4M3,
                 device: str = "cuda"):
        lib = load_library()
        nbytes = lib.coopt_cache_bytes(num_blocks, num_kv_heads, head_dim, dtype)
        if nbytes == 0:
            raise CooptError(-2, "coopt_cache_bytes")
        self.data = torch.zeros(nbytes, dtype=torch.uint8, device=device)
        self.num_blocks, self.num_kv_heads, self.head_dim, self.dtype = num_blocks, num_kv_heads, head_dim, dtype
        self.granule_bytes = lib.coopt_granule_bytes(head_dim, dtype)
        self.desc = coopt_cache(self.data.data_ptr(), num_blocks, num_kv_heads, head_dim, BLOCK_SIZE, dtype)

    def ref(self):
        return ctypes.byref(self.desc)


def cache_offset(cache: Cache, block: int, kv_head: int, which: int, token: int, dim: int) -> int:
    return load_library().coopt_cache_offset(cache.ref(), block, kv_head, which, token, dim)


def scale_offset(cache: Cache, block: int, kv_head: int, which: int) -> int:
    return load_library().coopt_scale_offset(cache.ref(), block, kv_head, which)


def kv_write(cache: Cache, k: torch.Tensor, v: torch.Tensor, slot_mapping: torch.Tensor) -> None:
    """coopt_kv_write: k, v bf16 [T, Hkv, D] (token stride taken from the tensor), slots int64 [T]."""
    assert k.dtype == torch.bfloat16 and v.dtype == torch.bfloat16 and slot_mapping.dtype == torch.int64
    assert k.is_cuda and v.is_cuda and slot_mapping.is_cuda and slot_mapping.is_contiguous()
    assert k.shape == v.shape and k.stride() == v.stride() and k.stride(2) == 1 and k.stride(1) == k.shape[2]
    st = load_library().coopt_kv_write(cache.ref(), _ptr(k), _ptr(v), k.stride(0) if k.shape[0] > 1 else k.shape[1] * k.shape[2],
                                       _ptr(slot_mapping), k.shape[0], _stream())
    _check(st, "coopt_kv_write")


def workspace_bytes(batch: int, num_q_heads: int, num_kv_heads: int, head_dim: int, max_blocks_per_seq: int,
                    chunk_size: int = 0, total_q: Optional[int] = None) -> int:
    return load_library().coopt_workspace_bytes(batch, num_q_heads, num_kv_heads, head_dim, max_blocks_per_seq,
                                                chunk_size, batch if total_q is None else total_q)


def workspace_init(workspace: torch.Tensor) -> None:
    _check(load_library().coopt_workspace_init(_ptr(workspace), workspace.numel(), _stream()), "coopt_workspace_init")


def new_workspace(batch: int, num_q_heads: int, num_kv_heads: int, head_dim: int, max_blocks_per_seq: int,
                  chunk_size: int = 0, total_q: Optional[int] = None, device: str = "cuda") -> torch.Tensor:
    """Allocate (torch) and initialise a workspace large enough for the given call."""
    n = workspace_bytes(batch, num_q_heads, num_kv_heads, head_dim, max_blocks_per_seq, chunk_size, total_q)
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    workspace_init(ws)
    return ws


def workspace_status(workspace: torch.Tensor) -> int:
    """Device-side status word (synchronises)."""
    return int(workspace[:4].view(torch.int32).item())


def paged_decode(cache: Cache, q: torch.Tensor, block_table: torch.Tensor, context_lens: torch.Tensor,
                 sm_scale: float, workspace: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """coopt_paged_decode: q bf16 [B, Hq, D] -> out bf16 [B, Hq, D]."""
    assert q.dtype == torch.bfloat16 and q.is_contiguous() and q.is_cuda
    assert block_table.dtype == torch.int32 and block_table.is_contiguous() and context_lens.dtype == torch.int32
    if out is None:
        out = torch.empty_like(q)
    st = load_library().coopt_paged_decode(cache.ref(), _ptr(q), _ptr(out), _ptr(block_table), block_table.shape[1],
                                           _ptr(context_lens), q.shape[0], q.shape[1], float(sm_scale),
                                           _ptr(workspace), workspace.numel(), _stream())
    _check(st, "coopt_paged_decode")
    return out


def decode_step(cache: Cache, k_new: torch.Tensor, v_new: torch.Tensor, slot_mapping: torch.Tensor, q: torch.Tensor,
                block_table: torch.Tensor, context_lens: torch.Tensor, sm_scale: float, workspace: torch.Tensor,
                out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """coopt_decode_step: the new token of every sequence written, then decode attention, as one call."""
    assert q.dtype == torch.bfloat16 and q.is_contiguous() and block_table.dtype == torch.int32 and block_table.is_contiguous()
    assert k_new.dtype == torch.bfloat16 and v_new.dtype == torch.bfloat16 and k_new.is_contiguous() and v_new.is_contiguous()
    assert slot_mapping.dtype == torch.int64 and context_lens.dtype == torch.int32
    if out is None:
        out = torch.empty_like(q)
    st = load_library().coopt_decode_step(cache.ref(), _ptr(k_new), _ptr(v_new), k_new.shape[1] * k_new.shape[2], _ptr(slot_mapping),
                                          _ptr(q), _ptr(out), _ptr(block_table), block_table.shape[1], _ptr(context_lens),
                                          q.shape[0], q.shape[1], float(sm_scale), _ptr(workspace), workspace.numel(), _stream())
    _check(st, "coopt_decode_step")
    return out


def plan_bytes(batch: int, num_kv_heads: int, max_blocks_per_seq: int, chunk_size: int = 0) -> int:
    return load_library().coopt_plan_bytes(batch, num_kv_heads, max_blocks_per_seq, chunk_size)


def decode_plan(block_table: torch.Tensor, context_lens: torch.Tensor, num_kv_heads: int, num_blocks: int,
                chunk_size: int = 0, plan: Optional[torch.Tensor] = None) -> torch.Tensor:
    """coopt_decode_plan: the step's work decomposition, into ``plan`` (allocated here if not given)."""
    assert block_table.dtype == torch.int32 and block_table.is_contiguous() and block_table.is_cuda
    assert context_lens.dtype == torch.int32 and context_lens.is_cuda
    batch, width = block_table.shape
    if plan is None:
        plan = torch.empty(plan_bytes(batch, num_kv_heads, width, chunk_size), dtype=torch.uint8, device=block_table.device)
    st = load_library().coopt_decode_plan(_ptr(block_table), width, _ptr(context_lens), batch, num_kv_heads, num_blocks,
                                          int(chunk_size), _ptr(plan), plan.numel(), _stream())
    _check(st, "coopt_decode_plan")
    return plan


def decode_step_planned(cache: Cache, plan: torch.Tensor, q: torch.Tensor, max_blocks_per_seq: int, sm_scale: float,
                        workspace: torch.Tensor, k_new: Optional[torch.Tensor] = None, v_new: Optional[torch.Tensor] = None,
                        slot_mapping: Optional[torch.Tensor] = None, chunk_size: int = 0, flags: int = 0,
                        out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """coopt_decode_step_planned: append (if k_new, v_new, slot_mapping are given) and attend in one launch."""
    assert q.dtype == torch.bfloat16 and q.is_contiguous() and q.is_cuda
    stride = 0
    if k_new is not None:
        assert k_new.dtype == torch.bfloat16 and v_new.dtype == torch.bfloat16 and k_new.is_contiguous() and v_new.is_contiguous()
        assert slot_mapping.dtype == torch.int64 and slot_mapping.is_contiguous()
        stride = k_new.shape[1] * k_new.shape[2]
    if out is None:
        out = torch.empty_like(q)
    null = ctypes.c_void_p(None)
    st = load_library().coopt_decode_step_planned(
        cache.ref(), _ptr(plan), plan.numel(), _ptr(k_new) if k_new is not None else null,
        _ptr(v_new) if v_new is not None else null, stride, _ptr(slot_mapping) if slot_mapping is not None else null,
        _ptr(q), _ptr(out), max_blocks_per_seq, q.shape[0], q.shape[1], int(chunk_size), float(sm_scale), _ptr(workspace),
        workspace.numel(), int(flags), _stream())
    _check(st, "coopt_decode_step_planned")
    return out


class LayerSet:
    """The host array of coopt_layer_io entries of a model's layers, built once (it only holds pointers)."""

    def __init__(self, layers):
        """``layers``: list of dicts with cache, q, out and optionally k_new, v_new, slot_mapping (CUDA tensors)."""
        self.keep = layers
        self.array = (coopt_layer_io * len(layers))()
        for i, L in enumerate(layers):
            io = self.array[i]
            io.cache = ctypes.pointer(L["cache"].desc)
            for name in ("k_new", "v_new", "slot_mapping"):
                t = L.get(name)
                setattr(io, name, t.data_ptr() if t is not None else None)
            io.q, io.out = L["q"].data_ptr(), L["out"].data_ptr()
        k = layers[0].get("k_new")
        self.kv_stride = k.shape[1] * k.shape[2] if k is not None else 0


def decode_layers(layer_set: LayerSet, block_table: torch.Tensor, context_lens: torch.Tensor, num_q_heads: int,
                  sm_scale: float, plan: torch.Tensor, workspace: torch.Tensor, flags: int = 0) -> None:
    """coopt_decode_layers: one plan, then one fused step per layer, enqueued back to back."""
    st = load_library().coopt_decode_layers(layer_set.array, len(layer_set.array), layer_set.kv_stride, _ptr(block_table),
                                            block_table.shape[1], _ptr(context_lens), block_table.shape[0], num_q_heads,
                                            float(sm_scale), _ptr(plan), plan.numel(), _ptr(workspace), workspace.numel(),
                                            int(flags), _stream())
    _check(st, "coopt_decode_layers")


def paged_decode_static(cache: Cache, q: torch.Tensor, block_table: torch.Tensor, context_lens: torch.Tensor,
                        sm_scale: float, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """coopt_paged_decode_static: as ``paged_decode`` but the scratch memory is the fixed array inside
    the library, for callers that cannot allocate a workspace (see the header).  ``out`` is still the
    caller's; pass one in if even the output must not be allocated here."""
    assert q.dtype == torch.bfloat16 and q.is_contiguous() and q.is_cuda
    assert block_table.dtype == torch.int32 and block_table.is_contiguous() and context_lens.dtype == torch.int32
    if out is None:
        out = torch.empty_like(q)
    st = load_library().coopt_paged_decode_static(cache.ref(), _ptr(q), _ptr(out), _ptr(block_table),
                                                  block_table.shape[1], _ptr(context_lens), q.shape[0], q.shape[1],
                                                  float(sm_scale), _stream())
    _check(st, "coopt_paged_decode_static")
    return out


def paged_chunked(cache: Cache, q: torch.Tensor, cu_q_lens: torch.Tensor, block_table: torch.Tensor,
                  context_lens: torch.Tensor, chunk_size: int, causal: bool, sm_scale: float,
                  workspace: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """coopt_paged_chunked: q bf16 [total_q, Hq, D]; cu_q_lens int32 [B + 1] on the device."""
    assert q.dtype == torch.bfloat16 and q.is_contiguous() and q.is_cuda
    assert block_table.dtype == torch.int32 and block_table.is_contiguous()
    assert cu_q_lens.dtype == torch.int32 and context_lens.dtype == torch.int32
    if out is None:
        out = torch.empty_like(q)
    batch = context_lens.shape[0]
    st = load_library().coopt_paged_chunked(cache.ref(), _ptr(q), _ptr(out), _ptr(cu_q_lens), _ptr(block_table),
                                            block_table.shape[1], _ptr(context_lens), batch, q.shape[1], q.shape[0],
                                            int(chunk_size), int(bool(causal)), float(sm_scale), _ptr(workspace),
                                            workspace.numel(), _stream())
    _check(st, "coopt_paged_chunked")
    return out


def chunk_partials(workspace: torch.Tensor, batch: int, num_q_heads: int, head_dim: int, max_blocks_per_seq: int,
                   chunk_size: int):
    """Views (o_c, m_c, l_c) of the per-chunk partials a q_len == 1 chunked call left in the workspace."""
    o, m, l = ctypes.c_size_t(), ctypes.c_size_t(), ctypes.c_size_t()
    mc = ctypes.c_int32()
    _check(load_library().coopt_chunk_partials(batch, num_q_heads, head_dim, max_blocks_per_seq, chunk_size,
                                               ctypes.byref(o), ctypes.byref(m), ctypes.byref(l), ctypes.byref(mc)),
           "coopt_chunk_partials")
    rows = batch * num_q_heads * mc.value
    f = lambda off, n: workspace[off:off + 4 * n].view(torch.float32)
    return (f(o.value, rows * head_dim).view(batch, num_q_heads, mc.value, head_dim),
            f(m.value, rows).view(batch, num_q_heads, mc.value), f(l.value, rows).view(batch, num_q_heads, mc.value))


def selftest_bounded_wait(limit_ns: int):
    """coopt_selftest_bounded_wait: returns (status word, microseconds waited) after synchronising."""
    res = torch.zeros(2, dtype=torch.int32, device="cuda")
    st = load_library().coopt_selftest_bounded_wait(int(limit_ns), ctypes.c_void_p(res.data_ptr()),
                                                    ctypes.c_void_p(res.data_ptr() + 4), _stream())
    _check(st, "coopt_selftest_bounded_wait")
    torch.cuda.synchronize()
    return int(res[0].item()), int(res[1].item())


def step_staging_layout(batch: int, num_q_heads: int, num_kv_heads: int, head_dim: int, max_blocks_per_seq: int) -> coopt_step_layout:
    lay = coopt_step_layout()
    _check(load_library().coopt_step_staging_layout(batch, num_q_heads, num_kv_heads, head_dim, max_blocks_per_seq,
                                                    ctypes.byref(lay)), "coopt_step_staging_layout")
    return lay


def decode_step_host(cache: Cache, step_inputs: torch.Tensor, out: torch.Tensor, max_blocks_per_seq: int, num_q_heads: int,
                     sm_scale: float, staging: torch.Tensor, plan: torch.Tensor, workspace: torch.Tensor) -> None:
    """coopt_decode_step_host: ``step_inputs`` (uint8, packed per step_staging_layout) and ``out`` are HOST tensors
    (page-locked ones are read and written in place by the kernel, pageable ones go through copies); asynchronous:
    ``out`` holds the result once the stream has been synchronised."""
    assert not step_inputs.is_cuda and step_inputs.is_contiguous() and not out.is_cuda and out.is_contiguous()
    st = load_library().coopt_decode_step_host(cache.ref(), _ptr(step_inputs), _ptr(out), max_blocks_per_seq, out.shape[0],
                                               num_q_heads, float(sm_scale), _ptr(staging), staging.numel(), _ptr(plan),
                                               plan.numel(), _ptr(workspace), workspace.numel(), _stream())
    _check(st, "coopt_decode_step_host")
