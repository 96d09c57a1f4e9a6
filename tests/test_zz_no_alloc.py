"""coopt_paged_decode_static: the decode call for users who cannot give the library a workspace
because they cannot allocate device memory where they call from (a plug-in's enqueue hook, a
server whose pool already owns the whole device, a bare C host program).  Its scratch is a fixed
array inside the library, shared by all calls, so the checks are: same result as the ordinary
call, still the same on a second call that finds the first call's leftovers in the array, and a
clear refusal when the problem needs more scratch than the array has."""
import ctypes

import pytest
import torch

from oracle import attention
from paper_2602_09323_b200 import binding, build, workloads
from tests import helpers

STATIC_SCRATCH_BYTES = 4 * 1024 * 1024


def test_problems_beyond_the_built_in_scratch_are_refused_on_the_host():
    build.build()
    lib = binding.load_library()
    cache = binding.coopt_cache(0x1000, 4, 8, 128, 16, 0)
    # 512 sequences x 8 kv heads x 32768 blocks: the split plan alone needs far more than 4 MiB
    assert lib.coopt_workspace_bytes(512, 40, 8, 128, 32768, 0, 512) > STATIC_SCRATCH_BYTES
    rc = lib.coopt_paged_decode_static(ctypes.byref(cache), 0x100, 0x100, 0x100, 32768, 0x100, 512, 40, 0.1, None)
    assert rc == -3 and "workspace" in binding.status_string(rc)
    assert lib.coopt_paged_decode_static(None, 0x100, 0x100, 0x100, 8, 0x100, 2, 8, 0.1, None) == -1


def test_every_other_refusal_also_comes_before_the_shared_array_is_touched():
    """Bad arguments are turned away by the host checks, which run before the array's address is even
    looked up: these calls need no GPU, so nothing can have been enqueued."""
    build.build()
    lib = binding.load_library()
    ok = binding.coopt_cache(0x1000, 4, 8, 128, 16, 0)
    call = lambda c, q, hq: lib.coopt_paged_decode_static(ctypes.byref(c), q, 0x100, 0x100, 8, 0x100, 2, hq, 0.1, None)
    assert call(ok, None, 40) == -1                                           # null q
    assert call(ok, 0x100, 42) == -2                                          # 42 query heads over 8 kv heads
    assert call(ok, 0x100, 8 * 9) == -2                                       # group size 9
    assert call(binding.coopt_cache(0x1000, 4, 8, 96, 16, 0), 0x100, 40) == -2    # head_dim 96
    assert call(binding.coopt_cache(0x1000, 4, 8, 128, 32, 0), 0x100, 40) == -2   # block size 32
    assert call(binding.coopt_cache(0x1001, 4, 8, 128, 16, 0), 0x100, 40) == -1   # misaligned cache


@pytest.mark.gpu
def test_static_scratch_variant_matches_the_workspace_variant_twice_in_a_row():
    """Both entry points run the same kernel with the same split plan, so the outputs must be equal bit for
    bit -- on the first call, and on a second call that finds the first one's leftovers in the array -- and
    they must match the float64 oracle like every other decode result."""
    w = workloads.make_workload("no_alloc", [700, 15, 2000, 0, 333], 10, 2, 128, seed=21)
    cache = helpers.gpu_fill(w)
    want, _ = helpers.gpu_decode(w, cache)                      # ordinary entry point, caller's workspace
    q, table, lens = w.q.cuda(), w.block_table.cuda(), w.context_lens_tensor.cuda()
    codes, scales = helpers.oracle_fp8_cache(w)
    ref = attention.paged_attention(w.q.float().numpy(), (codes, scales), w.block_table.numpy(), w.context_lens)
    for call in range(2):
        out = torch.full_like(q, float("nan"))
        binding.paged_decode_static(cache, q, table, lens, w.sm_scale, out=out)
        torch.cuda.synchronize()
        assert torch.equal(out, want), f"call {call}: differs from the workspace variant"
        helpers.check_attention(out, ref, what=f"static scratch, call {call}")
    # a different problem right after, through the same array
    w2 = workloads.config_tiny(seed=3)
    cache2 = helpers.gpu_fill(w2)
    want2, _ = helpers.gpu_decode(w2, cache2)
    got2 = binding.paged_decode_static(cache2, w2.q.cuda(), w2.block_table.cuda(), w2.context_lens_tensor.cuda(),
                                       w2.sm_scale)
    torch.cuda.synchronize()
    assert torch.equal(got2, want2)
