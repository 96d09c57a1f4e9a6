"""Device-side error reporting: problems found by a kernel end up in the workspace status word (or the
status word handed to the self-test), nothing faults, and the context stays usable."""
import pytest
import torch

from oracle import attention
from paper_2602_09323_b200 import binding, workloads
from tests import helpers

pytestmark = pytest.mark.gpu


def test_out_of_range_block_id_is_reported_and_never_dereferenced():
    """One entry of a valid context names a block the cache does not have, another is negative: the
    kernel substitutes block 0 for both (so the output is finite), reports COOPT_ERR_INVALID_ARG in the
    status word, and the same workspace serves a correct call once it has been initialised again."""
    w = workloads.make_workload("bad_id", [300, 90, 1000], 10, 2, 128, seed=41)
    cache = helpers.gpu_fill(w)
    q, lens = w.q.cuda(), w.context_lens_tensor.cuda()
    bad = w.block_table.clone()
    bad[0, 3] = w.num_blocks + 7
    bad[2, 40] = -5
    ws = binding.new_workspace(w.batch, 10, 2, 128, w.block_table.shape[1])
    out = binding.paged_decode(cache, q, bad.cuda(), lens, w.sm_scale, ws)
    torch.cuda.synchronize()
    assert binding.workspace_status(ws) == -1 and "invalid" in binding.status_string(-1)
    assert torch.isfinite(out.float()).all()
    binding.workspace_init(ws)
    good = binding.paged_decode(cache, q, w.block_table.cuda(), lens, w.sm_scale, ws)
    torch.cuda.synchronize()
    assert binding.workspace_status(ws) == 0
    codes, scales = helpers.oracle_fp8_cache(w)
    ref = attention.paged_attention(w.q.float().numpy(), (codes, scales), w.block_table.numpy(), w.context_lens)
    helpers.check_attention(good, ref, what="after a reported bad id")
    assert torch.equal(out[1], good[1])            # the sequence without a bad entry was not disturbed


def test_chunked_call_with_an_uneven_split_of_the_same_total_is_reported():
    """total_q == batch does not by itself mean one query token per sequence: q_lens = [2, 0, 1] has the same
    total as [1, 1, 1].  The decode-style path is only valid for the latter and says so in the status word."""
    w = workloads.make_workload("uneven", [100, 50, 70], 8, 2, 64, seed=43)
    cache = helpers.gpu_fill(w)
    ws = binding.new_workspace(3, 8, 2, 64, w.block_table.shape[1], 64, 3)
    cu = torch.tensor([0, 2, 2, 3], dtype=torch.int32).cuda()
    binding.paged_chunked(cache, w.q.cuda(), cu, w.block_table.cuda(), w.context_lens_tensor.cuda(), 64, True, w.sm_scale, ws)
    torch.cuda.synchronize()
    assert binding.workspace_status(ws) == -1
    binding.workspace_init(ws)
    binding.paged_chunked(cache, w.q.cuda(), w.cu_q_lens.cuda(), w.block_table.cuda(), w.context_lens_tensor.cuda(), 64, True,
                          w.sm_scale, ws)
    torch.cuda.synchronize()
    assert binding.workspace_status(ws) == 0


def test_a_bounded_wait_that_runs_out_reports_a_timeout_and_returns():
    """The wait used by every role of the tcgen05 kernels, on a barrier nobody arrives on, with a 1 ms limit:
    the warp gives up, the status word says COOPT_ERR_TIMEOUT, and the device keeps working."""
    status, waited_us = binding.selftest_bounded_wait(1_000_000)
    assert status == -5 and "timed out" in binding.status_string(status)
    assert 900 <= waited_us < 50_000
    x = torch.arange(1024, device="cuda").sum().item()      # the context is still usable
    assert x == 1023 * 512
