"""GPU parity of the planned decode path: coopt_decode_plan once, then coopt_decode_step_planned (append +
attention in one launch) or coopt_decode_layers (a model's layers back to back), against the two-call path
bit for bit and against the float64 oracle."""
import numpy as np
import pytest
import torch

from oracle import attention, kv_cache
from paper_2602_09323_b200 import binding, workloads
from tests import helpers

pytestmark = pytest.mark.gpu


def _plan_and_ws(w, chunk=0, num_blocks=None):
    table, lens = w.block_table.cuda(), w.context_lens_tensor.cuda()
    plan = binding.decode_plan(table, lens, w.num_kv_heads, num_blocks or w.num_blocks, chunk)
    ws = binding.new_workspace(w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, table.shape[1], chunk, w.batch)
    return plan, ws, table, lens


@pytest.mark.parametrize("lens,hq,hkv,d", [([700, 15, 2000, 0, 333], 10, 2, 128), ([1, 16, 17, 0, 333], 16, 2, 64),
                                           ([int(x) for x in np.random.default_rng(0).integers(1, 80, 200)], 8, 2, 64),
                                           ([40000], 8, 1, 128), ([2048] * 32, 40, 8, 128)])
def test_planned_call_without_append_equals_the_plain_call(lens, hq, hkv, d):
    w = workloads.make_workload("planned", lens, hq, hkv, d, seed=51)
    cache = helpers.gpu_fill(w)
    want, _ = helpers.gpu_decode(w, cache)
    plan, ws, table, _ = _plan_and_ws(w)
    for rep in range(2):                                   # the plan and the workspace serve any number of launches
        got = binding.decode_step_planned(cache, plan, w.q.cuda(), table.shape[1], w.sm_scale, ws)
        torch.cuda.synchronize()
        assert binding.workspace_status(ws) == 0
        assert torch.equal(got, want), f"launch {rep}"


@pytest.mark.parametrize("chunk", [16, 2048])
def test_planned_chunked_call_equals_the_plain_chunked_call(chunk):
    w = workloads.make_workload("planned_chunks", [1, 100, 777, 2049, 5000], 10, 2, 128, seed=52)
    cache = helpers.gpu_fill(w)
    want, ws0 = helpers.gpu_decode(w, cache, chunk_size=chunk)
    plan, ws, table, _ = _plan_and_ws(w, chunk)
    got = binding.decode_step_planned(cache, plan, w.q.cuda(), table.shape[1], w.sm_scale, ws, chunk_size=chunk)
    torch.cuda.synchronize()
    assert binding.workspace_status(ws) == 0 and torch.equal(got, want)
    for a, b in zip(binding.chunk_partials(ws, w.batch, 10, 128, table.shape[1], chunk),
                    binding.chunk_partials(ws0, w.batch, 10, 128, table.shape[1], chunk)):
        n = [(L + chunk - 1) // chunk for L in w.context_lens]
        for bi, nb in enumerate(n):
            assert torch.equal(a[bi, :, :nb], b[bi, :, :nb])


@pytest.mark.parametrize("hq,hkv,d", [(10, 2, 128), (16, 2, 64), (4, 4, 128)])
def test_fused_step_equals_write_then_decode_bit_for_bit(hq, hkv, d):
    """Token by token over the last 40 positions of every sequence (block boundaries are crossed, scales grow
    and resident codes are re-expressed, a block is opened anew): the one-launch step and the two separate
    calls must leave identical cache bytes and identical outputs; the outputs match the oracle at the end.
    Sequence 4 is skipped every third step through a negative slot (Eq. 5)."""
    w = workloads.make_workload("fused", [300, 64, 2048, 1500, 47, 900], hq, hkv, d, seed=17)
    steps = 40
    rows = np.concatenate([np.arange(w.kv_offsets[b], w.kv_offsets[b] + L - steps) for b, L in enumerate(w.context_lens)])
    rows_t = torch.from_numpy(rows).cuda()
    k, v, slots = w.k.cuda(), w.v.cuda(), w.slot_mapping.cuda()
    table, q = w.block_table.cuda(), w.q.cuda()
    caches = []
    for _ in range(2):
        c = binding.Cache(w.num_blocks, hkv, d)
        binding.kv_write(c, k[rows_t], v[rows_t], slots[rows_t])
        caches.append(c)
    ws = [binding.new_workspace(w.batch, hq, hkv, d, table.shape[1]) for _ in range(2)]
    plan = torch.empty(binding.plan_bytes(w.batch, hkv, table.shape[1]), dtype=torch.uint8, device="cuda")
    outs = [None, None]
    skipped = []
    for step in range(steps):
        new = torch.tensor([w.kv_offsets[b] + L - steps + step for b, L in enumerate(w.context_lens)]).cuda()
        lens = torch.tensor([L - steps + step + 1 for L in w.context_lens], dtype=torch.int32).cuda()
        k_new, v_new, s_new = k[new].contiguous(), v[new].contiguous(), slots[new].contiguous()
        if step % 3 == 1:
            s_new[4] = -1
            skipped.append(int(new[4]))
        binding.decode_plan(table, lens, hkv, w.num_blocks, plan=plan)
        outs[0] = binding.decode_step_planned(caches[0], plan, q, table.shape[1], w.sm_scale, ws[0], k_new, v_new, s_new)
        binding.kv_write(caches[1], k_new, v_new, s_new)
        outs[1] = binding.paged_decode(caches[1], q, table, lens, w.sm_scale, ws[1])
        torch.cuda.synchronize()
        assert binding.workspace_status(ws[0]) == 0 and binding.workspace_status(ws[1]) == 0
        assert torch.equal(caches[0].data, caches[1].data), f"step {step}: cache bytes differ"
        assert torch.equal(outs[0], outs[1]), f"step {step}: outputs differ"
    codes, scales = kv_cache.new_cache(w.num_blocks, hkv, d)
    kf, vf, sf = w.k.float().numpy(), w.v.float().numpy(), w.slot_mapping.numpy().copy()
    sf[skipped] = -1
    kv_cache.kv_write(codes, scales, kf[rows], vf[rows], sf[rows])
    for step in range(steps):
        new = np.array([w.kv_offsets[b] + L - steps + step for b, L in enumerate(w.context_lens)])
        kv_cache.kv_write(codes, scales, kf[new], vf[new], sf[new])
    helpers.check_cache_bit_exact(caches[0], codes, scales, what="fused step")
    ref = attention.paged_attention(w.q.float().numpy(), (codes, scales), w.block_table.numpy(), w.context_lens)
    # skipped tokens left zero codes in their slots on both sides; the oracle reads them like the kernel does
    helpers.check_attention(outs[0], ref, what="fused step")


@pytest.mark.parametrize("flags", [0, binding.FLAG_OVERLAP_PREVIOUS])
def test_layers_call_equals_layer_by_layer_calls(flags):
    """Four layers share block table, context lengths, plan and workspace; each has its own cache, new token
    and query.  Every layer's cache bytes and output must equal coopt_kv_write + coopt_paged_decode on that
    layer, with and without letting a layer start while the one before it drains, on two steps in a row."""
    n_layers, hq, hkv, d = 4, 10, 2, 128
    base = workloads.make_workload("layers", [300, 64, 2048, 1500, 47, 900, 17, 3], hq, hkv, d, seed=61)
    table = base.block_table.cuda()
    max_blocks = table.shape[1]
    ws = binding.new_workspace(base.batch, hq, hkv, d, max_blocks)
    ws2 = binding.new_workspace(base.batch, hq, hkv, d, max_blocks)
    plan = torch.empty(binding.plan_bytes(base.batch, hkv, max_blocks), dtype=torch.uint8, device="cuda")
    lens_full = base.context_lens
    layers = []
    for l in range(n_layers):
        w = workloads.make_workload("layers", lens_full, hq, hkv, d, seed=61 + 100 * l)   # other values, the base's placement
        w = workloads.Workload(**{**w.__dict__, "block_table": base.block_table, "slot_mapping": base.slot_mapping,
                                  "num_blocks": base.num_blocks})
        layers.append(w)
    for step in range(2):
        lens_now = [L - 1 + step for L in lens_full]          # step 0 appends position L - 2, step 1 position L - 1
        lens_t = torch.tensor(lens_now, dtype=torch.int32).cuda()
        new_rows = torch.tensor([base.kv_offsets[b] + L - 1 for b, L in enumerate(lens_now)])
        ios, want = [], []
        for l, w in enumerate(layers):
            if step == 0:
                hist = np.concatenate([np.arange(base.kv_offsets[b], base.kv_offsets[b] + L - 2) for b, L in enumerate(lens_full)])
                w.cache_a = helpers.gpu_fill(w, calls=[hist])
                w.cache_b = helpers.gpu_fill(w, calls=[hist])
            k_new, v_new = w.k[new_rows].contiguous().cuda(), w.v[new_rows].contiguous().cuda()
            s_new = w.slot_mapping[new_rows].contiguous().cuda()
            q = w.q.cuda()
            ios.append({"cache": w.cache_a, "k_new": k_new, "v_new": v_new, "slot_mapping": s_new, "q": q,
                        "out": torch.full_like(q, float("nan"))})
            binding.kv_write(w.cache_b, k_new, v_new, s_new)
            want.append(binding.paged_decode(w.cache_b, q, table, lens_t, w.sm_scale, ws2))
        binding.decode_layers(binding.LayerSet(ios), table, lens_t, hq, base.sm_scale, plan, ws, flags)
        torch.cuda.synchronize()
        assert binding.workspace_status(ws) == 0
        for l, w in enumerate(layers):
            assert torch.equal(w.cache_a.data, w.cache_b.data), f"step {step} layer {l}: cache bytes differ"
            assert torch.equal(ios[l]["out"], want[l]), f"step {step} layer {l}: outputs differ"
    # the last layer against the oracle
    w = layers[-1]
    hist = np.concatenate([np.arange(base.kv_offsets[b], base.kv_offsets[b] + L - 2) for b, L in enumerate(lens_full)])
    calls = [hist] + [np.array([base.kv_offsets[b] + L - 2 + s for b, L in enumerate(lens_full)]) for s in range(2)]
    codes, scales = helpers.oracle_fp8_cache(w, calls=calls)
    ref = attention.paged_attention(w.q.float().numpy(), (codes, scales), w.block_table.numpy(), lens_full)
    helpers.check_attention(ios[-1]["out"], ref, what="layers")


def test_a_plan_of_another_problem_and_a_misplaced_slot_are_reported():
    w = workloads.make_workload("mismatch", [300, 90, 1000], 10, 2, 128, seed=71)
    cache = helpers.gpu_fill(w)
    plan, ws, table, lens = _plan_and_ws(w)
    # a plan made for a cache with another number of blocks
    other = binding.decode_plan(table, lens, w.num_kv_heads, w.num_blocks + 1)
    out = torch.full_like(w.q.cuda(), 7.0)
    binding.decode_step_planned(cache, other, w.q.cuda(), table.shape[1], w.sm_scale, ws, out=out)
    torch.cuda.synchronize()
    assert binding.workspace_status(ws) == -1
    assert (out == 7).all()                                  # the launch did nothing
    binding.workspace_init(ws)
    # the new token's slot does not name the sequence's last position
    last = torch.tensor([w.kv_offsets[b] + L - 1 for b, L in enumerate(w.context_lens)])
    k_new, v_new = w.k[last].contiguous().cuda(), w.v[last].contiguous().cuda()
    s_bad = w.slot_mapping[last].clone()
    s_bad[1] = w.slot_mapping[w.kv_offsets[1]]               # first position of sequence 1 instead of its last
    binding.decode_step_planned(cache, plan, w.q.cuda(), table.shape[1], w.sm_scale, ws, k_new, v_new, s_bad.cuda())
    torch.cuda.synchronize()
    assert binding.workspace_status(ws) == -1


@pytest.mark.parametrize("pinned", [True, False])
def test_host_step_equals_the_planned_step_bit_for_bit(pinned):
    """coopt_decode_step_host with page-locked buffers (queries and new tokens read in place, result stored in
    place) and with pageable ones (staged through copies): cache bytes and outputs identical to coopt_decode_plan +
    coopt_decode_step_planned on device tensors, and within tolerance of the oracle."""
    hq, hkv, d = 10, 2, 128
    w = workloads.make_workload("host_step", [300, 64, 2048, 1500, 47, 900, 17, 1], hq, hkv, d, seed=23)
    hist = np.concatenate([np.arange(w.kv_offsets[b], w.kv_offsets[b] + L - 1) for b, L in enumerate(w.context_lens)])
    new = torch.tensor([w.kv_offsets[b] + L - 1 for b, L in enumerate(w.context_lens)])
    k_new, v_new, s_new = w.k[new].contiguous(), w.v[new].contiguous(), w.slot_mapping[new].contiguous()
    table = w.block_table.clamp(min=0)
    max_blocks = table.shape[1]
    lay = binding.step_staging_layout(w.batch, hq, hkv, d, max_blocks)
    host_in = torch.zeros(lay.in_bytes, dtype=torch.uint8)
    for off, t in ((lay.q, w.q), (lay.k_new, k_new), (lay.v_new, v_new), (lay.slot_mapping, s_new), (lay.block_table, table),
                   (lay.context_lens, w.context_lens_tensor)):
        raw = t.contiguous().view(torch.uint8).reshape(-1)
        host_in[off:off + raw.numel()] = raw
    host_out = torch.full_like(w.q, float("nan"))
    if pinned:
        host_in, host_out = host_in.pin_memory(), host_out.pin_memory()
    staging = torch.empty(lay.total_bytes, dtype=torch.uint8, device="cuda")
    plan = torch.empty(binding.plan_bytes(w.batch, hkv, max_blocks), dtype=torch.uint8, device="cuda")
    ws = binding.new_workspace(w.batch, hq, hkv, d, max_blocks)
    cache_a, cache_b = helpers.gpu_fill(w, calls=[hist]), helpers.gpu_fill(w, calls=[hist])
    binding.decode_step_host(cache_a, host_in, host_out, max_blocks, hq, w.sm_scale, staging, plan, ws)
    torch.cuda.synchronize()
    assert binding.workspace_status(ws) == 0
    plan_b = binding.decode_plan(table.cuda(), w.context_lens_tensor.cuda(), hkv, w.num_blocks)
    want = binding.decode_step_planned(cache_b, plan_b, w.q.cuda(), max_blocks, w.sm_scale, ws, k_new.cuda(), v_new.cuda(), s_new.cuda())
    torch.cuda.synchronize()
    assert torch.equal(cache_a.data, cache_b.data)
    assert torch.equal(host_out.cuda(), want)
    codes, scales = helpers.oracle_fp8_cache(w, calls=[hist, new.numpy()])
    ref = attention.paged_attention(w.q.float().numpy(), (codes, scales), w.block_table.numpy(), w.context_lens)
    helpers.check_attention(host_out, ref, what=f"host step, {'page-locked' if pinned else 'pageable'} buffers")
