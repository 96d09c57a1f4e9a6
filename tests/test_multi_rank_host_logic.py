"""The N > 1 path of the benchmark on CPU: two gloo ranks, each with its own timings; the job's number
comes from the slowest rank and counts every rank's tokens (the path shards by sequence, no exchange),
and the reference arm runs on rank 0 only."""
import json
import os
import subprocess
import sys

import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local = [10.0 + 5.0 * rank, 0.040 + 0.010 * (world - 1 - rank)]      # rank 1 is slower on [0], rank 0 on [1]
    got = bench.max_over_ranks(local)
    dist.barrier()
    value = bench.job_tokens_per_second(world, 32, 100, got[0])
    out.put((rank, got, value))
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_timing_and_the_job_value():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29000 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, value in res:
        assert got == [15.0, 0.050]                               # element-wise maximum over the two ranks
        assert abs(value - 2 * 32 * 100 / 15.0e-3) < 1e-6         # both ranks' tokens over the slowest rank's time


def test_single_process_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.0, 4.0]) == [3.0, 4.0]
    assert bench.job_tokens_per_second(1, 32, 10, 2.0) == 32 * 10 / 2.0e-3


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
