"""The N>1 path of the benchmark on CPU: two gloo ranks (no GPU).  The hot path shards by sequence with no data-path
collective; what crosses ranks is only the max of the device-timed duration."""
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms = bench.dist_max(1.0 + rank, torch.device("cpu"), world)       # rank 1 is the slow one
        out[rank] = (ms, bench.whole_job_tokens_per_s(world, 4, ms), bench.shard_plan(world, 4))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_take_the_max_time_and_sum_the_tokens():
    world = 2
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for r in (0, 1):
        ms, value, plan = res[r]
        assert ms == 2.0                                   # max over ranks, identical on both
        assert value == pytest.approx(2 * 4 / 2.0e-3)      # whole-job tokens/s
        assert plan["scaling"] == "weak" and plan["total_sequences"] == 8 and plan["collective"] is None


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1", MASTER_ADDR="127.0.0.1", MASTER_PORT="29999")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0 and p.stdout.strip() == ""
