"""The N > 1 logic of bench.py on CPU ranks (gloo): the slowest rank's time decides, the job's value is the
sum of the ranks' work over that time, and the reference arm runs on rank 0 only.  The data path itself is
replicas only -- no collective -- so there is nothing else to exchange."""
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
        ms = bench.max_over_ranks(10.0 + 5.0 * rank, "cpu")         # rank 1 is the slow one
        out[rank] = (ms, bench.whole_job_value(3.0e12, ms, world))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_value_on_two_gloo_ranks():
    world, port = 2, 29000 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        got = dict(out)
    for rank in range(world):
        ms, value = got[rank]
        assert ms == 15.0                                  # the maximum over ranks, on every rank
        assert value == pytest.approx(2 * 3.0e12 / 15e-3 / 1e12)


def test_max_over_ranks_is_identity_without_a_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(7.5, "cpu") == 7.5
    assert bench.whole_job_value(1e12, 1000.0, 1) == pytest.approx(1.0)


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
