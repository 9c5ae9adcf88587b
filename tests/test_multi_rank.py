"""The N > 1 logic of bench.py on CPU ranks (gloo): the slowest rank's time decides, the job's value is the
sum of the ranks' work over that time, and the reference arm runs on rank 0 only.  The data path itself is
replicas only -- no collective.  The one exchange the method itself implies (one scale per tensor, so the amax of a
sharded tensor is MAX-reduced) is `dp.allreduce_amax`, checked here on two ranks against the unsharded tensors."""
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


def _amax_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import numpy as np
    from oracle import tweo_oracle as orc
    from paper_2511_23225_b200 import dp, synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # X [M, K] with an outlier channel and dY [M, N], tokens sharded over the ranks; W replicated
        x = synth.normal_with_outlier_channels_bf16(900, (64, 96))
        dy = synth.normal_bf16(901, (64, 80), 1e-3)
        w = synth.normal_bf16(902, (80, 96), 0.02)
        rows = slice(rank * 32, (rank + 1) * 32)
        local = torch.tensor([float(orc.amax_bf16(x[rows])), float(orc.amax_bf16(w)), float(orc.amax_bf16(dy[rows]))])
        before = local.clone()
        dp.allreduce_amax(local)
        # delayed scaling on the exchanged values: every rank must arrive at the scales of the unsharded tensors
        scales = []
        for v, fmt in zip(local.tolist(), (orc.E4M3, orc.E4M3, orc.E5M2)):
            hist = np.zeros(16, dtype=np.float32)
            scales.append(float(orc.delayed_scaling_update(hist, np.float32(v), fmt, np.float32(1.0))[0]))
        out[rank] = (before.tolist(), local.tolist(), scales)
    finally:
        dist.destroy_process_group()


def test_amax_exchange_gives_every_rank_the_scales_of_the_unsharded_tensors():
    import numpy as np
    from oracle import tweo_oracle as orc
    from paper_2511_23225_b200 import synth
    world, port = 2, 31000 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_amax_worker, args=(world, port, out), nprocs=world, join=True)
        got = dict(out)
    x = synth.normal_with_outlier_channels_bf16(900, (64, 96))
    dy = synth.normal_bf16(901, (64, 80), 1e-3)
    w = synth.normal_bf16(902, (80, 96), 0.02)
    full = [float(orc.amax_bf16(t)) for t in (x, w, dy)]
    want = [float(orc.scale_from_amax(np.float32(a), f)[0]) for a, f in zip(full, (orc.E4M3, orc.E4M3, orc.E5M2))]
    assert got[0][0] != got[1][0]                          # the shards do differ in their maxima
    for rank in range(world):
        assert got[rank][1] == full                        # amax of the whole tensor, on every rank
        assert got[rank][2] == want                        # hence one scale per tensor


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
