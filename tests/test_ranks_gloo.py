"""Two CPU processes (gloo) exercise the benchmark's multi-rank arithmetic: the step time is the
maximum over ranks, throughput counts every rank's work, images are dealt out without overlap, and
only rank 0 of the reference arm does anything."""
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2411_00288_b200 import ranks

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), LOCAL_RANK=str(rank),
                      WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert ranks.env_ranks() == (rank, rank, world)
        ms = ranks.max_over_ranks(1.0 + 2.0 * rank, torch.device("cpu"))  # rank 1 is the slow one
        out[rank] = (ms, ranks.job_throughput(10.0, world, ms), ranks.shard_images(33, world, rank))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_max_time_and_throughput():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    assert set(out.keys()) == {0, 1}
    for r in range(world):
        ms, thr, _ = out[r]
        assert ms == 3.0                        # the maximum, on every rank
        assert abs(thr - 2 * 10.0 / 3e-3) < 1e-6  # both ranks' work over the slowest rank's time
    (a0, a1), (b0, b1) = out[0][2], out[1][2]
    assert (a0, a1, b0, b1) == (0, 17, 17, 33)  # contiguous, disjoint, complete


def test_single_process_needs_no_group():
    assert ranks.max_over_ranks(2.5, torch.device("cpu")) == 2.5
    assert ranks.shard_images(32, 1, 0) == (0, 32)
    assert [ranks.shard_images(10, 4, r) for r in range(4)] == [(0, 3), (3, 6), (6, 8), (8, 10)]


def test_reference_arm_other_ranks_exit_quietly():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "1"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
