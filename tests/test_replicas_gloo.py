"""The multi-GPU path is N independent replicas whose only shared step is timing; its host logic
(barrier, max over ranks, whole-job throughput, rank-0 reporting) runs here as two gloo ranks on CPU."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), LOCAL_RANK=str(rank),
                      WORLD_SIZE=str(world))
    from paper_1901_05350_b200 import replicas

    assert replicas.env_rank_world() == (rank, rank, world)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        replicas.barrier()
        mine = 10.0 + 5.0 * rank          # rank 1 is the slow one: 15 ms
        slowest = replicas.max_over_ranks(mine)
        value = replicas.whole_job_throughput(units_per_rank_per_step=128, steps=3, elapsed_ms_this_rank=mine)
        replicas.barrier()
        with open(os.path.join(out_dir, f"rank{rank}.txt"), "w") as fh:
            fh.write(f"{slowest} {value}")
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_whole_job(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    for rank in range(world):
        slowest, value = map(float, open(tmp_path / f"rank{rank}.txt").read().split())
        assert slowest == 15.0
        assert value == pytest.approx(2 * 128 * 3 / 15e-3)


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    from paper_1901_05350_b200 import replicas

    assert replicas.max_over_ranks(7.5) == 7.5
    assert replicas.whole_job_throughput(128, 2, 4.0) == pytest.approx(128 * 2 / 4e-3)
    replicas.barrier()


def test_reference_arm_runs_on_rank_zero_only(tmp_path):
    """Under torchrun the reference arm prints one line from rank 0; other ranks exit 0 silently."""
    import subprocess

    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0", "--gpus", "2"], env=env, capture_output=True, text=True, timeout=120)
    assert res.returncode == 0 and res.stdout.strip() == ""
