"""The N > 1 path of the benchmark on CPU: independent replicas, max-over-ranks timing, no
collective on the data path.  Two gloo ranks stand in for two GPUs."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, results):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = [1.0 + rank, 5.0 - rank]                       # rank 1 is slower on the first, faster on the second
    got = bench.max_over_ranks(mine, dist, "cpu")
    value = bench.job_throughput(1000, 10, world, got[0])
    dist.barrier()
    results[rank] = (got, value)
    dist.destroy_process_group()


def test_max_over_ranks_and_job_throughput_two_ranks():
    world, port = 2, 29500 + os.getpid() % 2000
    with mp.Manager() as m:
        results = m.dict()
        mp.spawn(_worker, args=(world, port, results), nprocs=world, join=True)
        for rank in range(world):
            got, value = results[rank]
            assert got == [2.0, 5.0]                      # the slowest replica sets the time
            assert value == pytest.approx(2 * 1000 * 10 / 2.0 / 1e9)


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([0.25, 0.5], None, "cpu") == [0.25, 0.5]
    assert bench.job_throughput(4_000_000_000, 2, 1, 1.0) == pytest.approx(8.0)


def test_reference_arm_runs_on_rank_zero_only(monkeypatch):
    sys.path.insert(0, ROOT)
    import bench
    monkeypatch.setenv("RANK", "1")
    monkeypatch.setenv("WORLD_SIZE", "2")
    args = type("A", (), dict(workload="tiny", steps=1, warmup=0))()
    assert bench.run_reference(args) is None               # other ranks exit without work
    monkeypatch.setenv("RANK", "0")
    line = bench.run_reference(args)
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["gpu_launches"] == 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["value"] > 0
