"""The N > 1 path of the benchmark on CPU: the launcher that starts one process per GPU,
independent replicas, max-over-ranks timing, no collective on the data path.  Two gloo ranks
stand in for two GPUs."""
import json
import os
import subprocess
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


def test_launcher_starts_the_ranks_and_rank_zero_prints_one_line():
    """bench.launch_ranks is what `bench.py --gpus N` calls when no launcher started it; here it
    starts two CPU ranks of a stand-in script that uses the benchmark's rank set-up, its
    max-over-ranks and its throughput formula."""
    sys.path.insert(0, ROOT)
    import bench
    proc = bench.launch_ranks(2, os.path.join(ROOT, "tests", "_rank_standin.py"), ["--gpus", "2"],
                              need_devices=False, capture=True)
    assert proc.returncode == 0, proc.stderr[-2000:]
    lines = [ln for ln in proc.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1                                   # rank 0 alone reports
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["args"] == ["--gpus", "2"]
    assert line["slowest"] == [2.0, 5.0]
    assert line["value"] == pytest.approx(2 * 1000 * 10 / 2.0 / 1e9)


def test_asking_for_more_gpus_than_there_are_fails_loudly():
    """`bench.py --gpus N` never runs fewer replicas than it was asked for."""
    proc = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "1000", "--steps", "1"],
                          stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True,
                          env={k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")})
    assert proc.returncode != 0
    assert "--gpus 1000 was asked for" in proc.stderr and "refusing" in proc.stderr
    assert not any(ln.startswith("{") for ln in proc.stdout.splitlines())
    # a launcher's world size that disagrees with the flag is an error too, not a silent override
    proc = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "4", "--steps", "1"],
                          stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True,
                          env=dict(os.environ, WORLD_SIZE="2", RANK="0", LOCAL_RANK="0"))
    assert proc.returncode != 0 and "disagrees with WORLD_SIZE=2" in proc.stderr


def test_nccl_start_up_log_is_summarised(tmp_path, monkeypatch):
    """What the benchmark reports about the communicator comes from NCCL's own start-up log."""
    sys.path.insert(0, ROOT)
    import bench
    log = tmp_path / ("nccl_host_%d.log" % os.getpid())
    log.write_text("host:1:1 [0] NCCL INFO NCCL version 2.28.9+cuda12.9\n"
                   "host:1:2 [0] NCCL INFO comm 0x55 rank 0 nranks 4 cudaDev 0 nvmlDev 0 busId 1000 commId 0x1 - Init START\n"
                   "host:1:2 [0] NCCL INFO NVLS multicast support is available on dev 0\n"
                   "host:1:2 [0] NCCL INFO comm 0x55 rank 0 nranks 4 cudaDev 0 - Init COMPLETE\n")
    monkeypatch.setenv("NCCL_DEBUG_FILE", str(tmp_path / "nccl_%h_%p.log"))
    got = bench.nccl_log_summary()
    assert got["nranks"] == 4 and got["version"].startswith("2.28.9") and got["nvls"] is True
    monkeypatch.setenv("NCCL_DEBUG_FILE", str(tmp_path / "absent_%h_%p.log"))
    assert bench.nccl_log_summary() == {}
