"""A stand-in for one rank of the benchmark, for the launcher test on a machine without
GPUs: it goes through the benchmark's own rank set-up (gloo instead of NCCL), reports a
made-up step time that depends on the rank, takes the maximum over ranks with the benchmark's
own function and lets rank 0 print one JSON line."""
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402


def main() -> None:
    world, rank, local, dist = bench.init_ranks("gloo")
    mine = [1.0 + rank, 5.0 - rank]                       # the last rank is slowest on the first, fastest on the second
    got = bench.max_over_ranks(mine, dist, "cpu")
    value = bench.job_throughput(1000, 10, world, got[0])
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"n_gpus": world, "slowest": got, "value": value, "args": sys.argv[1:],
                          "local_rank": local}), flush=True)


if __name__ == "__main__":
    main()
