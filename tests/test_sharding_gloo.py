"""One rank per device, the host side on CPU: four gloo ranks in two groups (3 + 1) each ask
the library for their own share of every bucket (pure host calls, no GPU) and exchange what
they got; together the members of a group must own every transport element of the bucket
exactly once, in member order, and agree with the oracle."""
import os
import sys

import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, results):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    from oracle import kt_oracle as oracle
    from paper_2505_10183_b200 import binding as kt
    from paper_2505_10183_b200 import workloads as W
    dist.init_process_group("gloo", rank=rank, world_size=world)
    group_of = [0, 0, 1, 0]
    members = [r for r in range(world) if group_of[r] == group_of[rank]]
    me = members.index(rank)
    wl = W.mobilenet_v2()
    cap = 2 << 20                                           # several buckets
    unit = kt.kt_work_unit(kt.KT_F32)
    plan = kt.kt_plan_buckets(wl.numel, cap)
    mine = {}
    for b in [-1] + list(range(plan.n_buckets)):
        got = kt.kt_shard_ranges(wl.numel, cap, unit, b, len(members))
        assert got == oracle.shard_ranges(wl.numel, cap, unit, b, len(members))
        mine[b] = got[me]
    everyone = [None] * world
    dist.all_gather_object(everyone, (group_of[rank], me, mine))
    ok = True
    for g in (0, 1):
        shares = sorted((m, r) for gg, m, r in everyone if gg == g)
        for b in [-1] + list(range(plan.n_buckets)):
            lo = 0 if b < 0 else plan.bucket_start[b]
            n = plan.transport_numel if b < 0 else plan.bucket_numel[b]
            at = lo
            for _, ranges in shares:                        # member order: each share starts where the last ended
                s, c = ranges[b]
                ok = ok and (c == 0 or s == at)
                at += c
            ok = ok and at == lo + n
    results[rank] = (ok, plan.n_buckets)
    dist.barrier()
    dist.destroy_process_group()


def test_four_ranks_own_every_element_once():
    world, port = 4, 29700 + os.getpid() % 2000
    with mp.Manager() as m:
        results = m.dict()
        mp.spawn(_rank, args=(world, port, results), nprocs=world, join=True)
        assert all(results[r][0] for r in range(world))
        assert results[0][1] >= 3
