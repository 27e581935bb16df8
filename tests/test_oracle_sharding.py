"""Pins of the oracle's one-rank-per-device functions (shard_ranges, sharded_sync_step):
a hand-worked case, brute-force re-derivation from the definition, closed forms, and the
invariant that sharding changes who computes an element, never its value."""
import random

import numpy as np
import pytest

from paper_2505_10183_b200 import workloads as W

F32, BF16 = 0, 1


def units_by_brute_force(oracle, numel, cap, unit, bucket):
    """All work units of a range as (start, length), in transport order, written straight from
    the definition: tensors in reverse list order, each owning the transport from its offset to
    the next tensor's offset, cut every `unit` elements from its own start."""
    plan = oracle.bucket_plan(numel, cap)
    order = list(range(len(numel) - 1, -1, -1))
    units = []
    for i, t in enumerate(order):
        if bucket >= 0 and plan.bucket_of[t] != bucket:
            continue
        start = int(plan.tensor_offset[t])
        end = int(plan.tensor_offset[order[i + 1]]) if i + 1 < len(order) else plan.transport_numel
        at = start
        while at < end:
            units.append((at, min(unit, end - at)))
            at += unit
    return units, plan


def test_hand_worked_case(oracle):
    # six tensors; in the transport (reverse list order, 8-element alignment) they sit at
    #   432 @ 0, 16 @ 432, 4608 @ 448, 32 @ 5056, 5120 @ 5088, 10 @ 10208, total 10240.
    # Units of 2048: 1 + 1 + 3 (2048, 2048, 512) + 1 + 3 (2048, 2048, 1024) + 1 (32, padding included) = 10.
    numel = [10, 5120, 32, 4608, 16, 432]
    assert oracle.bucket_plan(numel, 25 << 20).tensor_offset.tolist() == [10208, 5088, 5056, 448, 432, 0]
    # two members: units 0-4 and 5-9
    assert oracle.shard_ranges(numel, 25 << 20, 2048, -1, 2) == [(0, 5056), (5056, 5184)]
    # three members: units 0-2, 3-5, 6-9  (floor(10/3) = 3, floor(20/3) = 6)
    assert oracle.shard_ranges(numel, 25 << 20, 2048, -1, 3) == [(0, 2496), (2496, 2592), (5088, 5152)]
    # one member owns everything; ten members one unit each; twenty: every second one is empty
    assert oracle.shard_ranges(numel, 25 << 20, 2048, -1, 1) == [(0, 10240)]
    ten = oracle.shard_ranges(numel, 25 << 20, 2048, -1, 10)
    assert [n for _, n in ten] == [432, 16, 2048, 2048, 512, 32, 2048, 2048, 1024, 32]
    twenty = oracle.shard_ranges(numel, 25 << 20, 2048, -1, 20)
    assert [n for _, n in twenty] == [0, 432, 0, 16, 0, 2048, 0, 2048, 0, 512, 0, 32, 0, 2048, 0, 2048, 0, 1024, 0, 32]


def test_single_flat_tensor_closed_form(oracle):
    # one tensor of n elements: extent = n rounded up to 64, U = ceil(extent / unit);
    # member m owns [floor(mU/M) * unit, min(floor((m+1)U/M) * unit, extent))
    for n, unit, M in ((100, 2048, 4), (1 << 20, 2048, 4), (1 << 20, 4096, 3), (1_000_003, 2048, 7), (5000, 4096, 2)):
        extent = -(-n // 64) * 64
        U = -(-extent // unit)
        want = []
        for m in range(M):
            lo, hi = (m * U // M) * unit, min(((m + 1) * U // M) * unit, extent)
            want.append((lo, hi - lo) if hi > lo else None)
        got = oracle.shard_ranges([n], 1 << 62, unit, -1, M)
        for g, w in zip(got, want):
            if w is None:
                assert g[1] == 0
            else:
                assert g == w


@pytest.mark.parametrize("seed", range(4))
def test_ranges_follow_the_definition_on_random_lists(oracle, seed):
    rnd = random.Random(300 + seed)
    sizes = [0, 1, 7, 8, 9, 63, 64, 65, 500, 2047, 2048, 2049, 4096, 5000, 10000, 40000]
    for _ in range(60):
        numel = [rnd.choice(sizes) for _ in range(rnd.randint(1, 12))]
        if sum(numel) == 0:
            numel[0] = 3
        cap = rnd.choice([64, 4096, 40000, 1 << 20, 1 << 40])
        unit = rnd.choice([2048, 4096, 64])
        M = rnd.randint(1, 9)
        plan = oracle.bucket_plan(numel, cap)
        for bucket in [-1] + list(range(plan.n_buckets)):
            units, _ = units_by_brute_force(oracle, numel, cap, unit, bucket)
            got = oracle.shard_ranges(numel, cap, unit, bucket, M)
            U = len(units)
            lo_range = 0 if bucket < 0 else int(plan.bucket_start[bucket])
            n_range = plan.transport_numel if bucket < 0 else int(plan.bucket_numel[bucket])
            # the units tile the range
            assert sum(n for _, n in units) == n_range
            owner = np.full(plan.transport_numel, -1)
            for m, (lo, n) in enumerate(got):
                mine = units[m * U // M:(m + 1) * U // M]
                if not mine:
                    assert n == 0
                    continue
                assert (lo, n) == (mine[0][0], sum(x for _, x in mine))      # whole units, contiguous
                assert (owner[lo:lo + n] == -1).all()                       # no element has two owners
                owner[lo:lo + n] = m
            inside = owner[lo_range:lo_range + n_range]
            assert (inside >= 0).all() and (np.diff(inside) >= 0).all()     # every element owned, in member order
            assert (owner[:lo_range] == -1).all() and (owner[lo_range + n_range:] == -1).all()
            counts = [len(units[m * U // M:(m + 1) * U // M]) for m in range(M)]
            assert max(counts) - min(counts) <= 1                           # balanced to one unit


def test_bad_arguments(oracle):
    for args in (([5], 1 << 20, 0, -1, 2), ([5], 1 << 20, 2048, 1, 2), ([5], 1 << 20, 2048, -2, 2), ([5], 1 << 20, 2048, -1, 0)):
        with pytest.raises(oracle.OracleError):
            oracle.shard_ranges(*args)


def problem(rnd, dtype):
    K = rnd.randint(2, 9)
    G = rnd.randint(1, min(K, 3))
    group_of = list(range(G)) + [rnd.randrange(G) for _ in range(K - G)]
    rnd.shuffle(group_of)
    shares = [rnd.randint(1, 90) for _ in range(K)]
    numel = [rnd.choice([1, 5, 64, 100, 2047, 2048, 2050, 4097, 9000]) for _ in range(rnd.randint(1, 8))]
    wl = W.Workload("sharded", 60 + rnd.randint(0, 30), [(n,) for n in numel], dtype, group_of, shares,
                    bucket_cap_bytes=rnd.choice([4096, 40000, 1 << 30]))
    grads = [[W.as_numpy(t) for t in W.split_tensors(W.rank_gradients(wl, r, "cpu"), wl.numel)] for r in range(K)]
    return wl, grads


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_sharding_changes_who_computes_an_element_not_its_value(oracle, dtype):
    rnd = random.Random(77 if dtype == "f32" else 78)
    dt = F32 if dtype == "f32" else BF16
    for i in range(12):
        wl, grads = problem(rnd, dtype)
        unit = 2048 if dtype == "f32" else 4096
        scale = rnd.choice([1.0, 1.0 / 3.0])
        odt = rnd.choice([F32, BF16])
        want, parts, _, plan = oracle.sync_step(grads, wl.numel, dt, wl.group_of, wl.shares, wl.G,
                                                wl.bucket_cap_bytes, scale, odt)
        got, host, _ = oracle.sharded_sync_step(grads, wl.numel, dt, wl.group_of, wl.shares, wl.G,
                                                wl.bucket_cap_bytes, unit, scale, odt, per_bucket=bool(i % 2))
        for g in range(wl.G):
            assert np.array_equal(host[g].view(np.uint32), parts[g].view(np.uint32))
        for r in range(wl.K):
            for t in range(wl.T):
                assert np.array_equal(got[r][t], want[t]) or (np.isnan(want[t]).any())
                assert got[r][t].tobytes() == want[t].tobytes()
