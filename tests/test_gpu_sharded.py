"""One rank per device, on the hardware at hand (one GPU).

Two layers.  (1) The ranks of a job emulated in ONE process: one context per rank, each bound
to its rank with kt_shard_bind, all reading the same device's memory through ordinary
pointers.  This runs the kernels' share arithmetic -- shares that start and end in the middle
of tensors, empty shares, ragged lists, misaligned tensors, both dtypes -- on many random
problems.  (2) The ranks as separate PROCESSES on the one GPU: gradients and outputs of the
group mates are reached through addresses mapped with kt_ipc_open (the peer-mapped path a
multi-GPU node takes), partials cross a host-memory block that all processes map, ranks
meet at host-side barriers (gloo); no kernel waits for another process.  Every result is
compared with the oracle bit for bit.
"""
import os
import random
import sys

import numpy as np
import pytest
import torch

from paper_2505_10183_b200 import workloads as W

import _harness as H
import test_gpu_random as TR

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def kt():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    from paper_2505_10183_b200 import binding
    torch.cuda.set_device(0)
    return binding


def run_emulated(kt, oracle, wl, host, dev, out_dtype, scale, per_bucket, relay, in_place=False, narrow=False):
    """All ranks of the job as contexts of one process.  Every rank reduces its share of every
    range; the shares of a group land in one buffer per group, which stands for the host
    memory all ranks can reach (with relay=True they really cross pinned host memory)."""
    K, G, T = wl.K, wl.G, wl.T
    dt = H.ORACLE_DT[wl.dtype]
    odt = {torch.float32: 0, torch.bfloat16: 1}[out_dtype]
    unit = kt.kt_work_unit(dt)
    members = [[r for r in range(K) if wl.group_of[r] == g] for g in range(G)]
    outs = dev if in_place else [[torch.full((m,), float("nan"), dtype=out_dtype, device="cuda") for m in wl.numel]
                                 for _ in range(K)]
    ctxs = []
    for r in range(K):
        ctx = kt.kt_groups_init(wl.group_of, wl.shares, G)
        kt.kt_shard_bind(ctx, r, wl.group_of)
        if narrow:                                       # the library's bf16 transport (an extension)
            kt.kt_set_transport_dtype(ctx, kt.KT_BF16)
        kt.kt_bucket_pack(ctx, [dev[q] for q in members[wl.group_of[r]]], wl.bucket_cap_bytes)
        ctxs.append(ctx)
    plan = kt.kt_plan_query(ctxs[0])
    n = plan.transport_numel
    poison = float(np.float32(-7.25e33))
    tdt = torch.bfloat16 if narrow else torch.float32
    own = [torch.full((G, n), poison, dtype=tdt, device="cuda") for _ in range(K)]   # every rank's device rows
    poison = float(own[0][0, 0]) if n else poison                                 # the value as the buffer holds it
    shared = list(torch.full((G, n), poison, dtype=tdt).pin_memory()) if relay else None   # the host block all ranks reach
    buckets = list(range(plan.n_buckets)) if per_bucket else [-1]
    side = torch.cuda.Stream()
    # the ranges the library hands out are the oracle's
    for b in buckets:
        for g in range(G):
            want = oracle.shard_ranges(wl.numel, wl.bucket_cap_bytes, unit, b, len(members[g]))
            for m, r in enumerate(members[g]):
                lo, cnt, M = kt.kt_shard_query(ctxs[r], b)
                assert (lo, cnt) == want[m] and M == len(members[g])
                assert kt.kt_shard_query(ctxs[members[g][0]], b, member=m)[:2] == want[m]
    want_out, want_parts, _, _ = oracle.sync_step(host, wl.numel, dt, wl.group_of, wl.shares, G,
                                                  wl.bucket_cap_bytes, scale, odt, 1 if narrow else 0)
    bits = torch.int16 if narrow else torch.int32
    if G == 1:
        for b in buckets:
            for r in range(K):
                kt.kt_sync_direct(ctxs[r], [outs[q] for q in members[0]], scale=scale, bucket=b)
    else:
        for b in buckets:
            for r in range(K):
                g = wl.group_of[r]
                kt.kt_hier_reduce(ctxs[r], kt.KT_INTRA, list(own[r]), bucket=b)
                if relay:
                    kt.kt_stage_to_host(ctxs[r], kt.KT_D2H, list(own[r]), shared, bucket=b, side_stream=side)
        torch.cuda.synchronize()                       # stands for the barrier between the two halves
        for r in range(K):                             # a rank wrote its own share of its own group's row, nothing else
            g = wl.group_of[r]
            mask = torch.zeros(n, dtype=torch.bool, device="cuda")
            for b in buckets:
                lo, cnt, _ = kt.kt_shard_query(ctxs[r], b)
                mask[lo:lo + cnt] = True
            part = torch.from_numpy(want_parts[g].view(np.int16) if narrow else want_parts[g]).cuda()
            assert torch.equal(own[r][g][mask].view(bits), part[mask].view(bits))
            assert bool((own[r][g][~mask] == poison).all())
            for h in range(G):
                if h != g:
                    assert bool((own[r][h] == poison).all())
        if relay:
            for g in range(G):
                H.assert_bit_equal(shared[g], want_parts[g], "host partial %d" % g)
        for b in buckets:
            for r in range(K):
                g = wl.group_of[r]
                if relay:
                    kt.kt_stage_to_host(ctxs[r], kt.KT_H2D, list(own[r]), shared, bucket=b, side_stream=side)
                    kt.kt_stage_wait(ctxs[r], kt.KT_H2D, bucket=b)
                else:                                  # without the relay: read the other groups' rows where their owners wrote them
                    lo, cnt, _ = kt.kt_shard_query(ctxs[r], b)
                    for h in range(G):
                        if h != g:
                            for q in members[h]:
                                qlo, qcnt, _ = kt.kt_shard_query(ctxs[q], b)
                                a, z = max(lo, qlo), min(lo + cnt, qlo + qcnt)
                                if z > a:
                                    own[r][h][a:z].copy_(own[q][h][a:z])
                kt.kt_unpack_scale(ctxs[r], list(own[r]), [outs[q] for q in members[g]], scale=scale, bucket=b)
    torch.cuda.synchronize()
    for r in range(K):
        for t in range(T):
            H.assert_bit_equal(outs[r][t], want_out[t], "rank %d out[%d]" % (r, t))
    for ctx in ctxs:
        kt.kt_destroy(ctx)


@pytest.mark.parametrize("name", ["tiny", "mobilenet_v2", "resnet18", "resnet50"])
def test_emulated_ranks_named_configurations(kt, oracle, name):
    wl = W.by_name(name)
    wl.shares = H.shares_of(wl, kt)
    odt = H.TORCH_DT[wl.dtype]
    for per_bucket, relay, in_place in ((True, True, False), (False, False, True)):
        host, dev = H.device_gradients(wl)
        run_emulated(kt, oracle, wl, host, dev, odt, 1.0, per_bucket, relay, in_place)


@pytest.mark.parametrize("seed", range(6))
def test_emulated_ranks_random_problems(kt, oracle, seed):
    rnd = random.Random(8800 + seed)
    for _ in range(12):
        wl = TR.random_problem(rnd)
        if rnd.random() < 0.5:                          # longer tensors: shares that begin and end mid-tensor
            wl = W.Workload("random_long", wl.config_id, [(rnd.choice([5000, 20000, 70001, 300000]),) for _ in range(rnd.randint(1, 4))],
                            wl.dtype, wl.group_of, wl.shares, bucket_cap_bytes=rnd.choice([40000, 1 << 20, 1 << 40]))
        host, dev = H.device_gradients(wl, misalign=rnd.choice([0, 0, 1, 3]))
        out_dtype = rnd.choice([torch.float32, torch.bfloat16])
        in_place = out_dtype == H.TORCH_DT[wl.dtype] and rnd.random() < 0.4
        run_emulated(kt, oracle, wl, host, dev, out_dtype, rnd.choice([1.0, 1.0 / 3.0]), rnd.random() < 0.5,
                     rnd.random() < 0.5, in_place)


@pytest.mark.parametrize("name", ["tiny", "mobilenet_v2", "resnet50"])
def test_emulated_ranks_with_the_bf16_transport(kt, oracle, name):
    """The narrow transport (an extension of this library) on shares: the partial a member stores
    is rounded once, where the oracle rounds it."""
    wl = W.by_name(name)
    wl.shares = H.shares_of(wl, kt)
    host, dev = H.device_gradients(wl)
    run_emulated(kt, oracle, wl, host, dev, H.TORCH_DT[wl.dtype], 0.5, True, True, False, narrow=True)
    run_emulated(kt, oracle, wl, host, dev, torch.float32, 1.0, False, False, False, narrow=True)


def run_emulated_broadcast(kt, oracle, wl, root, per_bucket, misalign=0):
    """Model synchronisation with every rank a context of its own: the root sends (whole range)
    and copies down; every rank of another group copies ITS SHARE up into a receive buffer of
    its own and unpacks it into all members of its group; nobody else does anything."""
    K, G = wl.K, wl.G
    dt = H.ORACLE_DT[wl.dtype]
    tdt = H.TORCH_DT[wl.dtype]
    host, dev = H.device_gradients(wl, misalign=misalign)
    members = [[r for r in range(K) if wl.group_of[r] == g] for g in range(G)]
    ctxs = []
    for r in range(K):
        ctx = kt.kt_groups_init(wl.group_of, [1] * K, G)
        kt.kt_shard_bind(ctx, r, wl.group_of)
        kt.kt_bucket_pack(ctx, [dev[q] for q in members[wl.group_of[r]]], wl.bucket_cap_bytes)
        ctxs.append(ctx)
    plan = kt.kt_plan_query(ctxs[0])
    n = plan.transport_numel
    buckets = list(range(plan.n_buckets)) if per_bucket else [-1]
    want, flat, _ = oracle.broadcast(host, root, wl.numel, dt, wl.bucket_cap_bytes)
    send = torch.full((n,), 7.0, dtype=tdt, device="cuda")
    shared = torch.full((n,), 7.0, dtype=tdt).pin_memory()
    recvs = {r: torch.full((n,), 7.0, dtype=tdt, device="cuda") for r in range(K)}
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    g_root = wl.group_of[root]
    for b in buckets:                                   # the root's half
        for r in range(K):                              # everybody may call; only the root acts
            kt.kt_bcast_send(ctxs[r], root, send, bucket=b)
        kt.kt_bcast_relay(ctxs[root], root, send, shared, [None] * G, s1, s2, bucket=b)
        kt.kt_stage_wait(ctxs[root], kt.KT_D2H, bucket=b, timeout_ms=20000)
    torch.cuda.synchronize()                            # stands for the barrier
    H.assert_bit_equal(shared, flat, "what crossed the host")
    for b in buckets:                                   # the other groups' half
        for r in range(K):
            if r == root:
                continue
            rows = [recvs[r] if g == wl.group_of[r] else None for g in range(G)]
            kt.kt_bcast_relay(ctxs[r], root, None, shared, rows, s1, s2, bucket=b)
            if wl.group_of[r] != g_root:
                kt.kt_stage_wait(ctxs[r], kt.KT_H2D, bucket=b)
            kt.kt_bcast_recv(ctxs[r], root, rows, bucket=b)
    torch.cuda.synchronize()
    for r in range(K):
        for t in range(wl.T):
            H.assert_bit_equal(dev[r][t], want[r][t], "rank %d tensor %d" % (r, t))
    # a rank outside the root's group copied up its own share and nothing else
    for r in range(K):
        if wl.group_of[r] == g_root:
            assert bool((recvs[r] == 7.0).all())
            continue
        mask = torch.zeros(n, dtype=torch.bool, device="cuda")
        for b in buckets:
            lo, cnt, _ = kt.kt_shard_query(ctxs[r], b)
            mask[lo:lo + cnt] = True
        assert bool((recvs[r][~mask] == 7.0).all())
        m = mask.cpu().numpy()
        assert np.array_equal(H.bits(W.as_numpy(recvs[r]))[m], H.bits(flat)[m])
    for ctx in ctxs:
        kt.kt_destroy(ctx)


@pytest.mark.parametrize("name", ["tiny", "mobilenet_v2", "resnet18"])
def test_emulated_ranks_broadcast_named_configurations(kt, oracle, name):
    for dtype, root, per_bucket in (("f32", 0, False), ("bf16", None, True)):
        wl = W.by_name(name)
        wl.dtype = dtype
        run_emulated_broadcast(kt, oracle, wl, wl.K - 1 if root is None else root, per_bucket)


@pytest.mark.parametrize("seed", range(3))
def test_emulated_ranks_broadcast_random_problems(kt, oracle, seed):
    rnd = random.Random(9900 + seed)
    for _ in range(12):
        wl = TR.random_problem(rnd)
        if rnd.random() < 0.4:
            wl = W.Workload("random_long", wl.config_id, [(rnd.choice([5000, 20000, 70001]),) for _ in range(rnd.randint(1, 3))],
                            wl.dtype, wl.group_of, wl.shares, bucket_cap_bytes=rnd.choice([40000, 1 << 20, 1 << 40]))
        run_emulated_broadcast(kt, oracle, wl, rnd.randrange(wl.K), rnd.random() < 0.5, misalign=rnd.choice([0, 0, 1, 3]))


def test_calls_that_need_all_ranks_are_refused_on_a_bound_context(kt):
    wl = W.tiny()
    _, dev = H.device_gradients(wl)
    ctx = kt.kt_groups_init(wl.group_of, wl.shares, wl.G)
    with pytest.raises(kt.KtError) as e:
        kt.kt_shard_bind(ctx, 4, wl.group_of)
    assert e.value.status == kt.KT_ERR_INVALID
    kt.kt_shard_bind(ctx, 2, wl.group_of)
    with pytest.raises(kt.KtError) as e:                 # a bound context takes its group's lists only
        kt.kt_bucket_pack(ctx, dev, wl.bucket_cap_bytes)
    assert e.value.status == kt.KT_ERR_SHAPE
    kt.kt_bucket_pack(ctx, dev[2:], wl.bucket_cap_bytes)
    n = kt.kt_plan_query(ctx).transport_numel
    rows = list(torch.zeros(wl.G, n, device="cuda"))
    pinned = list(torch.zeros(wl.G, n).pin_memory())
    out = [[torch.empty_like(t) for t in dev[0]]]
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    for call in (lambda: kt.kt_relay_through_host(ctx, rows, pinned, rows, s1, s2),
                 lambda: kt.kt_sync_direct(ctx, out),
                 lambda: kt.kt_allreduce(ctx, out, rows, pinned, rows, s1, s2)):
        with pytest.raises(kt.KtError) as e:
            call()
        assert e.value.status == kt.KT_ERR_STATE
    kt.kt_hier_reduce(ctx, kt.KT_INTRA, rows)           # what it is for still works
    torch.cuda.synchronize()
    kt.kt_destroy(ctx)


# ------------------------------------------------------------------ ranks as processes
CASES = [
    # name, shapes / workload, dtype, group_of, shares, cap, out dtype, per_bucket, in_place
    dict(name="tiny", wl="tiny", per_bucket=False, in_place=False),
    dict(name="ragged_3_plus_2", wl="mobilenet_v2", group_of=[0, 0, 1, 0, 1], shares=[40, 29, 19, 40, 29], per_bucket=True,
         in_place=True),
    dict(name="resnet18", wl="resnet18", per_bucket=True, in_place=False),
    dict(name="one_group_bf16", wl="tiny", dtype="bf16", group_of=[0, 0, 0, 0], shares=[5, 7, 11, 13], per_bucket=False,
         in_place=True),
    dict(name="bf16_to_f32", wl="tiny", dtype="bf16", out_dtype="f32", group_of=[0, 1, 1, 1], shares=[64, 64, 32, 32],
         per_bucket=True, in_place=False),
    dict(name="narrow_transport", wl="mobilenet_v2", group_of=[0, 1, 0, 1], shares=[79, 49, 79, 49], per_bucket=True,
         in_place=False, narrow=True),
]


def case_workload(case, world):
    if "numel" in case:          # a drawn problem: flat tensors of the listed sizes
        wl = W.Workload(case["name"], case["config_id"], [(m,) for m in case["numel"]], case["dtype"],
                        list(case["group_of"]), list(case["shares"]), bucket_cap_bytes=case["cap"])
        return wl if wl.K == world else None
    wl = W.by_name(case["wl"])
    if "dtype" in case:
        wl.dtype = case["dtype"]
    if "group_of" in case:
        wl.group_of, wl.shares, wl.step_times = list(case["group_of"]), list(case["shares"]), None
    if wl.shares is None:
        from oracle import kt_oracle
        wl.shares = kt_oracle.schedule(wl.step_times, wl.global_batch).tolist()
    return wl if wl.K == world else None


def rank_main(rank, world, port, cases):
    """One rank of the job: its own process, its own CUDA context on device 0."""
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import torch.distributed as dist
    from oracle import kt_oracle as oracle
    from paper_2505_10183_b200 import binding as kt
    from paper_2505_10183_b200.sharded import ShardedSync
    torch.cuda.set_device(0)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    for case in cases:
        wl = case_workload(case, world)
        if wl is None:
            continue
        dt = H.ORACLE_DT[wl.dtype]
        odt_name = case.get("out_dtype", wl.dtype)
        host = [[W.as_numpy(t) for t in W.split_tensors(W.rank_gradients(wl, r, "cpu"), wl.numel)] for r in range(wl.K)]
        mine = [t.cuda() for t in W.split_tensors(W.rank_gradients(wl, rank, "cpu"), wl.numel)]
        outs = None if case["in_place"] else [torch.full((m,), float("nan"), dtype=H.TORCH_DT[odt_name], device="cuda")
                                              for m in wl.numel]
        narrow = case.get("narrow", False)
        job = ShardedSync(rank, wl.group_of, wl.shares, mine, outs, wl.bucket_cap_bytes, host_group=None,
                          per_bucket=case["per_bucket"], narrow_transport=narrow)
        assert job.my_range(-1 if not case["per_bucket"] else 0) == oracle.shard_ranges(
            wl.numel, wl.bucket_cap_bytes, kt.kt_work_unit(dt), -1 if not case["per_bucket"] else 0,
            len(job.members))[job.member]
        scales = [1.0] if case["in_place"] else [1.0, 0.5]      # in place the inputs are gone after one step
        shares = list(wl.shares)
        for scale in scales:
            job.step(scale=scale)
            # with one group no partial is ever stored: the narrow transport has nothing to round
            want, _, _, _ = oracle.sync_step(host, wl.numel, dt, wl.group_of, shares, wl.G, wl.bucket_cap_bytes,
                                             scale, H.ORACLE_DT[odt_name], 1 if narrow and wl.G > 1 else 0)
            # the scheduler moves samples from the first rank to the last between steps: new weights
            shares = [shares[0] - 1] + shares[1:-1] + [shares[-1] + 1] if shares[0] > 1 and wl.K > 1 else shares
            job.set_shares(shares)
            result = mine if case["in_place"] else outs
            for t in range(wl.T):
                H.assert_bit_equal(result[t], want[t], "%s rank %d out[%d] scale %g" % (case["name"], rank, t, scale))
        job.close()
    dist.barrier()
    dist.destroy_process_group()


def random_cases(rnd, world, count):
    """Drawn problems for `world` ranks: ragged tensor lists, group layouts, shares, dtypes,
    bucket caps, output dtypes, in place or not, bucket by bucket or not, either transport."""
    cases = []
    while len(cases) < count:
        wl = TR.random_problem(rnd)
        if wl.K != world:
            continue
        numel = list(wl.numel)
        if rnd.random() < 0.3:
            numel = [rnd.choice([5000, 20000, 70001]) for _ in range(rnd.randint(1, 3))]
        in_place = rnd.random() < 0.4
        case = dict(name="drawn_%d" % len(cases), numel=numel, config_id=wl.config_id, dtype=wl.dtype, group_of=wl.group_of,
                    shares=wl.shares, cap=wl.bucket_cap_bytes, per_bucket=rnd.random() < 0.5, in_place=in_place,
                    narrow=rnd.random() < 0.25)
        if not in_place:
            case["out_dtype"] = rnd.choice(["f32", "bf16"])
        cases.append(case)
    return cases


@pytest.mark.parametrize("world", [3])
def test_ranks_as_processes_on_drawn_problems(world):
    import random
    import torch.multiprocessing as mp
    if not torch.cuda.is_available():
        pytest.fail("this test needs a CUDA device")
    cases = random_cases(random.Random(5150), world, 14)
    port = 29600 + (os.getpid() * 13 + world) % 2000
    mp.spawn(rank_main, args=(world, port, cases), nprocs=world, join=True)


@pytest.mark.parametrize("world", [4, 5])
def test_ranks_as_processes_over_mapped_memory(world):
    """`world` processes share the one GPU; each is a rank with its own context.  A failing
    comparison in any rank fails the test."""
    import torch.multiprocessing as mp
    if not torch.cuda.is_available():
        pytest.fail("this test needs a CUDA device")
    cases = [c for c in CASES if case_workload(c, world) is not None]
    assert cases
    port = 29600 + (os.getpid() * 7 + world) % 2000
    mp.spawn(rank_main, args=(world, port, cases), nprocs=world, join=True)


def leaving_rank_main(rank, world, port):
    """Ranks 0..2 keep stepping; rank 3 stops after the first step, between steps, with none of
    its kernels or copies in flight, and simply stays away from the next one."""
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import time
    import torch.distributed as dist
    from oracle import kt_oracle as oracle
    from paper_2505_10183_b200 import binding as kt
    from paper_2505_10183_b200.sharded import ShardedSync
    torch.cuda.set_device(0)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = W.tiny()
    host = [[W.as_numpy(t) for t in W.split_tensors(W.rank_gradients(wl, r, "cpu"), wl.numel)] for r in range(wl.K)]
    mine = [t.cuda() for t in W.split_tensors(W.rank_gradients(wl, rank, "cpu"), wl.numel)]
    outs = [torch.full((m,), float("nan"), device="cuda") for m in wl.numel]
    job = ShardedSync(rank, wl.group_of, wl.shares, mine, outs, wl.bucket_cap_bytes)
    job.step()                                              # everybody takes part in the first step
    job.wait_ms = 400                                       # from now on a rank is missed after 0.4 s
    want, _, _, _ = oracle.sync_step(host, wl.numel, 0, wl.group_of, wl.shares, wl.G, wl.bucket_cap_bytes)
    for t in range(wl.T):
        H.assert_bit_equal(outs[t], want[t], "rank %d out[%d]" % (rank, t))
    if rank != world - 1:
        t0 = time.time()
        try:
            job.step()
            raise AssertionError("rank %d: the step went through without rank %d" % (rank, world - 1))
        except kt.KtError as e:                             # the wait ended on the host, with a status
            assert e.status == kt.KT_ERR_TIMEOUT and time.time() - t0 < 10.0
        # the device is untouched by the failed step and still works
        probe = torch.empty(wl.numel[0], device="cuda")
        kt.kt_cast(mine[0].to(torch.bfloat16), probe)
        torch.cuda.synchronize()
        assert bool(torch.isfinite(probe).all())
    dist.barrier()                                          # the survivors and the leaver agree to stop
    job.close(meet=False)
    dist.barrier()
    dist.destroy_process_group()


def test_a_rank_that_stays_away_between_steps_is_noticed_on_the_host():
    """Failure handling of the one-rank-per-device path: nothing on any GPU waits for the missing
    rank, so the others get KT_ERR_TIMEOUT from the host barrier and keep a usable device."""
    import torch.multiprocessing as mp
    if not torch.cuda.is_available():
        pytest.fail("this test needs a CUDA device")
    mp.spawn(leaving_rank_main, args=(4, 29600 + (os.getpid() * 11) % 2000), nprocs=4, join=True)


BCAST_CASES = [
    dict(wl="tiny", root=0, per_bucket=False),
    dict(wl="tiny", root=3, per_bucket=True, dtype="bf16"),
    dict(wl="mobilenet_v2", root=2, group_of=[0, 0, 1, 0, 1], per_bucket=True),
    dict(wl="resnet18", root=1, per_bucket=True),
    dict(wl="tiny", root=2, group_of=[0, 0, 0, 0], per_bucket=False),          # one group: no host relay at all
]


def bcast_rank_main(rank, world, port, cases):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import torch.distributed as dist
    from oracle import kt_oracle as oracle
    from paper_2505_10183_b200.sharded import ShardedSync
    torch.cuda.set_device(0)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    for case in cases:
        if "numel" in case:
            wl = case_workload(case, world)
            if wl is None:
                continue
            case = dict(case, wl=case["name"])
        else:
            wl = W.by_name(case["wl"])
            wl.dtype = case.get("dtype", wl.dtype)
            if "group_of" in case:
                wl.group_of = list(case["group_of"])
            if wl.K != world:
                continue
        dt = H.ORACLE_DT[wl.dtype]
        host = [[W.as_numpy(t) for t in W.split_tensors(W.rank_gradients(wl, r, "cpu"), wl.numel)] for r in range(wl.K)]
        params = [t.cuda() for t in W.split_tensors(W.rank_gradients(wl, rank, "cpu"), wl.numel)]     # every rank starts with its own values
        job = ShardedSync(rank, wl.group_of, [1] * wl.K, params, None, wl.bucket_cap_bytes, per_bucket=case["per_bucket"])
        job.broadcast(case["root"])
        want, _, _ = oracle.broadcast(host, case["root"], wl.numel, dt, wl.bucket_cap_bytes)
        for t in range(wl.T):
            H.assert_bit_equal(params[t], want[rank][t], "%s root %d: rank %d tensor %d" % (case["wl"], case["root"], rank, t))
        job.broadcast(case["root"])                              # again: nothing may change
        for t in range(wl.T):
            H.assert_bit_equal(params[t], want[rank][t], "second broadcast: rank %d tensor %d" % (rank, t))
        job.close()
    dist.barrier()
    dist.destroy_process_group()


def test_broadcast_with_ranks_as_processes_on_drawn_problems():
    import torch.multiprocessing as mp
    if not torch.cuda.is_available():
        pytest.fail("this test needs a CUDA device")
    rnd = random.Random(6160)
    cases = [dict(c, root=rnd.randrange(3)) for c in random_cases(rnd, 3, 14)]
    mp.spawn(bcast_rank_main, args=(3, 29600 + (os.getpid() * 17 + 3) % 2000, cases), nprocs=3, join=True)


@pytest.mark.parametrize("world", [4, 5])
def test_broadcast_with_ranks_as_processes(world):
    """Model synchronisation over IPC-mapped tensors and the shared host block: every rank starts
    with its own values and must end with the root's, bit for bit."""
    import torch.multiprocessing as mp
    if not torch.cuda.is_available():
        pytest.fail("this test needs a CUDA device")
    cases = [c for c in BCAST_CASES if len(c.get("group_of", W.by_name(c["wl"]).group_of)) == world]
    assert cases
    mp.spawn(bcast_rank_main, args=(world, 29600 + (os.getpid() * 13 + world) % 2000, cases), nprocs=world, join=True)
