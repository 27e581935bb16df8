"""GPU parity of the hierarchical broadcast (kt_bcast_send / kt_bcast_relay / kt_bcast_recv)
against the CPU oracle: after the broadcast every rank's tensors, the flat send buffer, the
pinned host copy and every receive buffer hold the root's bytes, bit for bit."""
import random

import numpy as np
import pytest
import torch

from paper_2505_10183_b200 import workloads as W

import _harness as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def kt():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    from paper_2505_10183_b200 import binding
    torch.cuda.set_device(0)
    return binding


def bit_view(t: torch.Tensor) -> torch.Tensor:
    return t.view(torch.int32) if t.dtype == torch.float32 else t.view(torch.int16)


def run_broadcast(kt, oracle, wl, root, relay=True, per_bucket=False, chunk=1 << 20, shifts=None, special=False):
    tdt = H.TORCH_DT[wl.dtype]
    guard = 32
    host, bufs, dev = [], [], []
    for r in range(wl.K):
        ts = W.split_tensors(W.rank_gradients(wl, r, "cpu"), wl.numel)
        if special and r == root:      # patterns a careless copy would change
            for t in ts:
                if t.numel() >= 4:
                    bit_view(t)[:4] = torch.tensor([0x7FC1, 0x7F81, -0x8000, 0x0001] if wl.dtype == "bf16" else
                                                   [0x7FC00001, 0x7F800001, -0x80000000, 0x00000001],
                                                   dtype=bit_view(t).dtype)
        host.append([W.as_numpy(t) for t in ts])
        row = []
        for i, t in enumerate(ts):
            m = 0 if shifts is None else shifts(r, i)
            b = torch.full((t.numel() + 2 * guard + m,), -777.0, dtype=tdt, device="cuda")
            v = b[guard + m:guard + m + t.numel()]
            bit_view(v).copy_(bit_view(t))
            bufs.append((b, v))
            row.append(v)
        dev.append(row)
    ctx = kt.kt_groups_init(wl.group_of, [1] * wl.K, wl.G)
    kt.kt_bucket_pack(ctx, dev, wl.bucket_cap_bytes)
    plan = kt.kt_plan_query(ctx)
    n = plan.transport_numel
    send = torch.full((n,), float("nan"), dtype=tdt, device="cuda")
    g_root = wl.group_of[root]
    if relay:
        pinned = torch.full((n,), float("nan"), dtype=tdt).pin_memory()
        recv = [None if g == g_root else torch.full((n,), float("nan"), dtype=tdt, device="cuda") for g in range(wl.G)]
        s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    else:
        recv = [None if g == g_root else send for g in range(wl.G)]
    before = kt.kt_launch_count(ctx)
    for b in (range(plan.n_buckets) if per_bucket else [-1]):
        kt.kt_bcast_send(ctx, root, send, bucket=b)
        if relay:
            kt.kt_bcast_relay(ctx, root, send, pinned, recv, s1, s2, bucket=b, chunk_bytes=chunk)
            kt.kt_stage_wait(ctx, kt.KT_H2D, bucket=b)
        kt.kt_bcast_recv(ctx, root, recv, bucket=b)
    torch.cuda.synchronize()
    launches = kt.kt_launch_count(ctx) - before

    want, flat, o_plan = oracle.broadcast(host, root, wl.numel, H.ORACLE_DT[wl.dtype], wl.bucket_cap_bytes)
    assert plan.tensor_offset == o_plan.tensor_offset.tolist() and n == o_plan.transport_numel
    H.assert_bit_equal(send, flat, "send buffer")
    if relay:
        H.assert_bit_equal(pinned, flat, "pinned host copy")
        for g in range(wl.G):
            if g != g_root:
                H.assert_bit_equal(recv[g], flat, "recv[%d]" % g)
    for r in range(wl.K):
        for t in range(wl.T):
            H.assert_bit_equal(dev[r][t], want[r][t], "rank %d tensor %d" % (r, t))
    for b, v in bufs:
        lo = (v.data_ptr() - b.data_ptr()) // b.element_size()
        assert bool((b[:lo] == -777.0).all()) and bool((b[lo + v.numel():] == -777.0).all())
    kt.kt_destroy(ctx)
    return launches


@pytest.mark.parametrize("name", ["tiny", "resnet18", "resnet50", "mobilenet_v2"])
def test_named_configurations(kt, oracle, name):
    wl = W.by_name(name)
    launches = run_broadcast(kt, oracle, wl, root=0, special=True)
    assert launches == 2
    run_broadcast(kt, oracle, wl, root=wl.K - 1, per_bucket=True, chunk=(1 << 20) + 256)
    run_broadcast(kt, oracle, wl, root=1, relay=False)


def test_single_group_single_rank_and_singletons(kt, oracle):
    base = W.tiny()
    for group_of, root in (([0, 0, 0], 1), ([0], 0), ([0, 1, 2, 3], 2), ([1, 0, 1, 0, 2], 4)):
        wl = W.Workload("bcast_groups", 8, base.shapes, "f32", group_of, [1] * len(group_of))
        run_broadcast(kt, oracle, wl, root)


@pytest.mark.parametrize("seed", range(3))
def test_random_problems_with_misaligned_tensors(kt, oracle, seed):
    import test_gpu_random as TR
    rnd = random.Random(9000 + seed)
    for _ in range(25):
        wl = TR.random_problem(rnd)
        shifts = {}
        run_broadcast(kt, oracle, wl, root=rnd.randrange(wl.K), relay=rnd.random() < 0.6,
                      per_bucket=rnd.random() < 0.5, chunk=rnd.choice([256, 4096, 1 << 20]),
                      shifts=lambda r, t: shifts.setdefault((r, t), rnd.choice([0, 0, 0, 1, 2, 3, 5])),
                      special=True)


def test_error_codes(kt):
    wl = W.tiny()
    _, dev = H.device_gradients(wl)
    ctx = kt.kt_groups_init(wl.group_of, wl.shares, wl.G)
    send = torch.zeros(16384, device="cuda")
    with pytest.raises(kt.KtError) as e:
        kt.kt_bcast_send(ctx, 0, send)
    assert e.value.status == kt.KT_ERR_STATE
    kt.kt_bucket_pack(ctx, dev, wl.bucket_cap_bytes)
    for bad_root in (-1, wl.K):
        with pytest.raises(kt.KtError) as e:
            kt.kt_bcast_send(ctx, bad_root, send)
        assert e.value.status == kt.KT_ERR_INVALID
    with pytest.raises(kt.KtError) as e:
        kt.kt_bcast_send(ctx, 0, send[1:])
    assert e.value.status == kt.KT_ERR_ALIGN
    with pytest.raises(kt.KtError) as e:
        kt.kt_bcast_recv(ctx, 0, [None, None])
    assert e.value.status == kt.KT_ERR_INVALID
    with pytest.raises(kt.KtError) as e:
        kt.kt_bcast_send(ctx, 0, send, bucket=3)
    assert e.value.status == kt.KT_ERR_SHAPE
    kt.kt_destroy(ctx)
