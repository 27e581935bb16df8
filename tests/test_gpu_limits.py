"""The limits of the library on the GPU against the oracle: the maximum rank and group counts
(64 ranks in 16 groups), a tensor list far longer than a CTA has threads (the tile look-up
then strides over the list), single-element tensors, and one rank more / one group more than
allowed being rejected on the host."""
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


def all_routes(kt, oracle, wl):
    host, dev = H.device_gradients(wl)
    out, transport, plan, ctx = H.run_gpu_path(kt, wl, dev, wl.shares)
    want, parts, _, _ = H.run_oracle_path(oracle, wl, host, wl.shares)
    for g in range(wl.G):
        H.assert_bit_equal(transport[g], parts[g], "transport[%d]" % g)
    for t in range(wl.T):
        H.assert_bit_equal(out[0][t], want[t], "out[%d]" % t)
    # the one-pass route on the same context
    direct = [[torch.full_like(o, float("nan")) for o in out[0]]]
    kt.kt_sync_direct(ctx, direct)
    torch.cuda.synchronize()
    for t in range(wl.T):
        H.assert_bit_equal(direct[0][t], want[t], "direct out[%d]" % t)
    # broadcast from the last rank over the same registered tensors
    root = wl.K - 1
    n = plan.transport_numel
    send = torch.zeros(n, dtype=H.TORCH_DT[wl.dtype], device="cuda")
    recv = [None if g == wl.group_of[root] else send for g in range(wl.G)]
    kt.kt_bcast_send(ctx, root, send)
    kt.kt_bcast_recv(ctx, root, recv)
    torch.cuda.synchronize()
    for r in range(wl.K):
        for t in range(wl.T):
            H.assert_bit_equal(dev[r][t], host[root][t], "bcast rank %d tensor %d" % (r, t))
    kt.kt_destroy(ctx)


def test_maximum_ranks_and_groups(kt, oracle):
    rnd = random.Random(64)
    group_of = [r % 16 for r in range(64)]
    rnd.shuffle(group_of)
    shares = [rnd.randint(1, 300) for _ in range(64)]
    for dtype in ("f32", "bf16"):
        wl = W.Workload("max_ranks", 60, [(5000,), (3,), (4096,), (2049,)], dtype, group_of, shares)
        all_routes(kt, oracle, wl)
    with pytest.raises(kt.KtError) as e:
        kt.kt_groups_init(list(range(17)), [1] * 17, 17)
    assert e.value.status == kt.KT_ERR_INVALID
    with pytest.raises(kt.KtError) as e:
        kt.kt_groups_init([0] * 65, [1] * 65, 1)
    assert e.value.status == kt.KT_ERR_INVALID


def test_three_thousand_small_tensors(kt, oracle):
    rnd = random.Random(3000)
    shapes = [(rnd.choice([1, 2, 7, 8, 9, 63, 64, 100, 513, 2048, 2050]),) for _ in range(3000)]
    wl = W.Workload("many_tensors", 61, shapes, "f32", [0, 1, 1, 0, 2], [3, 1, 4, 1, 5], bucket_cap_bytes=1 << 16)
    all_routes(kt, oracle, wl)
    plan = kt.kt_plan_buckets(wl.numel, wl.bucket_cap_bytes)
    assert plan.n_buckets > 10


def test_maximum_ranks_and_groups_with_one_context_per_rank(kt, oracle):
    """The same limits with every rank a context of its own (one rank per device, emulated in
    one process): 64 ranks in 16 groups of uneven sizes, shares that leave members of the big
    groups with an empty range on the short tensors; then one group of 64 (the one-pass route
    split 64 ways)."""
    import test_gpu_sharded as TS
    rnd = random.Random(640)
    group_of = [min(15, r // 3) for r in range(64)]            # 15 groups of 3 and one of 19
    shares = [rnd.randint(1, 300) for _ in range(64)]
    shapes = [(5,), (40000,), (1,), (2049,), (300000,), (17,)]
    for dtype, relay in (("f32", True), ("bf16", False)):
        wl = W.Workload("max_sharded", 72, shapes, dtype, group_of, shares, bucket_cap_bytes=1 << 20)
        host, dev = H.device_gradients(wl)
        TS.run_emulated(kt, oracle, wl, host, dev, H.TORCH_DT[dtype], 1.0 / 3.0, True, relay)
    wl = W.Workload("one_group_of_64", 73, shapes, "f32", [0] * 64, shares)
    host, dev = H.device_gradients(wl)
    TS.run_emulated(kt, oracle, wl, host, dev, torch.float32, 1.0, False, False, True)
    wl = W.Workload("max_sharded_bcast", 74, shapes, "bf16", group_of, shares, bucket_cap_bytes=1 << 20)
    TS.run_emulated_broadcast(kt, oracle, wl, 63, True)
