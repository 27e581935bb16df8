"""The loop a trainer runs with online adaptation (paper Section III-C, "Online Adaptation"):
measure step times, feed them to kt_adapt_observe, and when the shares change hand them to
kt_set_shares so that the next gradient synchronisation weights the ranks by their new batch
sizes.  Every synchronisation of the loop -- eager calls and a recorded step that is recorded
again after each change -- is compared with the oracle bit for bit, the oracle being driven by
its own adaptation state."""
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


@pytest.mark.parametrize("name,staged", [("tiny", False), ("mobilenet_v2", False), ("resnet18", True)])
def test_shares_change_mid_training(kt, oracle, name, staged):
    wl = W.by_name(name)
    K, B = wl.K, 256
    rng = np.random.default_rng(31)
    start = [B // K] * K                                    # training starts with equal batches
    host, dev = H.device_gradients(wl)
    ctx = kt.kt_groups_init(wl.group_of, start, wl.G)
    kt.kt_bucket_pack(ctx, dev, wl.bucket_cap_bytes)
    n = kt.kt_plan_query(ctx).transport_numel
    transport = [torch.full((n,), float("nan"), device="cuda") for _ in range(wl.G)]
    recv = [torch.full((n,), float("nan"), device="cuda") for _ in range(wl.G)]
    pinned = [torch.zeros(n).pin_memory() for _ in range(wl.G)]
    out = [[torch.full((m,), float("nan"), device="cuda") for m in wl.numel]]
    main, s1, s2 = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()

    def sync_once():
        kt.kt_hier_reduce(ctx, kt.KT_INTRA, transport, stream=main)
        src = transport
        if staged:
            kt.kt_relay_through_host(ctx, transport, pinned, recv, s1, s2, main_stream=main)
            kt.kt_stage_wait(ctx, kt.KT_H2D, main_stream=main)
            src = recv
        kt.kt_unpack_scale(ctx, src, out, stream=main)

    def record():
        torch.cuda.synchronize()
        kt.kt_graph_begin(ctx, main)
        sync_once()
        return kt.kt_graph_end(ctx, main)

    def check(shares, what):
        torch.cuda.synchronize()
        want, parts, _, _ = H.run_oracle_path(oracle, wl, host, shares)
        for g in range(wl.G):
            H.assert_bit_equal((recv if staged else transport)[g], parts[g], "%s: partial %d" % (what, g))
        for t in range(wl.T):
            H.assert_bit_equal(out[0][t], want[t], "%s: out[%d]" % (what, t))
        for t in out[0]:
            t.fill_(float("nan"))

    # per-sample speeds: the last quarter of the ranks is slower; later one fast rank throttles
    tau = np.array([1.0] * (K - K // 4) + [1.7] * (K // 4)) / 64.0
    ad_lib = kt.kt_adapt_create(start, B, 0.5, 3, 0.02)
    ad_ora = oracle.Adapter(start, B, 0.5, 3, 0.02)
    with torch.cuda.stream(main):
        sync_once()                                          # uploads tables, creates events
        check(start, "first step")
        graph = record()
        in_use, changes = list(start), 0
        for step in range(24):
            if step == 12:
                tau[0] *= 2.5
            times = (tau * np.array(in_use) * (1.0 + rng.uniform(-0.01, 0.01, size=K))).tolist()
            shares, changed = kt.kt_adapt_observe(ad_lib, times)
            assert changed == ad_ora.observe(times) and shares == ad_ora.shares.tolist()
            if changed:
                changes += 1
                in_use = shares
                kt.kt_set_shares(ctx, shares)                # weights of every later launch
                a, Wg = kt.kt_get_coefficients(ctx)
                oa, oW, _ = oracle.coefficients(wl.group_of, shares, wl.G)
                assert a == oa.tolist() and Wg == oW.tolist()
                sync_once()
                check(ad_ora.shares.tolist(), "eager step after change %d" % changes)
                kt.kt_graph_destroy(graph)
                graph = record()                             # a recording freezes the weights
            kt.kt_graph_launch(graph, main)
            check(ad_ora.shares.tolist(), "recorded step %d" % step)
        assert changes >= 2 and in_use != start
    kt.kt_graph_destroy(graph)
    kt.kt_adapt_destroy(ad_lib)
    kt.kt_destroy(ctx)
