"""Randomised GPU parity: many small problems with random rank counts, group layouts,
shares, ragged tensor lists, dtypes, per-tensor misalignment, bucket caps, output copies and
routes (fused / combined buffer / relay), each compared with the oracle bit for bit."""
import random

import numpy as np
import pytest
import torch

from paper_2505_10183_b200 import workloads as W

import _harness as H

pytestmark = pytest.mark.gpu

SIZES = [0, 1, 3, 7, 8, 9, 15, 16, 17, 63, 64, 65, 100, 511, 512, 1000, 2047, 2048, 2049, 4095, 4096, 4097,
         8191, 8192, 10000, 40000]


@pytest.fixture(scope="module")
def kt():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    from paper_2505_10183_b200 import binding
    torch.cuda.set_device(0)
    return binding


def random_problem(rnd):
    K = rnd.randint(1, 12)
    G = rnd.randint(1, min(K, 5))
    group_of = list(range(G)) + [rnd.randrange(G) for _ in range(K - G)]
    rnd.shuffle(group_of)
    shares = [rnd.randint(1, 200) for _ in range(K)]
    T = rnd.randint(1, 14)
    numel = [rnd.choice(SIZES) for _ in range(T)]
    if sum(numel) == 0:
        numel[0] = 5
    dtype = rnd.choice(["f32", "bf16"])
    cap = rnd.choice([64, 4096, 40000, 1 << 20, 1 << 40])
    wl = W.Workload("random", 50 + rnd.randint(0, 40), [(n,) for n in numel], dtype, group_of, shares,
                    bucket_cap_bytes=cap)
    return wl


def run_case(kt, oracle, rnd):
    wl = random_problem(rnd)
    tdt = H.TORCH_DT[wl.dtype]
    out_dtype = rnd.choice([torch.float32, torch.bfloat16])
    R = rnd.randint(1, min(3, wl.K))
    scale = rnd.choice([1.0, 0.5, 1.0 / 3.0, 1.0 / sum(wl.shares)])
    route = rnd.choice(["fused", "fused_buckets", "combined", "relay", "staged_buckets"])
    # device gradients, every tensor with its own random element misalignment
    host, dev = [], []
    for r in range(wl.K):
        ts = W.split_tensors(W.rank_gradients(wl, r, "cpu"), wl.numel)
        host.append([W.as_numpy(t) for t in ts])
        row = []
        for t in ts:
            m = rnd.choice([0, 0, 0, 1, 2, 3, 4, 5])
            buf = torch.empty(t.numel() + m, dtype=tdt, device="cuda")
            buf[m:].copy_(t)
            row.append(buf[m:])
        dev.append(row)
    kw = dict(out_dtype=out_dtype, R=R, scale=scale)
    if route == "fused_buckets":
        kw["per_bucket"] = True
    elif route == "combined":
        kw.update(use_combined=True, per_bucket=rnd.random() < 0.5)
    elif route == "relay":
        kw.update(staged=rnd.choice(["relay", "relay_all"]), relay_chunk=rnd.choice([256, 1024, 65536, 1 << 19, 1 << 22]))
    elif route == "staged_buckets":
        kw.update(staged=True, per_bucket=True)
    out, transport, plan, ctx = H.run_gpu_path(kt, wl, dev, wl.shares, **kw)
    odt = {torch.float32: 0, torch.bfloat16: 1}[out_dtype]
    o_out, o_parts, _, o_plan = H.run_oracle_path(oracle, wl, host, wl.shares, out_dtype=odt, scale=scale)
    what = "K=%d G=%d T=%d %s->%s route=%s" % (wl.K, wl.G, wl.T, wl.dtype, out_dtype, route)
    assert plan.tensor_offset == o_plan.tensor_offset.tolist(), what
    assert plan.transport_numel == o_plan.transport_numel, what
    for g in range(wl.G):
        H.assert_bit_equal(transport[g], o_parts[g], what + " transport[%d]" % g)
    for c in range(R):
        for t in range(wl.T):
            H.assert_bit_equal(out[c][t], o_out[t], what + " out[%d][%d]" % (c, t))
    kt.kt_destroy(ctx)


@pytest.mark.parametrize("seed", range(8))
def test_random_problems(kt, oracle, seed):
    rnd = random.Random(1000 + seed)
    for _ in range(25):
        run_case(kt, oracle, rnd)


def test_output_guard_bytes_untouched(kt, oracle):
    """Nothing is written outside the output tensors or the transport range: guard words
    around every buffer keep their pattern."""
    rnd = random.Random(77)
    for _ in range(10):
        wl = random_problem(rnd)
        tdt = H.TORCH_DT[wl.dtype]
        host, dev = H.device_gradients(wl)
        ctx = kt.kt_groups_init(wl.group_of, wl.shares, wl.G)
        kt.kt_bucket_pack(ctx, dev, wl.bucket_cap_bytes)
        n = kt.kt_plan_query(ctx).transport_numel
        guard = 64
        tbuf = [torch.full((n + 2 * guard,), -777.0, device="cuda") for _ in range(wl.G)]
        transport = [b[guard:guard + n] for b in tbuf]
        obuf = [torch.full((m + 2 * guard,), -777.0, dtype=tdt, device="cuda") for m in wl.numel]
        out = [[b[guard:guard + m] for b, m in zip(obuf, wl.numel)]]
        kt.kt_hier_reduce(ctx, kt.KT_INTRA, transport)
        kt.kt_unpack_scale(ctx, transport, out)
        torch.cuda.synchronize()
        for b in tbuf:
            assert bool((b[:guard] == -777.0).all()) and bool((b[-guard:] == -777.0).all())
        for b, m in zip(obuf, wl.numel):
            assert bool((b[:guard] == -777.0).all()) and bool((b[guard + m:] == -777.0).all())
        kt.kt_destroy(ctx)


def test_contexts_on_different_host_threads(kt, oracle):
    """Different contexts may be used from different host threads at the same time (the
    header's promise): four threads, each with contexts, streams and buffers of its own, run
    random problems side by side; every result equals the oracle's, and a failing call on one
    thread leaves its message on that thread only."""
    import threading
    failures = []

    def worker(i):
        try:
            torch.cuda.set_device(0)
            rnd = random.Random(31000 + i)
            with torch.cuda.stream(torch.cuda.Stream()):
                for _ in range(12):
                    run_case(kt, oracle, rnd)
                    if i == 0:                          # one thread keeps failing calls going
                        with pytest.raises(kt.KtError):
                            kt.kt_groups_init([0, 2], [1, 1], 3)
                        assert "outside" in kt.kt_last_error()
                    else:
                        assert kt.kt_last_error() == ""
        except BaseException as e:                      # reported by the main thread
            failures.append((i, repr(e)))

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(4)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not failures, failures
