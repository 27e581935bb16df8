"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the
same seeded inputs.  Bars: bit-exact for pack / unpack / casts / shares / plan; for the
reductions the kernels follow the oracle's operation order, so results are compared bit
for bit as well, and the stated tolerances (1e-6 relative for fp32 sources, 1e-2 for
bf16-sourced gradients) are checked against an fp64 weighted mean on top."""
import random

import numpy as np
import pytest
import torch

from paper_2505_10183_b200 import workloads as W

import _harness as H

pytestmark = pytest.mark.gpu

F32, BF16 = 0, 1


@pytest.fixture(scope="module")
def kt():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    from paper_2505_10183_b200 import binding
    torch.cuda.set_device(0)
    return binding


def compare_all(kt, oracle, wl, **kw):
    shares = H.shares_of(wl, kt)
    host, dev = H.device_gradients(wl, misalign=kw.pop("misalign", 0))
    out, transport, plan, ctx = H.run_gpu_path(kt, wl, dev, shares, **kw)
    o_out, o_parts, o_S, o_plan = H.run_oracle_path(
        oracle, wl, host, shares, scale=kw.get("scale", 1.0),
        out_dtype=None if kw.get("out_dtype") is None else {torch.float32: F32, torch.bfloat16: BF16}[kw["out_dtype"]])
    # plan: integers, exact
    assert plan.n_buckets == o_plan.n_buckets
    assert plan.tensor_offset == o_plan.tensor_offset.tolist()
    assert plan.bucket_of == o_plan.bucket_of.tolist()
    assert plan.bucket_start == o_plan.bucket_start.tolist()
    assert plan.bucket_numel == o_plan.bucket_numel.tolist()
    assert plan.transport_numel == o_plan.transport_numel
    # group partials incl. zero padding, then every output copy
    for g in range(wl.G):
        H.assert_bit_equal(transport[g], o_parts[g], "transport[%d]" % g)
    for c in range(len(out)):
        for t in range(wl.T):
            H.assert_bit_equal(out[c][t], o_out[t], "out[%d][%d]" % (c, t))
    kt.kt_destroy(ctx)
    return host, out, shares


def check_tolerance(oracle, wl, host, out, shares):
    """Stated tolerance against the fp64 weighted mean, forward-error denominator."""
    dt = H.ORACLE_DT[wl.dtype]
    xs = [np.concatenate(h) for h in host]
    F, absF = oracle.flat_reduce_f64(xs, dt, shares)
    got = np.concatenate([W.as_numpy(t) for t in out[0]])
    if got.dtype == np.uint16:
        got = oracle.bf16_to_f32(got)
        tol = 1e-2
    else:
        tol = 1e-6
    nz = absF > 0
    assert np.max(np.abs(got[nz] - F[nz]) / absF[nz]) <= tol


# ------------------------------------------------------------------ the named configurations
def test_tiny(kt, oracle):
    wl = W.tiny()
    host, out, shares = compare_all(kt, oracle, wl)
    check_tolerance(oracle, wl, host, out, shares)


def test_schedule_matches_oracle_and_named_values(kt, oracle):
    assert kt.kt_schedule([1.0, 1.0, 1.6, 1.6], 256) == [79, 79, 49, 49]
    assert kt.kt_schedule([1.0] * 4 + [1.4] * 2 + [2.1] * 2, 256) == [40, 40, 40, 40, 29, 29, 19, 19]
    rng = np.random.default_rng(0)
    for _ in range(500):
        K = int(rng.integers(1, 17))
        times = rng.uniform(0.2, 5.0, size=K).tolist()
        B = int(rng.integers(K, 2048))
        assert kt.kt_schedule(times, B) == oracle.schedule(times, B).tolist()


def test_resnet18_staged_as_benchmarked(kt, oracle):
    """Full size, in the launch configuration the benchmark times: one fused-reduce launch,
    the partials relayed bucket by bucket through pinned host memory as a chunk pipeline, one
    combine/unpack launch.  Every element is compared."""
    wl = W.resnet18()
    host, out, shares = compare_all(kt, oracle, wl, staged="relay_all", relay_chunk=4 << 20)
    assert shares == [79, 79, 49, 49]
    check_tolerance(oracle, wl, host, out, shares)
    # the relay bucket by bucket, and odd chunk sizes: ragged last chunk, chunk larger than a bucket
    compare_all(kt, oracle, wl, staged="relay")
    compare_all(kt, oracle, wl, staged="relay_all", relay_chunk=(1 << 20) + 256)
    compare_all(kt, oracle, wl, staged="relay", relay_chunk=1 << 30)


def test_relay_with_group_buffers_as_rows_of_one_allocation(kt, oracle):
    """The layout the benchmark uses: transport, pinned and receive buffers of the G groups
    back to back, so that the relay moves a chunk of all groups in one copy.  Chunk sizes
    that do and do not divide a row, three groups, and the per-bucket relay (which cannot merge)."""
    wl = W.resnet18()
    compare_all(kt, oracle, wl, staged="relay_all", relay_chunk=4 << 20, rows=True)
    compare_all(kt, oracle, wl, staged="relay_all", relay_chunk=(3 << 20) + 256, rows=True)
    compare_all(kt, oracle, wl, staged="relay", rows=True)
    compare_all(kt, oracle, W.mobilenet_v2(), staged="relay_all", relay_chunk=1 << 20, rows=True)
    compare_all(kt, oracle, W.tiny(), staged="relay_all", relay_chunk=256, rows=True)


def test_relay_merges_the_groups_copies_only_for_rows_of_one_allocation(kt):
    """Seen from outside through a recording's node count: with the G buffers of every set as
    rows of one allocation a chunk of all groups is one copy each way; with separately
    allocated buffers it is G copies each way."""
    wl = W.mobilenet_v2()                                   # three groups
    host, dev = H.device_gradients(wl)
    ctx = kt.kt_groups_init(wl.group_of, H.shares_of(wl, kt), wl.G)
    kt.kt_bucket_pack(ctx, dev, wl.bucket_cap_bytes)
    n = kt.kt_plan_query(ctx).transport_numel
    main, a, b = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    chunk = 1 << 30
    nodes = {}
    for layout in ("rows", "separate"):
        def buffers(pinned):
            if layout == "rows":
                whole = torch.zeros(wl.G, n)
                return list(whole.pin_memory() if pinned else whole.cuda())
            # separate allocations, with a gap so that they cannot be neighbours
            return [(torch.zeros(n + 4096).pin_memory() if pinned else torch.zeros(n + 4096, device="cuda"))[:n]
                    for _ in range(wl.G)]
        send, pinned, recv = buffers(False), buffers(True), buffers(False)
        torch.cuda.synchronize()
        kt.kt_graph_begin(ctx, main)
        kt.kt_relay_through_host(ctx, send, pinned, recv, a, b, bucket=-1, chunk_bytes=chunk, main_stream=main)
        kt.kt_stage_wait(ctx, kt.KT_H2D, bucket=-1, main_stream=main)
        g = kt.kt_graph_end(ctx, main)
        nodes[layout] = kt.kt_graph_nodes(g)
        kt.kt_graph_destroy(g)
    # one chunk covers everything: one copy down and one up when merged, G of each otherwise
    assert nodes["separate"] - nodes["rows"] == 2 * (wl.G - 1), nodes
    kt.kt_destroy(ctx)


@pytest.mark.parametrize("name", ["resnet18", "resnet50", "mobilenet_v2"])
def test_host_resident_step_as_benchmarked(kt, oracle, name):
    """The benchmark's end-to-end arm (gradients start in pinned host memory, buckets pipelined
    over both directions of the host link, results end in pinned host memory), run twice in a
    row, against the oracle on the same host bytes."""
    import bench
    wl = W.by_name(name)
    arm = bench.HostResidentStep(wl, kt, 4 << 20, device_values=False)
    shares = arm.prob.shares
    with torch.cuda.stream(arm.prob.main):
        arm.step()
        arm.step()
    torch.cuda.synchronize()
    host = [[W.as_numpy(t) for t in W.split_tensors(W.rank_gradients(wl, r, "cpu"), wl.numel)] for r in range(wl.K)]
    want, _, _, _ = H.run_oracle_path(oracle, wl, host, shares)
    for t, got in enumerate(arm.result_tensors()):
        H.assert_bit_equal(got, want[t], "%s out[%d]" % (name, t))
    assert arm.h2d_bytes >= wl.K * wl.N * wl.elem_size and arm.d2h_bytes >= wl.N * wl.elem_size
    kt.kt_destroy(arm.prob.ctx)


def test_resnet18_staged_bucket_by_bucket(kt, oracle):
    """The per-bucket route: reduce, copy down, copy up and unpack one bucket at a time."""
    wl = W.resnet18()
    compare_all(kt, oracle, wl, per_bucket=True, staged=True)
    compare_all(kt, oracle, W.tiny(), staged="relay", relay_chunk=256)


def test_resnet18_single_launch(kt, oracle):
    compare_all(kt, oracle, W.resnet18())


def test_resnet50_bf16(kt, oracle):
    wl = W.resnet50()
    host, out, shares = compare_all(kt, oracle, wl, per_bucket=True)
    check_tolerance(oracle, wl, host, out, shares)
    # fp32 output of bf16 sources: 1e-6-class accuracy is kept by the fp32 accumulation
    host, out, shares = compare_all(kt, oracle, wl, out_dtype=torch.float32)
    dt = H.ORACLE_DT[wl.dtype]
    F, absF = oracle.flat_reduce_f64([np.concatenate(h) for h in host], dt, shares)
    got = np.concatenate([W.as_numpy(t) for t in out[0]])
    assert np.max(np.abs(got - F) / absF) <= 1e-6


def test_mobilenet_v2_ragged(kt, oracle):
    wl = W.mobilenet_v2()
    host, out, shares = compare_all(kt, oracle, wl)
    assert shares == [40, 40, 40, 40, 29, 29, 19, 19]
    check_tolerance(oracle, wl, host, out, shares)


@pytest.mark.parametrize("name", ["tiny", "resnet18", "mobilenet_v2", "resnet50"])
def test_named_workloads_with_unequal_shares_inside_groups(kt, oracle, name):
    """The named configurations put equally fast devices in a group: in-group weights of 1/2
    and 1/4, with which every product of the reduce is exact and a fused multiply-add cannot
    differ from a multiply and an add.  The same tensor lists with shares that differ inside
    every group make each term of each chain round."""
    wl = W.by_name(name)
    wl.shares = {4: [83, 75, 45, 53], 8: [37, 41, 43, 47, 23, 31, 17, 17]}[wl.K]
    host, out, shares = compare_all(kt, oracle, wl)
    assert shares == wl.shares
    check_tolerance(oracle, wl, host, out, shares)


@pytest.mark.parametrize("K", [2, 4, 8, 16])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("nbytes", [4 << 10, 64 << 10, 1 << 20, 16 << 20])
def test_sweep_small_points(kt, oracle, K, dtype, nbytes):
    compare_all(kt, oracle, W.sweep_point(K, nbytes, dtype))


def check_sampled_windows(kt, oracle, K, nbytes, dtype, n_random=6):
    """A flat sweep point too large for the oracle to walk in full: device-generated values;
    2^20-element windows (the first, the last, and random ones at odd offsets) are copied to
    the host and checked element by element.  The path is element-wise, so a window's result
    depends on that window's inputs only."""
    wl = W.sweep_point(K, nbytes, dtype)
    shares = wl.shares
    n = wl.N
    dt = H.ORACLE_DT[dtype]
    dev = [[W.rank_gradients(wl, r, "cuda")] for r in range(wl.K)]
    ctx = kt.kt_groups_init(wl.group_of, shares, wl.G)
    kt.kt_bucket_pack(ctx, dev, wl.bucket_cap_bytes)
    plan = kt.kt_plan_query(ctx)
    assert plan.transport_numel == n and plan.n_buckets == 1
    transport = [torch.full((n,), float("nan"), device="cuda") for _ in range(wl.G)]
    out = [[torch.full((n,), float("nan"), dtype=H.TORCH_DT[dtype], device="cuda")]]
    direct = [[torch.full((n,), float("nan"), dtype=H.TORCH_DT[dtype], device="cuda")]]
    kt.kt_hier_reduce(ctx, kt.KT_INTRA, transport)
    kt.kt_unpack_scale(ctx, transport, out)
    kt.kt_sync_direct(ctx, direct)
    torch.cuda.synchronize()
    win = 1 << 20
    rng = np.random.default_rng(5 + K)
    starts = [0, n - win] + (rng.integers(0, n // win - 1, size=n_random) * win + 12344).tolist()
    for s in starts:
        s = int(min(max(s, 0), n - win))
        hx = [[W.as_numpy(dev[r][0][s:s + win])] for r in range(wl.K)]
        o_out, o_parts, _, _ = oracle.sync_step(hx, [win], dt, wl.group_of, shares, wl.G, 1 << 62)
        for g in range(wl.G):
            H.assert_bit_equal(transport[g][s:s + win], o_parts[g], "window %d transport[%d]" % (s, g))
        H.assert_bit_equal(out[0][0][s:s + win], o_out[0], "window %d out" % s)
        H.assert_bit_equal(direct[0][0][s:s + win], o_out[0], "window %d one-pass out" % s)
    # no window was skipped by the kernels: nothing of the NaN fill is left anywhere
    for t in transport + out[0] + direct[0]:
        assert not bool(torch.isnan(t).any())
    kt.kt_destroy(ctx)
    del dev, transport, out, direct
    torch.cuda.empty_cache()


@pytest.mark.parametrize("K", [4, 8, 16])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("nbytes", [64 << 20, 256 << 20, 1 << 30])
def test_sweep_large_points_sampled_windows(kt, oracle, K, dtype, nbytes):
    """The bucket sizes the bandwidth target is stated for (64 MiB and up per rank, the points
    the benchmark times among them), with 4, 8 and 16 ranks, fp32 and bf16 gradients."""
    check_sampled_windows(kt, oracle, K, nbytes, dtype)


def test_a_tensor_of_more_than_two_to_the_31_elements(kt, oracle):
    """One tensor per rank with 2^31 + 2^20 + 40 elements (8.6 GB of fp32 per rank, two ranks, two
    groups): element offsets no longer fit 32 bits; the windows checked include the last 2^20
    elements and one that straddles element 2^31."""
    n = (1 << 31) + (1 << 20) + 40
    wl = W.sweep_point(2, n * 4, "f32")
    assert wl.N == n
    dev = [[W.rank_gradients(wl, r, "cuda")] for r in range(wl.K)]
    ctx = kt.kt_groups_init(wl.group_of, wl.shares, wl.G)
    kt.kt_bucket_pack(ctx, dev, wl.bucket_cap_bytes)
    plan = kt.kt_plan_query(ctx)
    tn = plan.transport_numel
    assert tn == -(-n // 64) * 64
    transport = [torch.full((tn,), float("nan"), device="cuda") for _ in range(wl.G)]
    out = [[torch.full((n,), float("nan"), device="cuda")]]
    kt.kt_hier_reduce(ctx, kt.KT_INTRA, transport)
    kt.kt_unpack_scale(ctx, transport, out)
    torch.cuda.synchronize()
    win = 1 << 20
    for s in (0, (1 << 31) - win // 2, n - win, (1 << 30) + 12344):
        hx = [[W.as_numpy(dev[r][0][s:s + win])] for r in range(wl.K)]
        o_out, o_parts, _, _ = oracle.sync_step(hx, [win], F32, wl.group_of, wl.shares, wl.G, 1 << 62)
        for g in range(wl.G):
            H.assert_bit_equal(transport[g][s:s + win], o_parts[g], "window %d transport[%d]" % (s, g))
        H.assert_bit_equal(out[0][0][s:s + win], o_out[0], "window %d out" % s)
    assert not bool(torch.isnan(out[0][0]).any())
    assert bool((transport[0][n:] == 0).all()) and bool((transport[1][n:] == 0).all())      # the padding behind the tail
    # the one-pass route into the same output
    out[0][0].fill_(float("nan"))
    kt.kt_sync_direct(ctx, out)
    torch.cuda.synchronize()
    s = n - win
    hx = [[W.as_numpy(dev[r][0][s:s + win])] for r in range(wl.K)]
    o_out, _, _, _ = oracle.sync_step(hx, [win], F32, wl.group_of, wl.shares, wl.G, 1 << 62)
    H.assert_bit_equal(out[0][0][s:s + win], o_out[0], "one-pass, last window")
    assert not bool(torch.isnan(out[0][0]).any())
    kt.kt_destroy(ctx)
    del dev, transport, out
    torch.cuda.empty_cache()


# ------------------------------------------------------------------ variants and edge cases
def test_misaligned_sources_take_the_element_path(kt, oracle):
    for wl in (W.tiny(), W.sweep_point(4, 1 << 20, "bf16"), W.sweep_point(2, 1 << 20, "f32")):
        compare_all(kt, oracle, wl, misalign=1)
        compare_all(kt, oracle, wl, misalign=3)


def test_broadcast_copies_and_scale(kt, oracle):
    wl = W.tiny()
    compare_all(kt, oracle, wl, R=wl.K, scale=0.125)
    wl = W.mobilenet_v2()
    compare_all(kt, oracle, wl, R=3, scale=1.0 / 3.0)


def test_combined_buffer_route(kt, oracle):
    compare_all(kt, oracle, W.tiny(), use_combined=True)
    compare_all(kt, oracle, W.resnet18(), use_combined=True, per_bucket=True)


def test_bf16_out_from_f32_sources_and_back(kt, oracle):
    compare_all(kt, oracle, W.tiny(), out_dtype=torch.bfloat16)
    compare_all(kt, oracle, W.sweep_point(4, 1 << 20, "bf16"), out_dtype=torch.float32)


def test_empty_and_odd_tensors(kt, oracle):
    wl = W.Workload("odd", 7, [(0,), (1,), (7,), (2049,), (0,), (4096,), (13,)], "f32",
                    [0, 1, 1, 2, 0], [3, 5, 7, 11, 13], bucket_cap_bytes=5000 * 4)
    compare_all(kt, oracle, wl)
    compare_all(kt, oracle, wl, per_bucket=True, R=2)
    wl.dtype = "bf16"
    compare_all(kt, oracle, wl)


def test_single_rank_and_singleton_groups(kt, oracle):
    wl = W.Workload("one", 8, [(5000,)], "f32", [0], [7])
    host, out, _ = compare_all(kt, oracle, wl)
    assert np.array_equal(W.as_numpy(out[0][0]), host[0][0])          # K = 1: identity
    wl = W.Workload("singletons", 9, [(3000,), (17,)], "f32", [0, 1, 2, 3, 4], [5, 9, 17, 3, 30])
    compare_all(kt, oracle, wl)


def test_identical_ranks_and_equal_shares(kt, oracle):
    wl = W.tiny()
    flat = W.rank_gradients(wl, 0, "cpu")
    dev = [[t.cuda() for t in W.split_tensors(flat, wl.numel)] for _ in range(4)]
    out, *_ = H.run_gpu_path(kt, wl, dev, [64, 64, 64, 64])
    for t, ref in zip(out[0], W.split_tensors(flat, wl.numel)):
        assert torch.equal(t.cpu(), ref)                               # exact: all weights are powers of two
    # equal shares: arithmetic mean
    host, dev = H.device_gradients(wl)
    out, *_ = H.run_gpu_path(kt, wl, dev, [32] * 4)
    stack = np.stack([np.concatenate(h).astype(np.float64) for h in host])
    got = np.concatenate([W.as_numpy(t) for t in out[0]])
    assert np.max(np.abs(got - stack.mean(0)) / np.abs(stack).mean(0)) < 1e-6


@pytest.mark.parametrize("name", ["tiny", "mobilenet_v2"])
def test_two_kernel_route_in_place(kt, oracle, name):
    """The reduced gradients overwrite the registered gradient tensors of every rank (the usual
    in-place all-reduce): the fused reduce has read everything before the combine writes."""
    wl = W.by_name(name)
    shares = H.shares_of(wl, kt)
    host, dev = H.device_gradients(wl, misalign=1)
    ctx = kt.kt_groups_init(wl.group_of, shares, wl.G)
    kt.kt_bucket_pack(ctx, dev, wl.bucket_cap_bytes)
    n = kt.kt_plan_query(ctx).transport_numel
    transport = [torch.full((n,), float("nan"), device="cuda") for _ in range(wl.G)]
    kt.kt_hier_reduce(ctx, kt.KT_INTRA, transport)
    kt.kt_unpack_scale(ctx, transport, dev, scale=0.25)          # R = K copies: every rank's own tensors
    torch.cuda.synchronize()
    want, _, _, _ = H.run_oracle_path(oracle, wl, host, shares, scale=0.25)
    for r in range(wl.K):
        for t in range(wl.T):
            H.assert_bit_equal(dev[r][t], want[t], "rank %d tensor %d" % (r, t))
    kt.kt_destroy(ctx)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_special_values_pass_through_like_in_the_oracle(kt, oracle, dtype):
    """Infinities, NaNs, subnormals, signed zeros and the largest finite values among the
    gradients (an overflowed mixed-precision step looks like this): wherever the oracle's result
    is a NaN the kernels' is one too; everything else -- infinities, subnormal results (nothing
    is flushed to zero), the sign of a zero -- is bit-equal, on both routes."""
    wl = W.Workload("special", 11, [(4099,), (64,), (9,)], dtype, [0, 0, 1, 1, 1], [3, 5, 7, 2, 1])
    rng = np.random.default_rng(41)
    specials32 = np.array([np.inf, -np.inf, np.nan, 0.0, -0.0, 1e-45, -3e-41, 1.1754942e-38, 3.4028235e38, -3.4028235e38,
                           1e-30, 65504.0], np.float32)
    host, dev = [], []
    for r in range(wl.K):
        ts = []
        for t_i, n in enumerate(wl.numel):
            x = (rng.standard_normal(n) * 1e-3).astype(np.float32)
            where = rng.random(n) < 0.2
            x[where] = rng.choice(specials32, size=int(where.sum()))
            t = torch.from_numpy(x)
            ts.append(t.to(torch.bfloat16) if dtype == "bf16" else t)
        host.append([W.as_numpy(t) for t in ts])
        dev.append([t.cuda() for t in ts])
    for odt in (torch.float32, torch.bfloat16):
        out, transport, plan, ctx = H.run_gpu_path(kt, wl, dev, wl.shares, out_dtype=odt, scale=0.5)
        direct = [[torch.full_like(o, 1.0) for o in out[0]]]
        kt.kt_sync_direct(ctx, direct, scale=0.5)
        torch.cuda.synchronize()
        want, parts, _, _ = H.run_oracle_path(oracle, wl, host, wl.shares, out_dtype=0 if odt == torch.float32 else 1, scale=0.5)

        def same(got, exp, what):
            g = W.as_numpy(got)
            gf = g if g.dtype == np.float32 else oracle.bf16_to_f32(g)
            ef = exp if exp.dtype == np.float32 else oracle.bf16_to_f32(exp)
            nan = np.isnan(ef)
            assert np.array_equal(np.isnan(gf), nan), what
            assert np.array_equal(H.bits(g)[~nan], H.bits(exp)[~nan]), what
            return int(nan.sum()), int(np.isinf(ef).sum()), int(((ef != 0) & (np.abs(ef) < 1.1754942e-38)).sum())

        seen = np.zeros(3, int)
        for g in range(wl.G):
            seen += same(transport[g], parts[g], "partial %d" % g)
        for t in range(wl.T):
            same(out[0][t], want[t], "out[%d]" % t)
            same(direct[0][t], want[t], "one-pass out[%d]" % t)
        assert seen[0] > 0 and seen[1] > 0 and (seen[2] > 0 or dtype == "bf16")      # the cases did occur
        kt.kt_destroy(ctx)


def test_sum_then_divide_coefficients(kt, oracle):
    """Plain sums across the hierarchy with one final division (weights a_r = b_r, W_g = 1,
    scale 1/B) through kt_set_coefficients; oracle fed the same coefficients."""
    wl = W.tiny()
    shares = wl.shares
    host, dev = H.device_gradients(wl)
    ctx = kt.kt_groups_init(wl.group_of, shares, wl.G)
    kt.kt_set_coefficients(ctx, [float(b) for b in shares], [1.0] * wl.G)
    a, Wg = kt.kt_get_coefficients(ctx)
    assert a == [float(b) for b in shares] and Wg == [1.0] * wl.G
    kt.kt_bucket_pack(ctx, dev, wl.bucket_cap_bytes)
    plan = kt.kt_plan_query(ctx)
    tr = [torch.empty(plan.transport_numel, device="cuda") for _ in range(wl.G)]
    out = [[torch.empty(m, device="cuda") for m in wl.numel]]
    kt.kt_hier_reduce(ctx, kt.KT_INTRA, tr)
    kt.kt_unpack_scale(ctx, tr, out, scale=1.0 / sum(shares))
    torch.cuda.synchronize()
    oplan = oracle.bucket_plan(wl.numel, wl.bucket_cap_bytes)
    parts = oracle.intra_reduce(host, oplan, F32, wl.group_of, np.array(shares, np.float32), wl.G)
    S = oracle.combine(parts, np.ones(wl.G, np.float32))
    want = oracle.unpack_scale(S, oplan, np.float32(1.0 / sum(shares)), F32)
    for t in range(wl.T):
        H.assert_bit_equal(out[0][t], want[t])
    # and switching back to share-derived weights
    kt.kt_set_shares(ctx, shares)
    a, Wg = kt.kt_get_coefficients(ctx)
    oa, oW, _ = oracle.coefficients(wl.group_of, shares, wl.G)
    assert a == oa.tolist() and Wg == oW.tolist()
    kt.kt_destroy(ctx)


def test_standalone_pack(kt, oracle):
    for wl in (W.tiny(), W.mobilenet_v2()):
        for dtype in ("f32", "bf16"):
            wl.dtype = dtype
            host, dev = H.device_gradients(wl)
            ctx = kt.kt_groups_init(wl.group_of, H.shares_of(wl, kt), wl.G)
            n = kt.kt_plan_buckets(wl.numel, wl.bucket_cap_bytes).transport_numel
            flat = [torch.full((n,), 1.0, dtype=H.TORCH_DT[dtype], device="cuda") for _ in range(wl.K)]
            kt.kt_bucket_pack(ctx, dev, wl.bucket_cap_bytes, flat_out=flat)
            torch.cuda.synchronize()
            oplan = oracle.bucket_plan(wl.numel, wl.bucket_cap_bytes)
            for r in range(wl.K):
                H.assert_bit_equal(flat[r], oracle.pack(host[r], oplan, H.ORACLE_DT[dtype]), "flat[%d]" % r)
            kt.kt_destroy(ctx)


def test_cast_kernels_exhaustive(kt, oracle):
    # bf16 -> fp32: all 65 536 patterns
    h = torch.arange(65536, dtype=torch.int32).to(torch.int16).view(torch.bfloat16).cuda()
    f = torch.empty(65536, device="cuda")
    kt.kt_cast(h, f)
    want = oracle.bf16_to_f32(np.arange(65536, dtype=np.uint16))
    got = f.cpu().numpy()
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    # fp32 -> bf16: all 2^32 patterns, 2^26 at a time
    chunk = 1 << 26
    base = torch.arange(chunk, dtype=torch.int64, device="cuda")
    out = torch.empty(chunk, dtype=torch.bfloat16, device="cuda")
    from concurrent.futures import ThreadPoolExecutor
    pool = ThreadPoolExecutor(8)
    for c in range(64):
        bits = (base + c * chunk).to(torch.int32).contiguous()      # wraps to the signed pattern
        kt.kt_cast(bits.view(torch.float32), out)
        got = out.view(torch.int16).cpu().numpy().view(np.uint16)
        fb = bits.cpu().numpy().view(np.float32)
        parts = list(pool.map(oracle.f32_to_bf16, np.array_split(fb, 8)))
        want = np.concatenate(parts)
        nan = np.isnan(fb)
        assert np.array_equal(got[~nan], want[~nan]), "chunk %d" % c
        if nan.any():
            assert np.all(np.isnan(oracle.bf16_to_f32(got[nan])))
    pool.shutdown()


# ------------------------------------------------------------------ staging
def test_staging_bytes_and_ordering(kt, oracle):
    """Host bytes equal the device partials; the copy never starts before the reduce that
    feeds it has finished (the transport is poisoned right before the reduce is queued)."""
    wl = W.resnet18()
    shares = H.shares_of(wl, kt)
    host_g, dev = H.device_gradients(wl)
    ctx = kt.kt_groups_init(wl.group_of, shares, wl.G)
    kt.kt_bucket_pack(ctx, dev, wl.bucket_cap_bytes)
    plan = kt.kt_plan_query(ctx)
    n = plan.transport_numel
    tr = [torch.empty(n, device="cuda") for _ in range(wl.G)]
    pinned = [torch.zeros(n).pin_memory() for _ in range(wl.G)]
    side = torch.cuda.Stream()
    poison = float(np.float32(-7.25e33))
    for _ in range(3):
        for t in tr:
            t.fill_(poison)
        kt.kt_hier_reduce(ctx, kt.KT_INTRA, tr)
        kt.kt_stage_to_host(ctx, kt.KT_D2H, tr, pinned, side_stream=side)
        kt.kt_stage_wait(ctx, kt.KT_D2H, timeout_ms=20000)
        for g in range(wl.G):
            assert not (pinned[g] == poison).any()
            assert torch.equal(pinned[g], tr[g].cpu())
    _, o_parts, _, _ = H.run_oracle_path(oracle, wl, host_g, shares)
    for g in range(wl.G):
        H.assert_bit_equal(pinned[g], o_parts[g])
    kt.kt_destroy(ctx)


def test_relay_of_host_buffers_that_are_neighbours_but_separate_allocations(kt, oracle):
    """The relay moves a chunk of all groups in one copy when the G buffers of each set are rows
    of one allocation.  Lying back to back is not enough for that: here the device buffers are
    rows of one allocation, but the host buffers are two halves of one mapping that were
    page-locked by two separate calls -- neighbours in the address space, two allocations to the
    driver, which refuses a copy that runs across the seam.  The relay has to notice and copy
    group by group."""
    import ctypes
    import mmap
    wl = W.sweep_point(4, 4096 * 4, "f32")
    host, dev = H.device_gradients(wl)
    ctx = kt.kt_groups_init(wl.group_of, wl.shares, wl.G)
    kt.kt_bucket_pack(ctx, dev, wl.bucket_cap_bytes)
    n = kt.kt_plan_query(ctx).transport_numel
    nbytes = n * 4
    assert nbytes % mmap.PAGESIZE == 0
    block = mmap.mmap(-1, wl.G * nbytes)
    view = (ctypes.c_char * (wl.G * nbytes)).from_buffer(block)
    base = ctypes.addressof(view)
    for g in range(wl.G):
        kt.kt_host_register(base + g * nbytes, nbytes)
    crossed = None
    try:
        send = torch.full((wl.G, n), float("nan"), device="cuda")
        recv = torch.full((wl.G, n), float("nan"), device="cuda")
        pinned = kt.PtrArray.from_addresses([base + g * nbytes for g in range(wl.G)], keep=block)
        down, up = torch.cuda.Stream(), torch.cuda.Stream()
        kt.kt_hier_reduce(ctx, kt.KT_INTRA, list(send))
        kt.kt_relay_through_host(ctx, list(send), pinned, list(recv), down, up, bucket=-1, chunk_bytes=4096)
        kt.kt_stage_wait(ctx, kt.KT_H2D, bucket=-1)
        torch.cuda.synchronize()
        _, o_parts, _, _ = H.run_oracle_path(oracle, wl, host, wl.shares)
        crossed = np.frombuffer(view, dtype=np.float32).reshape(wl.G, n)
        for g in range(wl.G):
            H.assert_bit_equal(recv[g], o_parts[g], "received partial %d" % g)
            assert np.array_equal(H.bits(crossed[g].copy()), H.bits(o_parts[g])), "host copy of partial %d" % g
    finally:
        torch.cuda.synchronize()
        for g in range(wl.G):
            kt.kt_host_unregister(base + g * nbytes)
        kt.kt_destroy(ctx)
        del crossed, view
        block.close()


def test_whole_transport_goes_up_only_after_every_bucket_came_down(kt, oracle):
    """Mixed granularity on different copy streams: the partials go down bucket by bucket on one
    stream, the whole transport comes back up in one call on another.  The way up must wait
    for every bucket's way down (the pinned buffers are poisoned first)."""
    wl = W.resnet18()
    shares = H.shares_of(wl, kt)
    host_g, dev = H.device_gradients(wl)
    ctx = kt.kt_groups_init(wl.group_of, shares, wl.G)
    kt.kt_bucket_pack(ctx, dev, wl.bucket_cap_bytes)
    plan = kt.kt_plan_query(ctx)
    n = plan.transport_numel
    assert plan.n_buckets >= 2
    tr = [torch.empty(n, device="cuda") for _ in range(wl.G)]
    recv = [torch.empty(n, device="cuda") for _ in range(wl.G)]
    pinned = [torch.zeros(n).pin_memory() for _ in range(wl.G)]
    down, up = torch.cuda.Stream(), torch.cuda.Stream()
    poison = float(np.float32(-7.25e33))
    for _ in range(3):
        for p, r in zip(pinned, recv):
            p.fill_(poison)
            r.fill_(float("nan"))
        torch.cuda.synchronize()
        kt.kt_hier_reduce(ctx, kt.KT_INTRA, tr)
        for b in range(plan.n_buckets):
            kt.kt_stage_to_host(ctx, kt.KT_D2H, tr, pinned, bucket=b, side_stream=down)
        kt.kt_stage_to_host(ctx, kt.KT_H2D, recv, pinned, bucket=-1, side_stream=up)
        kt.kt_stage_wait(ctx, kt.KT_H2D, bucket=-1, timeout_ms=20000)
        torch.cuda.synchronize()
        for g in range(wl.G):
            assert not bool((recv[g] == poison).any())
    _, o_parts, _, _ = H.run_oracle_path(oracle, wl, host_g, shares)
    for g in range(wl.G):
        H.assert_bit_equal(recv[g], o_parts[g], "receive buffer %d" % g)
    kt.kt_destroy(ctx)


def random_staging_traffic(kt, oracle, rnd, rounds):
    """Steps queued back to back without any synchronisation, each choosing its own granularity
    for every phase (whole transport or bucket by bucket, for the reduce, the way down, the way
    up -- as two calls or as the chunked relay -- and the combine+unpack) and its own copy
    streams out of a pool of three.  From step to step the gradients are scaled by another power of two
    (exact), so a phase that ran ahead of the data it depends on, or picked up the data of the
    step before, shows in the result."""
    import test_gpu_random as TR
    wl = TR.random_problem(rnd)
    if rnd.random() < 0.5:        # more and larger buckets
        wl = W.Workload("random_long", wl.config_id, [(rnd.choice([5000, 20000, 70001, 300000]),) for _ in range(rnd.randint(2, 5))],
                        wl.dtype, wl.group_of, wl.shares, bucket_cap_bytes=rnd.choice([40000, 400000, 1 << 40]))
    host, dev = H.device_gradients(wl)
    base = [[t.clone() for t in row] for row in dev]
    ctx = kt.kt_groups_init(wl.group_of, wl.shares, wl.G)
    kt.kt_bucket_pack(ctx, dev, wl.bucket_cap_bytes)
    plan = kt.kt_plan_query(ctx)
    n, nb = plan.transport_numel, plan.n_buckets
    rows = rnd.random() < 0.5
    def buffers(pinned=False):
        if rows:
            whole = torch.zeros(wl.G, n)
            return list(whole.pin_memory() if pinned else whole.cuda())
        return [torch.zeros(n).pin_memory() if pinned else torch.zeros(n, device="cuda") for _ in range(wl.G)]
    tr, pinned, recv = buffers(), buffers(True), buffers()
    out_dtype = rnd.choice([torch.float32, torch.bfloat16])
    out = [[torch.zeros(m, dtype=out_dtype, device="cuda") for m in wl.numel]]
    want, _, _, _ = H.run_oracle_path(oracle, wl, host, wl.shares, out_dtype={torch.float32: F32, torch.bfloat16: BF16}[out_dtype])
    main = torch.cuda.Stream()
    pool = [torch.cuda.Stream() for _ in range(3)]
    every, whole = list(range(nb)), [-1]
    snapshots = []
    torch.cuda.synchronize()
    for r in range(rounds):
        factor = float(2 ** rnd.randint(-4, 4))
        with torch.cuda.stream(main):
            for row, brow in zip(dev, base):           # this step's gradients: the seeded ones times a power of two
                for t, b in zip(row, brow):
                    torch.mul(b, factor, out=t)
        reduce_by, down_by, up_by, unpack_by = (rnd.choice([every, whole]) for _ in range(4))
        relay = rnd.random() < 0.4
        for b in reduce_by:
            kt.kt_hier_reduce(ctx, kt.KT_INTRA, tr, bucket=b, stream=main)
        if relay:
            a, c = rnd.sample(pool, 2)
            for b in down_by:
                kt.kt_relay_through_host(ctx, tr, pinned, recv, a, c, bucket=b, chunk_bytes=rnd.choice([256, 4096, 65536, 1 << 20]),
                                         main_stream=main)
            up_by = down_by
        else:
            for b in down_by:
                kt.kt_stage_to_host(ctx, kt.KT_D2H, tr, pinned, bucket=b, main_stream=main, side_stream=rnd.choice(pool))
            for b in up_by:
                kt.kt_stage_to_host(ctx, kt.KT_H2D, recv, pinned, bucket=b, main_stream=main, side_stream=rnd.choice(pool))
        for b in up_by:
            kt.kt_stage_wait(ctx, kt.KT_H2D, bucket=b, main_stream=main)
        for b in unpack_by:
            kt.kt_unpack_scale(ctx, recv, out, bucket=b, stream=main)
        with torch.cuda.stream(main):
            snapshots.append((factor, [t.clone() for t in out[0]]))
        if len(snapshots) >= 6 or r == rounds - 1:
            torch.cuda.synchronize()
            for factor, got in snapshots:
                for t in range(wl.T):
                    w = want[t]
                    if w.dtype == np.uint16:
                        w = oracle.f32_to_bf16(oracle.bf16_to_f32(w) * np.float32(factor))
                    else:
                        w = w * np.float32(factor)
                    H.assert_bit_equal(got[t], w, "step with factor %g, out[%d]" % (factor, t))
            snapshots = []
    kt.kt_destroy(ctx)


@pytest.mark.parametrize("seed", range(4))
def test_random_staging_granularities_and_streams(kt, oracle, seed):
    rnd = random.Random(8800 + seed)
    for _ in range(5):
        random_staging_traffic(kt, oracle, rnd, rounds=14)


# ------------------------------------------------------------------ error paths
def test_error_codes(kt):
    E = kt.KtError
    with pytest.raises(E) as e:
        kt.kt_groups_init([0, 2], [1, 1], 3)
    assert e.value.status == kt.KT_ERR_INVALID
    with pytest.raises(E):
        kt.kt_groups_init([0, 1], [1, 0])
    ctx = kt.kt_groups_init([0, 0, 1], [1, 2, 3])
    tr = [torch.empty(64, device="cuda") for _ in range(2)]
    with pytest.raises(E) as e:
        kt.kt_hier_reduce(ctx, kt.KT_INTRA, tr)
    assert e.value.status == kt.KT_ERR_STATE
    g = [[torch.zeros(100, device="cuda")] for _ in range(3)]
    kt.kt_bucket_pack(ctx, g, 1 << 20)
    plan = kt.kt_plan_query(ctx)
    assert plan.transport_numel == 128
    tr = [torch.empty(128, device="cuda") for _ in range(2)]
    with pytest.raises(E) as e:
        kt.kt_hier_reduce(ctx, kt.KT_INTRA, tr, bucket=1)
    assert e.value.status == kt.KT_ERR_SHAPE
    with pytest.raises(E) as e:
        kt.kt_hier_reduce(ctx, kt.KT_INTER, tr, None)
    assert e.value.status == kt.KT_ERR_INVALID
    with pytest.raises(E) as e:
        kt.kt_hier_reduce(ctx, 7, tr)
    assert e.value.status == kt.KT_ERR_INVALID
    odd = torch.empty(132, device="cuda")[1:129]
    with pytest.raises(E) as e:
        kt.kt_hier_reduce(ctx, kt.KT_INTRA, [odd, tr[1]])
    assert e.value.status == kt.KT_ERR_ALIGN
    with pytest.raises(E) as e:
        kt.kt_stage_wait(ctx, kt.KT_D2H)
    assert e.value.status == kt.KT_ERR_STATE
    with pytest.raises(E) as e:
        kt.kt_unpack_scale(ctx, tr, [[torch.empty(100, device="cuda")] for _ in range(4)])
    assert e.value.status == kt.KT_ERR_SHAPE
    assert "R = 4" in kt.kt_last_error()
    # the context stays usable after errors
    kt.kt_hier_reduce(ctx, kt.KT_INTRA, tr)
    torch.cuda.synchronize()
    assert kt.kt_launch_count(ctx) == 1
    kt.kt_destroy(ctx)
    kt.kt_destroy(ctx)      # idempotent


def test_stage_wait_deadline_returns_timeout_status(kt):
    """A wait whose deadline passes returns KT_ERR_TIMEOUT to the host and leaves the
    context usable; nothing on the device is interrupted."""
    n = 1 << 28                                   # 1 GiB per buffer: tens of milliseconds on the host link
    ctx = kt.kt_groups_init([0, 1], [1, 1])
    g = [[torch.zeros(n, device="cuda")] for _ in range(2)]
    kt.kt_bucket_pack(ctx, g, 1 << 62)
    tr = [torch.ones(n, device="cuda") for _ in range(2)]
    pinned = [torch.zeros(n).pin_memory() for _ in range(2)]
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    kt.kt_stage_to_host(ctx, kt.KT_D2H, tr, pinned, side_stream=side)
    with pytest.raises(kt.KtError) as e:
        kt.kt_stage_wait(ctx, kt.KT_D2H, timeout_ms=0)
    assert e.value.status == kt.KT_ERR_TIMEOUT
    kt.kt_stage_wait(ctx, kt.KT_D2H, timeout_ms=60000)    # now it completes
    assert float(pinned[1][-1]) == 1.0
    kt.kt_destroy(ctx)
