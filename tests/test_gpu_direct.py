"""GPU parity of the direct route (kt_sync_direct: reduce, combine, scale, cast and unpack in
one pass, no transport buffers) against the CPU oracle, bit for bit: the kernel keeps the
oracle's operation order (group partials first, then the combine), so nothing may differ."""
import random

import numpy as np
import pytest
import torch

from paper_2505_10183_b200 import workloads as W

import _harness as H

pytestmark = pytest.mark.gpu

F32, BF16 = 0, 1
ODT = {torch.float32: F32, torch.bfloat16: BF16}


@pytest.fixture(scope="module")
def kt():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    from paper_2505_10183_b200 import binding
    torch.cuda.set_device(0)
    return binding


def guarded(numel, dtype, shift=0, guard=64):
    """A tensor of `numel` elements inside a larger allocation filled with a pattern; shift > 0
    moves it off the 16-byte boundary."""
    buf = torch.full((numel + 2 * guard + shift,), -777.0, dtype=dtype, device="cuda")
    return buf, buf[guard + shift:guard + shift + numel]


def run_direct(kt, oracle, wl, shares, host, dev, out_dtype=None, R=1, scale=1.0, per_bucket=False,
               out_shift=None):
    odt = H.TORCH_DT[wl.dtype] if out_dtype is None else out_dtype
    ctx = kt.kt_groups_init(wl.group_of, shares, wl.G)
    kt.kt_bucket_pack(ctx, dev, wl.bucket_cap_bytes)
    plan = kt.kt_plan_query(ctx)
    bufs, out = [], []
    for c in range(R):
        row = []
        for t, m in enumerate(wl.numel):
            b, v = guarded(m, odt, 0 if out_shift is None else out_shift(c, t))
            bufs.append((b, v))
            row.append(v)
        out.append(row)
    before = kt.kt_launch_count(ctx)
    for b in (range(plan.n_buckets) if per_bucket else [-1]):
        kt.kt_sync_direct(ctx, out, scale=scale, bucket=b)
    torch.cuda.synchronize()
    launched = kt.kt_launch_count(ctx) - before
    want, _, _, _ = oracle.sync_step(host, wl.numel, H.ORACLE_DT[wl.dtype], wl.group_of, shares, wl.G,
                                     wl.bucket_cap_bytes, scale, ODT[odt])
    for c in range(R):
        for t in range(wl.T):
            H.assert_bit_equal(out[c][t], want[t], "%s out[%d][%d]" % (wl.name, c, t))
    for b, v in bufs:       # nothing written outside the tensors
        lo = v.data_ptr() - b.data_ptr()
        lo //= b.element_size()
        assert bool((b[:lo] == -777.0).all()) and bool((b[lo + v.numel():] == -777.0).all())
    kt.kt_destroy(ctx)
    return out, launched


@pytest.mark.parametrize("name", ["tiny", "resnet18", "resnet50", "mobilenet_v2"])
def test_named_configurations(kt, oracle, name):
    wl = W.by_name(name)
    shares = H.shares_of(wl, kt)
    host, dev = H.device_gradients(wl)
    out, launched = run_direct(kt, oracle, wl, shares, host, dev)
    assert launched == 1
    # the stated tolerance against the fp64 weighted mean on top of the bit-for-bit check
    F, absF = oracle.flat_reduce_f64([np.concatenate(h) for h in host], H.ORACLE_DT[wl.dtype], shares)
    got = np.concatenate([W.as_numpy(t) for t in out[0]])
    tol = 1e-6
    if got.dtype == np.uint16:
        got, tol = oracle.bf16_to_f32(got), 1e-2
    nz = absF > 0
    assert np.max(np.abs(got[nz] - F[nz]) / absF[nz]) <= tol
    # bucket by bucket, several copies, a scale that is not a power of two
    run_direct(kt, oracle, wl, shares, host, dev, per_bucket=True, R=2, scale=1.0 / 3.0)


def test_matches_the_two_kernel_route_with_mixed_dtypes(kt, oracle):
    """fp32 gradients to bf16 outputs and bf16 gradients to fp32 outputs."""
    for wl, odt in ((W.mobilenet_v2(), torch.bfloat16), (W.sweep_point(8, 3 << 20, "bf16"), torch.float32)):
        shares = H.shares_of(wl, kt)
        host, dev = H.device_gradients(wl)
        run_direct(kt, oracle, wl, shares, host, dev, out_dtype=odt, scale=0.5)


def test_one_homogeneous_group_and_singletons(kt, oracle):
    """G = 1 (the homogeneous dispatch proper), K = 1, and every rank its own group."""
    base = W.tiny()
    for group_of, shares in (([0, 0, 0, 0], [5, 7, 11, 13]), ([0], [3]), ([0, 1, 2, 3], [1, 2, 3, 4])):
        wl = W.Workload("direct_groups", 7, base.shapes, "f32", group_of, shares)
        host, dev = H.device_gradients(wl)
        run_direct(kt, oracle, wl, shares, host, dev)


@pytest.mark.parametrize("seed", range(4))
def test_random_problems_misaligned_inputs_and_outputs(kt, oracle, seed):
    import test_gpu_random as TR
    rnd = random.Random(5000 + seed)
    for _ in range(25):
        wl = TR.random_problem(rnd)
        tdt = H.TORCH_DT[wl.dtype]
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
        shifts = {}
        run_direct(kt, oracle, wl, wl.shares, host, dev,
                   out_dtype=rnd.choice([torch.float32, torch.bfloat16]), R=rnd.randint(1, min(3, wl.K)),
                   scale=rnd.choice([1.0, 0.5, 1.0 / 3.0, 1.0 / sum(wl.shares)]),
                   per_bucket=rnd.random() < 0.5,
                   out_shift=lambda c, t: shifts.setdefault((c, t), rnd.choice([0, 0, 1, 2, 3, 4])))


@pytest.mark.parametrize("name,dtype", [("tiny", "f32"), ("mobilenet_v2", "f32"), ("resnet50", "bf16"), ("tiny", "bf16")])
def test_all_reduce_in_place(kt, oracle, name, dtype):
    """The outputs are the registered gradient tensors themselves: every rank's tensors are
    overwritten with the reduced gradient (R = K), and, in a second problem, only rank 1's
    (R = 1), the other ranks keeping their inputs.  Misaligned tensors included."""
    for R_all in (True, False):
        wl = W.by_name(name)
        wl.dtype = dtype
        shares = H.shares_of(wl, kt)
        host, dev = H.device_gradients(wl, misalign=0 if R_all else 3)
        ctx = kt.kt_groups_init(wl.group_of, shares, wl.G)
        kt.kt_bucket_pack(ctx, dev, wl.bucket_cap_bytes)
        out = dev if R_all else [dev[1]]
        kt.kt_sync_direct(ctx, out, scale=0.5)
        torch.cuda.synchronize()
        want, _, _, _ = H.run_oracle_path(oracle, wl, host, shares, scale=0.5)
        for r in range(wl.K):
            for t in range(wl.T):
                if R_all or r == 1:
                    H.assert_bit_equal(dev[r][t], want[t], "rank %d tensor %d" % (r, t))
                else:
                    H.assert_bit_equal(dev[r][t], host[r][t], "untouched rank %d tensor %d" % (r, t))
        kt.kt_destroy(ctx)


def test_error_codes(kt):
    wl = W.tiny()
    _, dev = H.device_gradients(wl)
    ctx = kt.kt_groups_init(wl.group_of, wl.shares, wl.G)
    out = [[torch.empty_like(t) for t in dev[0]]]
    with pytest.raises(kt.KtError) as e:          # before the plan exists
        kt.kt_sync_direct(ctx, kt.kt_ptrs([]), R=1, out_dtype=kt.KT_F32)
    assert e.value.status == kt.KT_ERR_STATE
    kt.kt_bucket_pack(ctx, dev, wl.bucket_cap_bytes)
    with pytest.raises(kt.KtError) as e:
        kt.kt_sync_direct(ctx, out, bucket=5)
    assert e.value.status == kt.KT_ERR_SHAPE
    with pytest.raises(kt.KtError) as e:
        kt.kt_sync_direct(ctx, kt.kt_ptrs(out[0]), R=wl.K + 1, out_dtype=kt.KT_F32)
    assert e.value.status == kt.KT_ERR_SHAPE
    kt.kt_destroy(ctx)


def test_allreduce_in_one_call_takes_the_route_the_groups_call_for(kt, oracle):
    """kt_allreduce: one group -> the direct kernel (1 launch, no buffers); several groups ->
    reduce, relay through pinned host memory, combine + unpack (2 launches); both equal the
    oracle bit for bit, twice in a row."""
    for wl in (W.Workload("one_group", 9, W.tiny().shapes, "f32", [0, 0, 0], [3, 2, 1]), W.tiny(), W.mobilenet_v2(),
               W.resnet18()):
        shares = H.shares_of(wl, kt)
        host, dev = H.device_gradients(wl)
        ctx = kt.kt_groups_init(wl.group_of, shares, wl.G)
        kt.kt_bucket_pack(ctx, dev, wl.bucket_cap_bytes)
        n = kt.kt_plan_query(ctx).transport_numel
        out = [[torch.full((m,), float("nan"), dtype=H.TORCH_DT[wl.dtype], device="cuda") for m in wl.numel]]
        kw = {}
        if wl.G > 1:
            kw = dict(transport=list(torch.full((wl.G, n), float("nan"), device="cuda")),
                      host_pinned=list(torch.zeros(wl.G, n).pin_memory()),
                      recv=list(torch.full((wl.G, n), float("nan"), device="cuda")),
                      d2h_stream=torch.cuda.Stream(), h2d_stream=torch.cuda.Stream())
        before = kt.kt_launch_count(ctx)
        kt.kt_allreduce(ctx, out, scale=0.5, **kw)
        kt.kt_allreduce(ctx, out, scale=0.5, **kw)
        torch.cuda.synchronize()
        assert kt.kt_launch_count(ctx) - before == (2 if wl.G == 1 else 4)
        want, parts, _, _ = H.run_oracle_path(oracle, wl, host, shares, scale=0.5)
        for t in range(wl.T):
            H.assert_bit_equal(out[0][t], want[t], "%s out[%d]" % (wl.name, t))
        if wl.G > 1:
            for g in range(wl.G):
                H.assert_bit_equal(kw["recv"][g], parts[g], "recv[%d]" % g)
            with pytest.raises(kt.KtError):
                kt.kt_allreduce(ctx, out)             # buffers are required with several groups
        kt.kt_destroy(ctx)
