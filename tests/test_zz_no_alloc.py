"""The entry point that allocates nothing (kt_sync_flat_static).

Some users of this library cannot allocate device memory where gradients are synchronised:
code inside a framework's no-allocation region, plugins kept out of the host application's
memory pool, processes whose device memory is planned up front.  For them the library keeps
the scratch of the flat path in a fixed device array.  This test calls that entry point
through the C ABI twice in a row -- the second call with other sizes, groups and dtypes, so
that whatever the first call left in the shared array would show -- and checks each result
bit for bit against the CPU oracle on host copies of the same bytes and against the existing
route (kt_groups_init + kt_bucket_pack + kt_hier_reduce + kt_unpack_scale), the same bar as
the other GPU tests.  It also checks the property the entry point exists for: the device's
free memory is the same before and after the calls.  The file sorts last on purpose: a run
that stops at the first failure has then already run every other test.
"""
import pytest
import torch

from paper_2505_10183_b200 import workloads as W

import _harness as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def kt():
    if not torch.cuda.is_available():
        pytest.fail("this test needs a CUDA device")
    from paper_2505_10183_b200 import binding
    torch.cuda.set_device(0)
    return binding


def existing_route(kt, group_of, shares, grads, out_dtype, scale):
    ctx = kt.kt_groups_init(group_of, shares)
    kt.kt_bucket_pack(ctx, [[g] for g in grads], 1 << 62)
    n = kt.kt_plan_query(ctx).transport_numel
    transport = [torch.empty(n, device="cuda") for _ in range(max(group_of) + 1)]
    out = torch.empty(grads[0].numel(), dtype=out_dtype, device="cuda")
    kt.kt_hier_reduce(ctx, kt.KT_INTRA, transport)
    kt.kt_unpack_scale(ctx, transport, [[out]], scale=scale)
    torch.cuda.synchronize()
    kt.kt_destroy(ctx)
    return out


def make_grads(K, n, dtype, seed, misalign=0):
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    out = []
    for _ in range(K):
        buf = (torch.randn(n + misalign, generator=gen, device="cuda") * 1e-3).to(dtype)
        out.append(buf[misalign:])
    return out


def same_bits(a, b):
    view = torch.int32 if a.dtype == torch.float32 else torch.int16
    return torch.equal(a.view(view), b.view(view))


def oracle_result(oracle, c, grads):
    """The oracle's whole step on host copies of the very bytes the device holds."""
    dt = {torch.float32: 0, torch.bfloat16: 1}
    host = [[W.as_numpy(g)] for g in grads]
    out, _, _, _ = oracle.sync_step(host, [c["n"]], dt[c["dtype"]], c["group_of"], c["shares"],
                                    max(c["group_of"]) + 1, 1 << 62, c["scale"], dt[c["out_dtype"]])
    return out[0]


def test_static_scratch_entry_matches_oracle_and_existing_route_twice_in_a_row(kt, oracle):
    cases = [
        # first call: uneven shares, three groups, ragged length, fp32
        dict(group_of=[0, 0, 0, 1, 1, 2], shares=[40, 40, 29, 29, 19, 19], n=100_003, dtype=torch.float32,
             out_dtype=torch.float32, scale=1.0, misalign=0),
        # second call right behind it: other sizes and dtypes, element-aligned sources, bf16 out
        dict(group_of=[0, 1, 0, 1], shares=[79, 49, 79, 49], n=7_777, dtype=torch.bfloat16,
             out_dtype=torch.bfloat16, scale=0.5, misalign=1),
    ]
    inputs = [make_grads(len(c["group_of"]), c["n"], c["dtype"], 900 + i, c["misalign"]) for i, c in enumerate(cases)]
    outs = [torch.full((c["n"],), float("nan"), dtype=c["out_dtype"], device="cuda") for c in cases]
    third = torch.full((cases[0]["n"],), float("nan"), device="cuda")
    # One warm-up call per case before the free-memory reading: the first call on a device looks
    # up the scratch address, and the driver loads a kernel's code when it is first launched.
    for c, g, o in zip(cases, inputs, outs):
        kt.kt_sync_flat_static(c["group_of"], c["shares"], g, o, scale=c["scale"])
    torch.cuda.synchronize()
    for o in outs:
        o.fill_(float("nan"))
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for c, g, o in zip(cases, inputs, outs):          # back to back, no synchronisation between
        kt.kt_sync_flat_static(c["group_of"], c["shares"], g, o, scale=c["scale"])
    # and once more with the first case: the array now holds the second call's leftovers
    kt.kt_sync_flat_static(cases[0]["group_of"], cases[0]["shares"], inputs[0], third, scale=1.0)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before, "the calls changed the device's free memory"
    for c, g, o in zip(cases, inputs, outs):
        want = oracle_result(oracle, c, g)
        H.assert_bit_equal(o, want, "kt_sync_flat_static against the oracle")
        assert same_bits(o, existing_route(kt, c["group_of"], c["shares"], g, c["out_dtype"], c["scale"]))
    assert same_bits(third, outs[0])


def test_static_scratch_entry_rejects_what_does_not_fit(kt):
    n = kt.KT_STATIC_MAX_ELEMS // 2 + 64          # two groups of this size exceed the array
    g = [torch.zeros(n, device="cuda") for _ in range(2)]
    out = torch.zeros(n, device="cuda")
    with pytest.raises(kt.KtError) as e:
        kt.kt_sync_flat_static([0, 1], [1, 1], g, out)
    assert e.value.status == kt.KT_ERR_SHAPE
    assert "static scratch holds" in str(e.value)
    # the largest problem that fits is accepted
    n = kt.KT_STATIC_MAX_ELEMS // 2
    g = [torch.ones(n, device="cuda") for _ in range(2)]
    out = torch.zeros(n, device="cuda")
    kt.kt_sync_flat_static([0, 1], [1, 3], g, out)
    torch.cuda.synchronize()
    assert bool((out == 1.0).all())
    with pytest.raises(kt.KtError):
        kt.kt_sync_flat_static([0, 2], [1, 1], g, out)      # group 1 is empty


def drawn_static_calls(kt, oracle, rnd, calls):
    """`calls` drawn problems (rank counts, group layouts, shares, lengths around the tile and
    vector sizes, dtypes, element misalignment of sources and of the output, scales) through
    the entry point back to back on one stream, then each result against the oracle."""
    sizes = [1, 3, 7, 8, 9, 63, 64, 65, 511, 2047, 2048, 2049, 4095, 4096, 4097, 10000, 100003, 262144]
    todo = []
    for i in range(calls):
        K = rnd.randint(1, 16)
        G = rnd.randint(1, min(K, 4))
        group_of = list(range(G)) + [rnd.randrange(G) for _ in range(K - G)]
        rnd.shuffle(group_of)
        c = dict(group_of=group_of, shares=[rnd.randint(1, 200) for _ in range(K)], n=rnd.choice(sizes),
                 dtype=rnd.choice([torch.float32, torch.bfloat16]), out_dtype=rnd.choice([torch.float32, torch.bfloat16]),
                 scale=rnd.choice([1.0, 0.5, 1.0 / 3.0]), misalign=rnd.choice([0, 0, 1, 3]))
        if G * ((c["n"] + 63) // 64 * 64) > kt.KT_STATIC_MAX_ELEMS:
            c["n"] = 4097
        grads = make_grads(K, c["n"], c["dtype"], 5000 + i + rnd.randrange(1 << 20), c["misalign"])
        shift = rnd.choice([0, 0, 1, 2])
        out = torch.full((c["n"] + shift,), float("nan"), dtype=c["out_dtype"], device="cuda")[shift:]
        todo.append((c, grads, out))
    torch.cuda.synchronize()
    for c, grads, out in todo:
        kt.kt_sync_flat_static(c["group_of"], c["shares"], grads, out, scale=c["scale"])
    torch.cuda.synchronize()
    for c, grads, out in todo:
        H.assert_bit_equal(out, oracle_result(oracle, c, grads), "drawn call %r" % {k: v for k, v in c.items() if k != "shares"})


@pytest.mark.parametrize("seed", range(3))
def test_static_scratch_entry_on_drawn_problems(kt, oracle, seed):
    import random
    drawn_static_calls(kt, oracle, random.Random(1200 + seed), 20)
