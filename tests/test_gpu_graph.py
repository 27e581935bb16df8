"""The recorded step (kt_graph_begin / kt_graph_end / kt_graph_launch): one submission replays
the fused reduce, the relay through pinned host memory and the combine+unpack.  Replays must
give the oracle's result bit for bit, on the data that is in the buffers at replay time."""
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


def check(kt, oracle, wl, host, out, shares):
    want, _, _, _ = H.run_oracle_path(oracle, wl, host, shares)
    for t in range(wl.T):
        H.assert_bit_equal(out[0][t], want[t], "%s out[%d]" % (wl.name, t))


@pytest.mark.parametrize("name", ["tiny", "mobilenet_v2", "resnet18"])
def test_recorded_step_replays_on_live_data(kt, oracle, name):
    import bench
    wl = W.by_name(name)
    prob = bench.Problem(wl, kt, device_values=False)
    host = [[W.as_numpy(t) for t in W.split_tensors(W.rank_gradients(wl, r, "cpu"), wl.numel)] for r in range(wl.K)]
    with torch.cuda.stream(prob.main):
        prob.step()                                   # uploads tables, creates events
        torch.cuda.synchronize()
        kt.kt_graph_begin(prob.ctx, prob.main)
        before = kt.kt_launch_count(prob.ctx)
        prob.step()
        graph = kt.kt_graph_end(prob.ctx, prob.main)
        assert kt.kt_launch_count(prob.ctx) - before == 2
        assert kt.kt_graph_nodes(graph) >= 2
        for t in prob.out[0]:
            t.fill_(float("nan"))                     # recording must not have run anything
        torch.cuda.synchronize()
        kt.kt_graph_launch(graph, prob.main)
        torch.cuda.synchronize()
        check(kt, oracle, wl, host, prob.out, prob.shares)
        # new gradient values in the same buffers: the replay reads what is there now
        for r in range(wl.K):
            for t in prob.grads[r]:
                t.mul_(-2.0 if r == 0 else 0.5)
        host2 = [[(h * np.float32(-2.0 if r == 0 else 0.5)) for h in host[r]] for r in range(wl.K)]
        kt.kt_graph_launch(graph, prob.main)
        kt.kt_graph_launch(graph, prob.main)
        torch.cuda.synchronize()
        check(kt, oracle, wl, host2, prob.out, prob.shares)
    kt.kt_graph_destroy(graph)
    kt.kt_destroy(prob.ctx)


def test_recording_a_sequence_that_cannot_be_recorded_reports_an_error(kt):
    """A first-ever kt_unpack_scale has to upload its destination table, which a recording
    cannot hold: the recording ends with an error status, the context stays usable."""
    import bench
    wl = W.tiny()
    prob = bench.Problem(wl, kt, device_values=False)
    with torch.cuda.stream(prob.main):
        kt.kt_hier_reduce(prob.ctx, kt.KT_INTRA, prob.transport, stream=prob.main)
        torch.cuda.synchronize()
        kt.kt_graph_begin(prob.ctx, prob.main)
        with pytest.raises(kt.KtError) as e:
            prob.step()
        assert e.value.status == kt.KT_ERR_STATE
        with pytest.raises(kt.KtError) as e:
            kt.kt_graph_end(prob.ctx, prob.main)
        assert e.value.status == kt.KT_ERR_STATE
        torch.cuda.synchronize()
        prob.step()                                   # eager execution still works
        torch.cuda.synchronize()
    assert bool(torch.isfinite(prob.out[0][0]).all())
    kt.kt_destroy(prob.ctx)


@pytest.mark.parametrize("name", ["tiny", "mobilenet_v2"])
def test_alternating_output_sets_eager_and_recorded(kt, oracle, name):
    """Double-buffered gradients: the caller alternates between two sets of output tensors (and
    a third route, the one-pass kernel, between two more).  Each set's destination table stays
    on the device, so alternating needs no new upload, each set can be part of a recording,
    and every result equals the oracle's bit for bit."""
    wl = W.by_name(name)
    shares = H.shares_of(wl, kt)
    host, dev = H.device_gradients(wl)
    ctx = kt.kt_groups_init(wl.group_of, shares, wl.G)
    kt.kt_bucket_pack(ctx, dev, wl.bucket_cap_bytes)
    n = kt.kt_plan_query(ctx).transport_numel
    transport = [torch.full((n,), float("nan"), device="cuda") for _ in range(wl.G)]
    sets = [[[torch.full((m,), float("nan"), device="cuda") for m in wl.numel]] for _ in range(4)]
    want, _, _, _ = H.run_oracle_path(oracle, wl, host, shares)
    main = torch.cuda.Stream()

    def run(i):
        if i < 2:
            kt.kt_hier_reduce(ctx, kt.KT_INTRA, transport, stream=main)
            kt.kt_unpack_scale(ctx, transport, sets[i], stream=main)
        else:
            kt.kt_sync_direct(ctx, sets[i], stream=main)

    def check(i, what):
        torch.cuda.synchronize()
        for t in range(wl.T):
            H.assert_bit_equal(sets[i][0][t], want[t], "%s: set %d out[%d]" % (what, i, t))
            sets[i][0][t].fill_(float("nan"))
        torch.cuda.synchronize()

    with torch.cuda.stream(main):
        for step in range(12):                       # back to back, no synchronisation between
            run(step % 4)
        for i in range(4):
            check(i, "eager")
        graphs = []
        for i in range(4):                           # every set is already on the device: recordable
            kt.kt_graph_begin(ctx, main)
            run(i)
            graphs.append(kt.kt_graph_end(ctx, main))
        for step in range(8):
            kt.kt_graph_launch(graphs[step % 4], main)
        for i in range(4):
            check(i, "recorded")
        # tables held by recordings are never replaced: five more sets share the remaining
        # tables in turn, and the recorded ones still replay correctly afterwards
        extra = [[[torch.full((m,), float("nan"), device="cuda") for m in wl.numel]] for _ in range(5)]
        for step in range(15):
            kt.kt_sync_direct(ctx, extra[step % 5], stream=main)
        torch.cuda.synchronize()
        for x in extra:
            for t in range(wl.T):
                H.assert_bit_equal(x[0][t], want[t], "churned set out[%d]" % t)
        kt.kt_graph_launch(graphs[0], main)
        kt.kt_graph_launch(graphs[3], main)
        check(0, "recorded, after other sets came and went")
        check(3, "recorded, after other sets came and went")
        # once every table is held by a recording, a new set is refused with a clear status
        for i in range(4):
            kt.kt_sync_direct(ctx, extra[i], stream=main)
            kt.kt_graph_begin(ctx, main)
            kt.kt_sync_direct(ctx, extra[i], stream=main)
            graphs.append(kt.kt_graph_end(ctx, main))
        with pytest.raises(kt.KtError) as e:
            kt.kt_sync_direct(ctx, extra[4], stream=main)
        assert e.value.status == kt.KT_ERR_STATE and "held by recorded steps" in str(e.value)
        kt.kt_bucket_pack(ctx, dev, wl.bucket_cap_bytes)      # a new plan releases them
        kt.kt_sync_direct(ctx, extra[4], stream=main)
        torch.cuda.synchronize()
        for t in range(wl.T):
            H.assert_bit_equal(extra[4][0][t], want[t], "after re-planning out[%d]" % t)
    for g in graphs:
        kt.kt_graph_destroy(g)
    kt.kt_destroy(ctx)


def test_destination_table_uploaded_on_one_stream_is_safe_to_use_on_another(kt, oracle):
    """A set of output tensors is first seen by a call on stream A, whose queue is long (the
    upload of its destination table sits behind a large fill); a call on stream B uses the same
    set right away.  B's kernel must wait for that upload, not for the rest of A."""
    wl = W.mobilenet_v2()
    shares = H.shares_of(wl, kt)
    host, dev = H.device_gradients(wl)
    ctx = kt.kt_groups_init(wl.group_of, shares, wl.G)
    kt.kt_bucket_pack(ctx, dev, wl.bucket_cap_bytes)
    n = kt.kt_plan_query(ctx).transport_numel
    transport = [torch.full((n,), float("nan"), device="cuda") for _ in range(wl.G)]
    out = [[torch.full((m,), float("nan"), device="cuda") for m in wl.numel]]
    want, _, _, _ = H.run_oracle_path(oracle, wl, host, shares)
    A, B = torch.cuda.Stream(), torch.cuda.Stream()
    ballast = torch.empty(2 << 30, dtype=torch.uint8, device="cuda")
    kt.kt_hier_reduce(ctx, kt.KT_INTRA, transport, stream=A)
    reduced = torch.cuda.Event()
    reduced.record(A)
    with torch.cuda.stream(A):
        for _ in range(4):
            ballast.fill_(1)                                    # A is busy for a while
    kt.kt_unpack_scale(ctx, transport, out, stream=A)           # first use of the set: upload queued on A
    B.wait_event(reduced)
    kt.kt_unpack_scale(ctx, transport, out, scale=1.0, stream=B)   # same set, other stream
    B.synchronize()
    for t in range(wl.T):
        H.assert_bit_equal(out[0][t], want[t], "out[%d] written from stream B" % t)
    torch.cuda.synchronize()
    kt.kt_destroy(ctx)


def random_table_traffic(kt, oracle, rnd, bursts):
    """Random traffic over a context's destination tables: more sets of output tensors than the
    context keeps tables for, written by the combine+unpack, by the one-pass kernel and by
    replayed recordings, on three streams, in bursts without any synchronisation inside a burst
    (so tables are replaced while kernels that read their neighbours are still queued), with new
    recordings, destroyed recordings and new plans in between.  After every burst each targeted
    set must hold the oracle's result and every other set must be untouched."""
    import test_gpu_random as TR
    wl = TR.random_problem(rnd)
    host, dev = H.device_gradients(wl, misalign=rnd.choice([0, 0, 1, 3]))
    ctx = kt.kt_groups_init(wl.group_of, wl.shares, wl.G)
    kt.kt_bucket_pack(ctx, dev, wl.bucket_cap_bytes)
    n = kt.kt_plan_query(ctx).transport_numel
    transport = [torch.full((n,), float("nan"), device="cuda") for _ in range(wl.G)]
    streams = [torch.cuda.Stream() for _ in range(3)]
    kt.kt_hier_reduce(ctx, kt.KT_INTRA, transport, stream=streams[0])
    torch.cuda.synchronize()
    scales = [1.0, 1.0 / 3.0]
    want = {}
    for code, dt in ((0, torch.float32), (1, torch.bfloat16)):
        for s in scales:
            want[dt, s] = H.run_oracle_path(oracle, wl, host, wl.shares, out_dtype=code, scale=s)[0]
    n_sets = 14
    sets = []
    for _ in range(n_sets):
        dt, R = rnd.choice([torch.float32, torch.bfloat16]), rnd.randint(1, min(2, wl.K))
        sets.append(dict(dtype=dt, tensors=[[torch.full((m,), float("nan"), dtype=dt, device="cuda") for m in wl.numel]
                                            for _ in range(R)]))
    graphs = []                                      # (graph, set index, scale)
    recorded_sets = set()

    def launch(i, scale, stream, one_pass):
        if one_pass:
            kt.kt_sync_direct(ctx, sets[i]["tensors"], scale=scale, stream=stream)
        else:
            kt.kt_unpack_scale(ctx, transport, sets[i]["tensors"], scale=scale, stream=stream)

    def verify(written):
        torch.cuda.synchronize()
        for i, st in enumerate(sets):
            for copy in st["tensors"]:
                for t in range(wl.T):
                    if i in written:
                        H.assert_bit_equal(copy[t], want[st["dtype"], written[i]][t], "set %d out[%d]" % (i, t))
                        copy[t].fill_(float("nan"))
                    else:
                        assert bool(torch.isnan(copy[t].float()).all()), "set %d was written by a call for another set" % i
        torch.cuda.synchronize()

    for _ in range(bursts):
        move = rnd.random()
        if move < 0.12 and len(recorded_sets) < 6:
            # a new recording: the set must have been used once, outside a recording
            i, scale, one_pass, s = rnd.randrange(n_sets), rnd.choice(scales), rnd.random() < 0.5, rnd.choice(streams)
            launch(i, scale, s, one_pass)
            verify({i: scale})
            kt.kt_graph_begin(ctx, s)
            launch(i, scale, s, one_pass)
            graphs.append((kt.kt_graph_end(ctx, s), i, scale))
            recorded_sets.add(i)
            verify({})                               # recording runs nothing
        elif move < 0.16 and graphs:
            g, _, _ = graphs.pop(rnd.randrange(len(graphs)))
            torch.cuda.synchronize()
            kt.kt_graph_destroy(g)
        elif move < 0.19:
            # a new plan: recordings are void (destroyed first), every table is free again
            torch.cuda.synchronize()
            for g, _, _ in graphs:
                kt.kt_graph_destroy(g)
            graphs, recorded_sets = [], set()
            kt.kt_bucket_pack(ctx, dev, wl.bucket_cap_bytes)
        else:
            written = {}
            for _ in range(rnd.randint(1, 7)):
                s = rnd.choice(streams)
                if graphs and rnd.random() < 0.3:
                    g, i, scale = rnd.choice(graphs)
                    if i in written:
                        continue
                    kt.kt_graph_launch(g, s)
                else:
                    i, scale = rnd.randrange(n_sets), rnd.choice(scales)
                    if i in written:
                        continue
                    launch(i, scale, s, rnd.random() < 0.5)
                written[i] = scale
            verify(written)
    torch.cuda.synchronize()
    for g, _, _ in graphs:
        kt.kt_graph_destroy(g)
    kt.kt_destroy(ctx)


@pytest.mark.parametrize("seed", range(4))
def test_random_traffic_over_the_destination_tables(kt, oracle, seed):
    import random
    rnd = random.Random(4100 + seed)
    for _ in range(3):
        random_table_traffic(kt, oracle, rnd, bursts=40)
