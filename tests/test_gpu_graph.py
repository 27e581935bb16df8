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
        with pytest.raises(kt.KtError):
            prob.step()
        with pytest.raises(kt.KtError) as e:
            kt.kt_graph_end(prob.ctx, prob.main)
        assert e.value.status == kt.KT_ERR_CUDA
        torch.cuda.synchronize()
        prob.step()                                   # eager execution still works
        torch.cuda.synchronize()
    assert bool(torch.isfinite(prob.out[0][0]).all())
    kt.kt_destroy(prob.ctx)
