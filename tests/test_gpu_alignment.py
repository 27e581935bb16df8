"""GPU parity with transport buffers at the least alignment the library accepts.

The header asks for 16-byte aligned transport, receive and combined buffers.  Kernels that move
eight floats per thread (bf16 gradients into an fp32 transport; an fp32 transport into bf16
outputs) use one 256-bit access when every base is 32-byte aligned and two 128-bit accesses
otherwise.  Allocators hand out 256-byte aligned memory, so the second form only runs when a
caller passes a view that starts 16 bytes into such a block: these tests do exactly that, for
both transport types and on every route, and compare with the oracle bit for bit.
"""
import random

import pytest
import torch

from paper_2505_10183_b200 import workloads as W

import _harness as H
import test_gpu_parity as P
import test_gpu_bf16_transport as B
import test_gpu_random as TR

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def kt():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    from paper_2505_10183_b200 import binding
    torch.cuda.set_device(0)
    return binding


def bf16(wl):
    wl.dtype = "bf16"
    return wl


def test_bf16_gradients_into_skewed_fp32_transport(kt, oracle):
    """Eight floats per thread are stored to the transport: the store side of the narrow form."""
    P.compare_all(kt, oracle, bf16(W.tiny()), skew16=True)
    P.compare_all(kt, oracle, bf16(W.tiny()), skew16=True, out_dtype=torch.float32, R=2, scale=0.5)
    P.compare_all(kt, oracle, W.sweep_point(4, 16 << 20, "bf16"), skew16=True)
    P.compare_all(kt, oracle, W.resnet50(), skew16=True, per_bucket=True)


def test_skewed_fp32_transport_into_bf16_outputs(kt, oracle):
    """Eight floats per thread are loaded from the transport: the load side of the narrow form."""
    P.compare_all(kt, oracle, W.tiny(), skew16=True, out_dtype=torch.bfloat16)
    P.compare_all(kt, oracle, W.sweep_point(4, 16 << 20, "f32"), skew16=True, out_dtype=torch.bfloat16)
    P.compare_all(kt, oracle, W.mobilenet_v2(), skew16=True, out_dtype=torch.bfloat16, R=2)
    # through the relay: the receive buffers, which the combine reads, are skewed as well
    P.compare_all(kt, oracle, W.resnet18(), skew16=True, out_dtype=torch.bfloat16, staged="relay_all")
    P.compare_all(kt, oracle, W.tiny(), skew16=True, out_dtype=torch.bfloat16, staged=True, per_bucket=True)


def test_skewed_bf16_transport(kt, oracle):
    """The narrow transport at 16-byte alignment, all four gradient / output type pairs."""
    for wl in (W.tiny(), bf16(W.tiny()), W.sweep_point(4, 16 << 20, "bf16"), W.sweep_point(2, 16 << 20, "f32")):
        for odt in (torch.float32, torch.bfloat16):
            B.compare(kt, oracle, wl, skew16=True, out_dtype=odt)


def test_combined_buffer_route_with_skewed_transport(kt, oracle):
    P.compare_all(kt, oracle, bf16(W.tiny()), skew16=True, use_combined=True, out_dtype=torch.bfloat16)


@pytest.mark.parametrize("seed", range(2))
def test_random_ragged_lists_with_skewed_transport(kt, oracle, seed):
    rnd = random.Random(4100 + seed)
    for _ in range(20):
        wl = TR.random_problem(rnd)
        out_dtype = rnd.choice([torch.float32, torch.bfloat16])
        kw = dict(out_dtype=out_dtype, R=rnd.randint(1, min(3, wl.K)), scale=rnd.choice([1.0, 1.0 / 3.0]), skew16=True)
        route = rnd.choice(["fused", "buckets", "relay", "staged_buckets"])
        if route == "buckets":
            kw["per_bucket"] = True
        elif route == "relay":
            kw.update(staged=rnd.choice(["relay", "relay_all"]), relay_chunk=rnd.choice([256, 65536, 1 << 22]))
        elif route == "staged_buckets":
            kw.update(staged=True, per_bucket=True)
        if rnd.random() < 0.3:
            B.compare(kt, oracle, wl, shares=wl.shares, **kw)
        else:
            wl_shares = wl.shares
            host, dev = H.device_gradients(wl, misalign=rnd.choice([0, 0, 1, 3]))
            out, transport, plan, ctx = H.run_gpu_path(kt, wl, dev, wl_shares, **kw)
            odt = {torch.float32: 0, torch.bfloat16: 1}[out_dtype]
            o_out, o_parts, _, _ = H.run_oracle_path(oracle, wl, host, wl_shares, out_dtype=odt, scale=kw["scale"])
            for g in range(wl.G):
                assert transport[g].data_ptr() % 32 == 16
                H.assert_bit_equal(transport[g], o_parts[g], "transport[%d]" % g)
            for c in range(len(out)):
                for t in range(wl.T):
                    H.assert_bit_equal(out[c][t], o_out[t], "out[%d][%d]" % (c, t))
            kt.kt_destroy(ctx)
