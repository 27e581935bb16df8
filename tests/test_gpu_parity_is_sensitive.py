"""The parity comparison must notice a difference of one rounding.

The GPU tests call the CUDA path correct when it equals the oracle bit for bit.  That means
something only if the comparison would fail for a path that computes almost the same: a chain
that rounds twice where it should round once, an order of summation turned round, a narrowing
that breaks ties the other way, padding that is not zero.  Each case plants one such mistake in
a temporary copy of the ORACLE (on the CPU; the CUDA path runs unchanged) and requires the same
comparison the parity tests use to report a mismatch on a named workload, while the unchanged
oracle still matches.
"""
import numpy as np
import pytest
import torch

import _harness as H
from _planted import load_oracle_copy, write_oracle_copy
from paper_2505_10183_b200 import workloads as W

pytestmark = pytest.mark.gpu

F32, BF16 = 0, 1
SHARES = [37, 41, 43, 47, 23, 31, 17, 17]

# (name, text in the oracle, replacement, output dtype of the run that has to show it)
ONE_ROUNDING_AWAY = [
    ("in-group terms as multiply then add", "acc = fmaf(a[r], x, acc);", "acc = acc + a[r] * x;", torch.float32),
    ("ranks of a group in descending order",
     "for (int r = 0; r < K; ++r) {\n                    if (group_of[r] != g)",
     "for (int r = K - 1; r >= 0; --r) {\n                    if (group_of[r] != g)", torch.float32),
    ("groups combined as multiply then add", "acc = fmaf(W[g], partials[g][i], acc);",
     "acc = acc + W[g] * partials[g][i];", torch.float32),
    ("groups combined in descending order",
     "float acc = W[0] * partials[0][i];\n        for (int g = 1; g < G; ++g)\n            acc = fmaf(W[g], partials[g][i], acc);",
     "float acc = W[G - 1] * partials[G - 1][i];\n        for (int g = G - 2; g >= 0; --g)\n            acc = fmaf(W[g], partials[g][i], acc);",
     torch.float32),
    ("scale as a division by the reciprocal", "float y = S[tensor_offset[t] + j] * scale;",
     "float y = S[tensor_offset[t] + j] / (1.0f / scale);", torch.float32),
    ("padding of the partials not zero", "P[i] = 0.0f;", "P[i] = -0.0f;", torch.float32),
    ("narrowing breaks ties away from zero", "u += 0x7FFFu + lsb;", "u += 0x8000u;", torch.bfloat16),
    ("narrowing truncates", "u += 0x7FFFu + lsb;", "u += 0u;", torch.bfloat16),
]


@pytest.fixture(scope="module")
def kt():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    from paper_2505_10183_b200 import binding
    torch.cuda.set_device(0)
    return binding


@pytest.fixture(scope="module")
def device_results(kt):
    """MobileNetV2's tensor list (8 ranks in groups of 4 + 2 + 2), with shares that differ inside
    every group -- the configuration's own shares give in-group weights of 1/4 and 1/2, with
    which every product is exact and a chain cannot show how it rounds -- and scale 1/3 so that
    the last multiply rounds too; once with fp32 and once with bf16 outputs."""
    wl = W.mobilenet_v2()
    shares = SHARES
    host, dev = H.device_gradients(wl)
    runs = {}
    for odt in (torch.float32, torch.bfloat16):
        out, transport, plan, ctx = H.run_gpu_path(kt, wl, dev, shares, out_dtype=odt, scale=1.0 / 3.0)
        runs[odt] = ([W.as_numpy(t) for t in out[0]], [W.as_numpy(t) for t in transport])
        kt.kt_destroy(ctx)
    return wl, shares, host, runs


def mismatches(oracle_module, wl, shares, host, run, out_dtype):
    """Elements (partials incl. padding, then outputs) in which the device run and this oracle
    differ: the quantity every parity test requires to be zero."""
    got_out, got_parts = run
    o_out, o_parts, _, _ = H.run_oracle_path(oracle_module, wl, host, shares, scale=1.0 / 3.0,
                                             out_dtype={torch.float32: F32, torch.bfloat16: BF16}[out_dtype])
    bad = 0
    for g in range(wl.G):
        bad += int(np.count_nonzero(H.bits(got_parts[g]) != H.bits(o_parts[g])))
    for t in range(wl.T):
        bad += int(np.count_nonzero(H.bits(got_out[t]) != H.bits(o_out[t])))
    return bad


def test_unchanged_oracle_matches(oracle, device_results):
    wl, shares, host, runs = device_results
    for odt, run in runs.items():
        assert mismatches(oracle, wl, shares, host, run, odt) == 0


@pytest.mark.parametrize("case", ONE_ROUNDING_AWAY, ids=[c[0] for c in ONE_ROUNDING_AWAY])
def test_comparison_reports_an_oracle_that_is_one_rounding_away(case, device_results, tmp_path):
    name, old, new, odt = case
    wl, shares, host, runs = device_results
    folder = str(tmp_path / "oracle_copy")
    write_oracle_copy(folder, name, old, new)
    wrong = load_oracle_copy(folder, "kt_oracle_planted_%d" % ONE_ROUNDING_AWAY.index(case))
    bad = mismatches(wrong, wl, shares, host, runs[odt], odt)
    assert bad > 0, "the comparison cannot tell the CUDA path from an oracle with: " + name
