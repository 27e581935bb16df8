"""Pins for the oracle's data path: bucket plan, pack/unpack, casts, the two-level
weighted reduce.  Each check compares the oracle with something that is not the oracle:
exact rational arithmetic on tiny inputs, numpy fp64 means, torch's bf16 cast, closed
forms and structural invariants."""
import random
from fractions import Fraction

import numpy as np
import pytest
import torch

from paper_2505_10183_b200 import workloads as W

F32, BF16 = 0, 1
MIB = 1 << 20


# ------------------------------------------------------------------ bucket plan
def check_plan_invariants(numel, cap_bytes, plan):
    cap = cap_bytes // 4
    T = len(numel)
    off = plan.tensor_offset.tolist()
    bof = plan.bucket_of.tolist()
    # reverse list order: the last tensor sits first in the transport
    order = list(range(T - 1, -1, -1))
    assert off[order[0]] == 0 and bof[order[0]] == 0
    end_prev, b_prev = 0, 0
    for k, t in enumerate(order):
        assert off[t] % 8 == 0
        assert off[t] >= end_prev                      # no overlap, order kept
        if bof[t] == b_prev:
            assert off[t] - end_prev < 8               # minimal padding inside a bucket
        else:
            assert bof[t] == b_prev + 1                # buckets are consecutive
            assert off[t] % 64 == 0 and off[t] - end_prev < 64
            assert off[t] == plan.bucket_start[bof[t]]
            # greedy: the tensor did not fit into the previous bucket
            prev_start = plan.bucket_start[b_prev]
            assert (-(-end_prev // 8) * 8 - prev_start) + numel[t] > cap
        end_prev, b_prev = off[t] + numel[t], bof[t]
    assert plan.n_buckets == b_prev + 1
    assert plan.transport_numel % 64 == 0 and 0 <= plan.transport_numel - end_prev < 64
    # cap respected unless a bucket holds one oversized tensor
    for b in range(plan.n_buckets):
        members = [t for t in range(T) if bof[t] == b]
        used = max(off[t] + numel[t] for t in members) - plan.bucket_start[b]
        assert used <= cap or len(members) == 1
    assert int(plan.bucket_numel.sum()) == plan.transport_numel
    assert plan.bucket_start.tolist() == np.concatenate([[0], np.cumsum(plan.bucket_numel)[:-1]]).tolist()


def test_plan_named_workloads(oracle):
    # tiny: one bucket, 10 218 elements padded to 10 240
    wl = W.tiny()
    p = oracle.bucket_plan(wl.numel, wl.bucket_cap_bytes)
    check_plan_invariants(wl.numel, wl.bucket_cap_bytes, p)
    assert p.n_buckets == 1 and p.transport_numel == 10240
    assert p.tensor_offset.tolist() == [9792, 9776, 5168, 5136, 16, 0]
    # ResNet-18 (10 classes): the head and the last block fill 18.5 MiB, the rest 24.1 MiB
    wl = W.resnet18()
    p = oracle.bucket_plan(wl.numel, 25 * MIB)
    check_plan_invariants(wl.numel, 25 * MIB, p)
    assert p.n_buckets == 2
    assert [round(n * 4 / MIB, 1) for n in p.bucket_numel] == [18.5, 24.1]
    # ResNet-50: five buckets under a 25 MiB fp32 cap; MobileNetV2: one
    wl = W.resnet50()
    p = oracle.bucket_plan(wl.numel, 25 * MIB)
    check_plan_invariants(wl.numel, 25 * MIB, p)
    assert p.n_buckets == 5
    wl = W.mobilenet_v2()
    p = oracle.bucket_plan(wl.numel, 25 * MIB)
    check_plan_invariants(wl.numel, 25 * MIB, p)
    assert p.n_buckets == 1


def test_plan_random_invariants(oracle):
    rnd = random.Random(5)
    for _ in range(300):
        T = rnd.randint(1, 40)
        numel = [rnd.choice([0, 1, 7, 8, 9, 63, 64, 65, 100, 1000, 4097]) for _ in range(T)]
        cap_bytes = rnd.choice([4, 32, 256, 1000, 4096, 20000, 1 << 40])
        p = oracle.bucket_plan(numel, cap_bytes)
        check_plan_invariants(numel, cap_bytes, p)


def test_plan_oversized_tensor_gets_own_bucket(oracle):
    p = oracle.bucket_plan([10, 5000, 10], 4000)   # cap = 1000 elements
    assert p.bucket_of.tolist() == [2, 1, 0]
    assert p.tensor_offset.tolist() == [5120, 64, 0]


# ------------------------------------------------------------------ casts
def test_bf16_widen_narrow_identity_all_patterns(oracle):
    h = np.arange(65536, dtype=np.uint16)
    f = oracle.bf16_to_f32(h)
    # widening is exact: same value as torch's bf16 -> fp32
    tf = torch.from_numpy(h.view(np.int16)).view(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(f.view(np.uint32), tf.view(np.uint32))
    back = oracle.f32_to_bf16(f)
    nan = np.isnan(f)
    assert np.array_equal(back[~nan], h[~nan])
    assert np.all(np.isnan(oracle.bf16_to_f32(back[nan])))


def test_f32_to_bf16_against_library_cast(oracle):
    # every upper half-word crossed with the lower half-words that decide rounding,
    # plus random ones: ties, just below / above a tie, all-ones, zero
    hi = np.arange(65536, dtype=np.uint32) << 16
    lows = [0x0000, 0x0001, 0x7FFF, 0x8000, 0x8001, 0xFFFF, 0x4000, 0xC000]
    rng = np.random.default_rng(11)
    lows += rng.integers(0, 65536, size=24).tolist()
    bits = (hi[:, None] | np.array(lows, dtype=np.uint32)[None, :]).reshape(-1)
    f = bits.view(np.float32)
    got = oracle.f32_to_bf16(f)
    want = torch.from_numpy(f.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    nan = np.isnan(f)
    assert np.array_equal(got[~nan], want[~nan])
    # NaN stays NaN with its sign
    g = oracle.bf16_to_f32(got[nan])
    assert np.all(np.isnan(g))
    assert np.array_equal(got[nan] >> 15, (bits[nan] >> 31).astype(np.uint16))


def test_f32_to_bf16_closed_forms(oracle):
    def one(x):
        return int(oracle.f32_to_bf16(np.array([x], np.float32))[0])
    assert one(1.0) == 0x3F80
    assert one(np.float32(1.0) + np.float32(2.0 ** -8)) == 0x3F80        # tie -> even (down)
    assert one(np.float32(1.0) + np.float32(3 * 2.0 ** -8)) == 0x3F82    # tie -> even (up)
    assert one(np.float32(1.0) + np.float32(2.0 ** -8) + np.float32(2.0 ** -20)) == 0x3F81
    assert one(3.4e38) == 0x7F80                                          # rounds up to +inf
    assert one(-0.0) == 0x8000
    assert one(np.float32(2.0 ** -140)) == one(np.float32(2.0 ** -140))   # subnormal: defined
    assert one(np.float32(2.0 ** -133)) == 0x0001                         # smallest bf16 subnormal


# ------------------------------------------------------------------ pack / unpack
def test_pack_unpack_identity(oracle):
    rng = np.random.default_rng(3)
    for dtype, npd in ((F32, np.float32), (BF16, np.uint16)):
        numel = [432, 16, 4608, 32, 5120, 10, 0, 1, 77]
        plan = oracle.bucket_plan(numel, 8000 * 4)
        if dtype == F32:
            tensors = [rng.standard_normal(n).astype(np.float32) for n in numel]
        else:
            tensors = [rng.integers(0, 0x7F80, size=n).astype(np.uint16) for n in numel]
        flat = oracle.pack(tensors, plan, dtype)
        # every tensor sits at its offset, everything else is zero
        mask = np.zeros(plan.transport_numel, bool)
        for t, x in enumerate(tensors):
            o = int(plan.tensor_offset[t])
            assert np.array_equal(flat[o:o + x.size], x)
            mask[o:o + x.size] = True
        assert not flat[~mask].any()
        if dtype == F32:
            out = oracle.unpack_scale(flat, plan, 1.0, F32)
            for x, y in zip(tensors, out):
                assert np.array_equal(x.view(np.uint32), y.view(np.uint32))


# ------------------------------------------------------------------ reduce
def exact_weighted_mean(xs, shares):
    """sum_r (b_r / B) x_r in exact rationals (xs: list over ranks of float lists)."""
    B = sum(shares)
    n = len(xs[0])
    return [sum(Fraction(b, B) * Fraction(float(x[i])) for b, x in zip(shares, xs)) for i in range(n)]


def run_path(oracle, grads, numel, dtype, group_of, shares, G, cap=25 * MIB, scale=1.0, out_dtype=None):
    out, partials, S, plan = oracle.sync_step(grads, numel, dtype, group_of, shares, G, cap, scale, out_dtype)
    return out, partials, S, plan


def test_brute_force_exact_rationals_tiny(oracle):
    """Distinct values everywhere, ragged shapes, three uneven groups, several buckets:
    a wrong index, weight, sign or a dropped term moves the result far outside the
    rounding bound."""
    rng = np.random.default_rng(17)
    numel = [5, 1, 12, 9, 3]
    group_of = [2, 0, 1, 0, 2, 0, 1]
    shares = [7, 64, 13, 21, 40, 5, 33]
    K, G = len(group_of), 3
    grads = [[rng.standard_normal(n).astype(np.float32) * (r + 1) for n in numel] for r in range(K)]
    out, partials, S, plan = run_path(oracle, grads, numel, F32, group_of, shares, G, cap=16 * 4)
    assert plan.n_buckets > 1
    for t, n in enumerate(numel):
        want = exact_weighted_mean([grads[r][t] for r in range(K)], shares)
        mag = exact_weighted_mean([np.abs(grads[r][t]) for r in range(K)], shares)
        for j in range(n):
            err = abs(Fraction(float(out[t][j])) - want[j])
            assert err <= mag[j] * Fraction(K + G + 2, 2 ** 24)
    # group partials are the group means
    for g in range(G):
        members = [r for r in range(K) if group_of[r] == g]
        for t, n in enumerate(numel):
            gs = [shares[r] for r in members]
            want = exact_weighted_mean([grads[r][t] for r in members], gs)
            mag = exact_weighted_mean([np.abs(grads[r][t]) for r in members], gs)
            o = int(plan.tensor_offset[t])
            for j in range(n):
                got = Fraction(float(partials[g][o + j]))
                assert abs(got - want[j]) <= mag[j] * Fraction(len(members) + 1, 2 ** 24)
    # padding of the transport is zero
    mask = np.zeros(plan.transport_numel, bool)
    for t, n in enumerate(numel):
        mask[int(plan.tensor_offset[t]):int(plan.tensor_offset[t]) + n] = True
    for g in range(G):
        assert not partials[g][~mask].any()


def test_identical_ranks_reproduce_input(oracle):
    rng = np.random.default_rng(1)
    numel = W.tiny().numel
    x = [rng.standard_normal(n).astype(np.float32) * 1e-3 for n in numel]
    # shares that make every coefficient a power of two: exact
    out, *_ = run_path(oracle, [x] * 4, numel, F32, [0, 0, 1, 1], [64, 64, 64, 64], 2)
    for a, b in zip(out, x):
        assert np.array_equal(a, b)
    # uneven shares: within a few ulp
    out, *_ = run_path(oracle, [x] * 4, numel, F32, [0, 0, 1, 1], [79, 79, 49, 49], 2)
    for a, b in zip(out, x):
        assert np.max(np.abs(a - b) / np.abs(b)) < 1e-6


def test_equal_shares_give_arithmetic_mean(oracle):
    rng = np.random.default_rng(2)
    numel = [1000, 37]
    K = 6
    grads = [[rng.standard_normal(n).astype(np.float32) * 1e-3 for n in numel] for _ in range(K)]
    out, *_ = run_path(oracle, grads, numel, F32, [0, 0, 0, 1, 1, 1], [32] * K, 2)
    for t in range(len(numel)):
        stack = np.stack([grads[r][t].astype(np.float64) for r in range(K)])
        mean = stack.mean(axis=0)
        scale = np.abs(stack).mean(axis=0)
        assert np.max(np.abs(out[t] - mean) / scale) < 1e-6


def test_single_rank_and_singleton_groups(oracle):
    rng = np.random.default_rng(4)
    numel = [257]
    x = [[rng.standard_normal(257).astype(np.float32)] for _ in range(5)]
    out, *_ = run_path(oracle, x[:1], numel, F32, [0], [9], 1)
    assert np.array_equal(out[0], x[0][0])                    # K = 1: identity
    # every rank its own group: the two-level mean is the flat one, operation by operation
    shares = [5, 9, 17, 3, 30]
    out, *_ = run_path(oracle, x, numel, F32, [0, 1, 2, 3, 4], shares, 5)
    _, _, w = oracle.coefficients([0, 1, 2, 3, 4], shares, 5)
    flat = oracle.flat_reduce_f32([xr[0] for xr in x], F32, w)
    assert np.array_equal(out[0], flat)


@pytest.mark.parametrize("dtype", [F32, BF16])
def test_hierarchical_equals_flat_within_tolerance(oracle, dtype):
    wl = W.tiny()
    K, G = 8, 3
    group_of = [0, 0, 0, 0, 1, 1, 2, 2]
    shares = [40, 40, 40, 40, 29, 29, 19, 19]
    gens = [torch.Generator().manual_seed(100 + r) for r in range(K)]
    flats = [torch.randn(wl.N, generator=g) * 1e-3 for g in gens]
    if dtype == BF16:
        flats = [f.to(torch.bfloat16) for f in flats]
    xs = [W.as_numpy(f) for f in flats]
    grads = [[W.as_numpy(t) for t in W.split_tensors(f, wl.numel)] for f in flats]
    out, _, _, plan = run_path(oracle, grads, wl.numel, dtype, group_of, shares, G, out_dtype=F32)
    got = np.concatenate(out)
    F, absF = oracle.flat_reduce_f64(xs, dtype, shares)
    # the fp64 routine itself against numpy
    x64 = np.stack([oracle.bf16_to_f32(x) if dtype == BF16 else x for x in xs]).astype(np.float64)
    wts = np.array(shares, np.float64) / sum(shares)
    assert np.allclose(F, (wts[:, None] * x64).sum(0), rtol=1e-13, atol=0)
    assert np.allclose(absF, (wts[:, None] * np.abs(x64)).sum(0), rtol=1e-13, atol=0)
    assert np.max(np.abs(got - F) / absF) < 1e-6
    # and against the one-level fp32 chain
    _, _, w = oracle.coefficients(group_of, shares, G)
    flat32 = oracle.flat_reduce_f32(xs, dtype, w)
    assert np.max(np.abs(got - flat32) / absF) < 1e-6
    if dtype == BF16:
        # narrowed output: within bf16 rounding of the fp64 mean
        out_b, *_ = run_path(oracle, grads, wl.numel, dtype, group_of, shares, G, out_dtype=BF16)
        got_b = oracle.bf16_to_f32(np.concatenate(out_b))
        assert np.max(np.abs(got_b - F) / np.maximum(np.abs(F), absF * 0.5)) < 1e-2


def _round_to_f32(x: Fraction) -> np.float32:
    """Correctly rounded (nearest, ties to even) binary32 value of an exact rational."""
    if x == 0:
        return np.float32(0.0)
    sign, mag = (-1 if x < 0 else 1), abs(x)
    e = mag.numerator.bit_length() - mag.denominator.bit_length()
    if Fraction(2) ** e > mag:
        e -= 1                                               # now 2^e <= mag < 2^(e+1)
    q = max(e, -126) - 23                                    # weight of the last kept bit (subnormals: fixed)
    scaled = mag / Fraction(2) ** q
    n = scaled.numerator // scaled.denominator
    rest = scaled - n
    if rest > Fraction(1, 2) or (rest == Fraction(1, 2) and n % 2 == 1):
        n += 1
    return np.float32(sign * float(Fraction(n) * Fraction(2) ** q))   # n * 2^q has at most 24 bits: exact in double


def test_reduction_chains_are_one_product_then_fused_multiply_adds_exactly(oracle):
    """The order and the roundings the oracle states -- first term one rounded product, every
    later term ONE rounding of a*x + acc -- checked element by element against exact rational
    arithmetic with a correctly rounded conversion written here.  A chain that rounded the
    product and the sum separately, started from zero, or took the ranks in another order
    fails this on inputs like these."""
    rng = np.random.default_rng(23)
    for d in np.concatenate([rng.standard_normal(500) * 1e-3, rng.standard_normal(200) * 1e-42, [0.0, 1.0, -2.5e38]]):
        assert _round_to_f32(Fraction(float(d))).tobytes() == np.float32(d).tobytes()      # the helper rounds as numpy does
    numel = [37, 8]
    group_of, shares, G = [0, 1, 0, 1, 0], [40, 29, 40, 19, 7], 2
    K = len(group_of)
    grads = [[(rng.standard_normal(n) * 1e-3).astype(np.float32) for n in numel] for _ in range(K)]
    a, Wg, w = oracle.coefficients(group_of, shares, G)
    plan = oracle.bucket_plan(numel, 25 * MIB)
    parts = oracle.intra_reduce(grads, plan, F32, group_of, a, G)
    S = oracle.combine(parts, Wg)
    flat = oracle.flat_reduce_f32([np.concatenate(g) for g in grads], F32, w)
    fr = lambda v: Fraction(float(v))

    def chain(weights, values):
        acc = _round_to_f32(fr(weights[0]) * fr(values[0]))
        for wt, v in zip(weights[1:], values[1:]):
            acc = _round_to_f32(fr(wt) * fr(v) + fr(acc))
        return acc

    separate_roundings_differ = 0
    for t, n in enumerate(numel):
        off = int(plan.tensor_offset[t])
        for j in range(n):
            want_parts = []
            for g in range(G):
                members = [r for r in range(K) if group_of[r] == g]
                want = chain([a[r] for r in members], [grads[r][t][j] for r in members])
                assert parts[g][off + j].tobytes() == want.tobytes()
                want_parts.append(want)
                two = np.float32(a[members[0]]) * grads[members[0]][t][j]
                for r in members[1:]:
                    two = np.float32(np.float32(a[r]) * grads[r][t][j]) + two
                separate_roundings_differ += two.tobytes() != want.tobytes()
            assert S[off + j].tobytes() == chain(list(Wg), want_parts).tobytes()
    pos = 0
    for t, n in enumerate(numel):
        for j in range(n):
            assert flat[pos].tobytes() == chain(list(w), [grads[r][t][j] for r in range(K)]).tobytes()
            pos += 1
    assert separate_roundings_differ > 0          # the inputs do tell the two kinds of chain apart


def test_unpack_scale_is_slicing_one_multiply_and_the_library_cast(oracle):
    """kto_unpack_scale pinned exactly, both output types: out[t][j] must be the fp32 product
    S[off_t + j] * scale (numpy's float32 multiply, one rounding) and, for bf16 outputs, torch's
    round-to-nearest-even cast of that product, bit for bit; padding never reaches an output."""
    rng = np.random.default_rng(12)
    numel = [1, 7, 4096, 513, 0, 10]
    plan = oracle.bucket_plan(numel, 3000 * 4)
    assert plan.n_buckets > 1
    S = (rng.standard_normal(plan.transport_numel) * 1e-3).astype(np.float32)
    S[::97] *= np.float32(1e30)                              # large magnitudes: rounding carries into the exponent
    S[5::101] = np.float32(3e-41)                            # subnormals
    covered = np.zeros(plan.transport_numel, bool)
    for t, n in enumerate(numel):
        covered[plan.tensor_offset[t]:plan.tensor_offset[t] + n] = True
    S_poisoned = S.copy()
    S_poisoned[~covered] = np.float32(np.nan)                # whatever sits in the padding
    for scale in (1.0, 0.5, 1.0 / 3.0, 1.0 / 256.0):
        for S_in in (S, S_poisoned):
            out32 = oracle.unpack_scale(S_in, plan, scale, F32)
            out16 = oracle.unpack_scale(S_in, plan, scale, BF16)
            for t, n in enumerate(numel):
                off = int(plan.tensor_offset[t])
                want32 = S[off:off + n] * np.float32(scale)
                assert out32[t].tobytes() == want32.tobytes()
                want16 = torch.from_numpy(want32.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
                assert out16[t].tobytes() == want16.tobytes()


def test_sum_then_divide_reading_agrees(oracle):
    """Weights a_r = b_r, W_g = 1 and a final scale 1/B (plain sums across the
    hierarchy, one division at the end) give the same mean within tolerance."""
    rng = np.random.default_rng(8)
    numel = [300, 11]
    group_of, shares, G = [0, 1, 1, 0], [64, 32, 32, 64], 2
    grads = [[rng.standard_normal(n).astype(np.float32) * 1e-3 for n in numel] for _ in range(4)]
    out, *_ = run_path(oracle, grads, numel, F32, group_of, shares, G)
    plan = oracle.bucket_plan(numel, 25 * MIB)
    parts = oracle.intra_reduce(grads, plan, F32, group_of, np.array(shares, np.float32), G)
    S = oracle.combine(parts, np.ones(G, np.float32))
    out2 = oracle.unpack_scale(S, plan, 1.0 / sum(shares), F32)
    for a, b in zip(out, out2):
        assert np.max(np.abs(a - b)) <= 4e-7 * np.max(np.abs(a))


def test_linearity_under_power_of_two_scaling(oracle):
    rng = np.random.default_rng(9)
    numel = [500]
    group_of, shares, G = [0, 0, 1], [10, 20, 30], 2
    grads = [[rng.standard_normal(500).astype(np.float32)] for _ in range(3)]
    base, *_ = run_path(oracle, grads, numel, F32, group_of, shares, G)
    scaled, *_ = run_path(oracle, [[g[0] * np.float32(8.0)] for g in grads], numel, F32, group_of, shares, G)
    assert np.array_equal(scaled[0], base[0] * np.float32(8.0))
    viaarg, *_ = run_path(oracle, grads, numel, F32, group_of, shares, G, scale=0.25)
    assert np.array_equal(viaarg[0], base[0] * np.float32(0.25))


def test_threaded_slices_equal_single_thread(oracle):
    rng = np.random.default_rng(10)
    n = 100_003
    x = [rng.standard_normal(n).astype(np.float32) for _ in range(4)]
    out, *_ = run_path(oracle, [[xr] for xr in x], [n], F32, [0, 0, 1, 1], [79, 79, 49, 49], 2)
    thr = oracle.sync_step_flat_threads(x, F32, [0, 0, 1, 1], [79, 79, 49, 49], 2, 1.0, F32, 3)
    assert np.array_equal(out[0], thr)


# ----------------------------------------------------------------------------- broadcast
@pytest.mark.parametrize("dtype", [F32, BF16])
def test_broadcast_hands_every_rank_the_roots_bytes(oracle, dtype):
    """Pin for the broadcast oracle: numpy's own array comparison on raw bit patterns, with
    values a careless copy would change (NaNs with payloads, signalling NaNs, -0, denormals,
    infinities), odd sizes and an empty tensor; the flat buffer holds the root's tensors at the
    plan's offsets and zeros elsewhere (checked by numpy slicing, not by the oracle's unpack)."""
    rng = np.random.default_rng(11)
    numel = [0, 1, 7, 8, 9, 64, 1000, 4097]
    K, root = 5, 3
    udt = np.uint32 if dtype == F32 else np.uint16
    special = np.array([0x7FC00001, 0x7F800001, 0xFFC12345, 0x80000000, 0x00000001, 0x807FFFFF,
                        0x7F800000, 0xFF800000], dtype=np.uint32)
    special = special if dtype == F32 else (special >> 16).astype(np.uint16) | np.uint16(1)
    ranks = []
    for r in range(K):
        row = []
        for n in numel:
            bits = rng.integers(0, np.iinfo(udt).max, size=n, dtype=udt, endpoint=True)
            bits[: min(n, special.size)] = special[: min(n, special.size)]
            row.append(bits.view(np.float32) if dtype == F32 else bits)
        ranks.append(row)
    before_root = [a.copy() for a in ranks[root]]
    out, flat, plan = oracle.broadcast(ranks, root, numel, dtype, 4096)
    covered = np.zeros(plan.transport_numel, bool)
    for t, n in enumerate(numel):
        off = int(plan.tensor_offset[t])
        assert np.array_equal(flat[off:off + n].view(udt), before_root[t].view(udt))
        covered[off:off + n] = True
    assert not flat.view(udt)[~covered].any()
    for r in range(K):
        for t in range(len(numel)):
            assert out[r][t].dtype == before_root[t].dtype
            assert np.array_equal(out[r][t].view(udt), before_root[t].view(udt)), (r, t)


# ----------------------------------------------------------------------------- bf16 transport (extension)
def test_bf16_transport_rounds_partials_once_and_stays_within_the_bf16_bar(oracle):
    """Pins for the oracle's bf16-transport reading: (1) where every partial is representable
    in bf16 the result equals the fp32-transport result bit for bit; (2) otherwise the error
    against the fp64 mean is bounded by the one extra rounding, 2^-8 of sum_g W_g |P_g| (bf16 keeps
    8 significant bits, so half a unit in the last place is 2^-8 relative), inside
    inside 1e-2; (3) the stored partials are the library cast of the fp32 partials."""
    rng = np.random.default_rng(4)
    numel = [5, 64, 1000, 4097]
    group_of, shares = [0, 0, 1, 1], [1, 1, 1, 1]          # a = 1/2, W = 1/2: powers of two
    # (1) values with few mantissa bits: sums of two, scaled by 1/2, stay bf16-representable
    coarse = [[(rng.integers(-8, 9, size=n) * 2.0 ** -10).astype(np.float32) for n in numel] for _ in range(4)]
    a = oracle.sync_step(coarse, numel, F32, group_of, shares, 2, 1 << 20)
    b = oracle.sync_step(coarse, numel, F32, group_of, shares, 2, 1 << 20, transport_dtype=BF16)
    for t in range(len(numel)):
        assert np.array_equal(a[0][t].view(np.uint32), b[0][t].view(np.uint32))
    # (2), (3) generic values
    shares = [79, 79, 49, 49]
    fine = [[(rng.standard_normal(n) * 1e-3).astype(np.float32) for n in numel] for _ in range(4)]
    out32, parts32, _, _ = oracle.sync_step(fine, numel, F32, group_of, shares, 2, 1 << 20)
    out16, parts16, _, _ = oracle.sync_step(fine, numel, F32, group_of, shares, 2, 1 << 20, transport_dtype=BF16)
    for g in range(2):
        lib = torch.from_numpy(parts32[g]).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        assert np.array_equal(parts16[g], lib)
    F, absF = oracle.flat_reduce_f64([np.concatenate(x) for x in fine], F32, shares)
    got = np.concatenate(out16)
    err = np.abs(got - F) / absF
    assert err.max() <= 2.0 ** -8 + 1e-6 and err.max() > 1e-6      # one bf16 rounding, and it is there
