"""Pins for the oracle's scheduler and weights (Section III-C; group weights of the
two-level mean).  Everything here compares the oracle with exact rational arithmetic,
closed forms or the paper's printed example -- never with the oracle itself."""
import os
import random
from fractions import Fraction
from math import floor

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "schedule_paper_example.txt")


def exact_quotas(times, B):
    """Section III-C allocation formula in exact rationals."""
    times = [Fraction(t) for t in times]
    tmin = min(times)
    scores = [tmin / t for t in times]
    total = sum(scores)
    return scores, [s / total * B for s in scores]


def exact_shares(times, B):
    """Largest-remainder repair of the rounded quotas, exact; None when a remainder
    tie between different quotas would make the result depend on rounding noise."""
    _, q = exact_quotas(times, B)
    base = [floor(x) for x in q]
    rem = [x - b for x, b in zip(q, base)]
    missing = B - sum(base)
    order = sorted(range(len(q)), key=lambda i: (-rem[i], i))
    if 0 < missing < len(q):
        cut_in, cut_out = order[missing - 1], order[missing]
        if rem[cut_in] == rem[cut_out] and times[cut_in] != times[cut_out]:
            return None
    for i in order[:missing]:
        base[i] += 1
    return base


def test_paper_example_scores_and_shares(oracle):
    rows = [l.split() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    speeds = [float(r[1]) for r in rows if r[0] != "global_batch"]
    scores = [Fraction(r[2]) for r in rows if r[0] != "global_batch"]
    B = int([r for r in rows if r[0] == "global_batch"][0][1])
    times = [Fraction(1) / Fraction(str(s)) for s in speeds]     # time is inverse speed
    got_scores, q = exact_quotas(times, B)
    assert got_scores == scores                                   # 1.0 and 0.7 as printed
    # 256 * 1/1.7 = 150.59, 256 * 0.7/1.7 = 105.41 -> nearest integers 151 and 105
    assert [round(x) for x in q] == [151, 105]
    got = oracle.schedule([float(t) for t in times], B)
    assert got.tolist() == [151, 105]
    # the score function on its own, oracle and library: the printed 1.0 and 0.7
    from paper_2505_10183_b200 import binding as kt
    for fn in (lambda t: oracle.scores(t).tolist(), kt.kt_scores):
        sc = fn([float(t) for t in times])
        assert sc[0] == 1.0 and abs(sc[1] - 0.7) < 1e-15
    import random
    rnd = random.Random(2)
    for _ in range(300):
        ts = [rnd.uniform(0.01, 50.0) for _ in range(rnd.randint(1, 64))]
        want = [Fraction(min(ts)) / Fraction(t) for t in ts]          # exact quotient of the doubles
        got_o, got_l = oracle.scores(ts).tolist(), kt.kt_scores(ts)
        assert got_o == got_l == [float(w) for w in want]             # one correctly rounded division
        assert max(got_o) == 1.0
    for bad in ([], [1.0, 0.0], [float("nan")], [float("inf"), 1.0]):
        with pytest.raises(oracle.OracleError):
            oracle.scores(bad)
        with pytest.raises(kt.KtError):
            kt.kt_scores(bad)


@pytest.mark.parametrize("times,B,expect", [
    ([1, 1, 1, 1], 256, [64, 64, 64, 64]),           # equal devices: equal split
    ([1, 1, 1], 256, [86, 85, 85]),                  # 85.33 each; the spare unit goes to rank 0
    ([2.5], 17, [17]),                               # one device takes everything
    ([1, 2], 3, [2, 1]),                             # quotas are integers already
    ([1, 3], 4, [3, 1]),
])
def test_closed_forms(oracle, times, B, expect):
    assert oracle.schedule(times, B).tolist() == expect


def test_named_configs_against_exact_rationals(oracle):
    for times, B in (([1, 1, Fraction(8, 5), Fraction(8, 5)], 256),
                     ([1] * 4 + [Fraction(7, 5)] * 2 + [Fraction(21, 10)] * 2, 256),
                     ([1] * 4 + [Fraction(7, 5)] * 2 + [Fraction(21, 10)] * 2, 512)):
        want = exact_shares(times, B)
        got = oracle.schedule([float(t) for t in times], B).tolist()
        assert got == want
        assert sum(got) == B
    # nearest rounding alone would give 510 for the last case: the repair is needed
    _, q = exact_quotas([1] * 4 + [Fraction(7, 5)] * 2 + [Fraction(21, 10)] * 2, 512)
    assert sum(round(x) for x in q) == 510


def test_random_against_exact_rationals(oracle):
    rnd = random.Random(1234)
    checked = 0
    for _ in range(600):
        K = rnd.randint(1, 6)
        times = [Fraction(rnd.randint(5, 60), 10) for _ in range(K)]
        B = rnd.randint(K, 600)
        want = exact_shares(times, B)
        _, q = exact_quotas(times, B)
        if want is None or any(abs(x - round(x)) < Fraction(1, 10 ** 9) and x != round(x) for x in q):
            continue
        if min(want) < 1:
            continue                 # the at-least-one rule is pinned separately
        # integer quotas are fine for floor() only if fp64 reproduces them; keep cases
        # whose quotas are either exactly integral from exactly representable inputs or
        # safely fractional
        if any(x == round(x) for x in q) and len(set(times)) > 1:
            continue
        got = oracle.schedule([float(t) for t in times], B).tolist()
        assert got == want, (times, B)
        checked += 1
    assert checked > 300


def test_invariants(oracle):
    rnd = random.Random(99)
    for _ in range(300):
        K = rnd.randint(1, 16)
        times = [rnd.uniform(0.2, 5.0) for _ in range(K)]
        B = rnd.randint(K, 2048)
        b = oracle.schedule(times, B)
        assert int(b.sum()) == B                       # the sum matches the global batch
        assert int(b.min()) >= 1                       # nobody idles
        _, q = exact_quotas(times, B)
        if min(q) >= 1:
            # rounding moves a share by less than one unit
            assert all(abs(int(bi) - qi) < 1 for bi, qi in zip(b, q))
            # when plain nearest rounding already sums to B it is the answer
            near = [floor(x + Fraction(1, 2)) for x in q]
            if sum(near) == B and all(abs((x - floor(x)) - Fraction(1, 2)) > Fraction(1, 10 ** 6) for x in q):
                assert b.tolist() == near
        for i in range(K):                             # a faster device never gets less
            for j in range(K):
                if times[i] < times[j]:
                    assert b[i] >= b[j]


def test_equal_times_tie_goes_to_lower_rank(oracle):
    assert oracle.schedule([3.0] * 5, 13).tolist() == [3, 3, 3, 2, 2]
    # equalised step time: share x time spreads by at most one sample's worth
    t = [1.0, 1.3, 2.0, 2.9]
    b = oracle.schedule(t, 1000)
    per = [bi * ti for bi, ti in zip(b, t)]
    assert max(per) - min(per) <= max(t)


def test_nobody_gets_zero(oracle):
    # quota of the slow rank is 0.0099 * 4: floor 0; it must still get one sample
    b = oracle.schedule([1.0, 1.0, 1.0, 100.0], 4)
    assert b.tolist() == [1, 1, 1, 1]
    b = oracle.schedule([1.0, 1.0, 1000.0], 10)
    # the unit comes from the largest share; between equal devices the higher index gives
    assert b.tolist() == [5, 4, 1]
    # between unequal devices with equal shares the slower one gives: 2,2,0 -> 2,1,1
    assert oracle.schedule([1.0, 1.2, 500.0], 4).tolist() == [2, 1, 1]


@pytest.mark.parametrize("times,B", [([1.0, 0.0], 8), ([1.0, -2.0], 8), ([1.0, float("nan")], 8),
                                     ([1.0, float("inf")], 8), ([1.0, 1.0, 1.0], 2), ([], 4)])
def test_invalid_inputs_rejected(oracle, times, B):
    with pytest.raises(ValueError):
        oracle.schedule(times, B)


# ------------------------------------------------------------------ weights
def test_weights_exact_and_sum_to_one(oracle):
    rnd = random.Random(7)
    for _ in range(200):
        K = rnd.randint(1, 16)
        G = rnd.randint(1, K)
        group_of = list(range(G)) + [rnd.randrange(G) for _ in range(K - G)]
        rnd.shuffle(group_of)
        shares = [rnd.randint(1, 300) for _ in range(K)]
        a, W, w = oracle.coefficients(group_of, shares, G)
        B = sum(shares)
        Bg = [sum(s for s, g in zip(shares, group_of) if g == gg) for gg in range(G)]
        # exact rationals: the in-group weights and the group weights each sum to one
        assert sum(Fraction(s, Bg[g]) for s, g in zip(shares, group_of)) == G
        assert sum(Fraction(x, B) for x in Bg) == 1
        for r in range(K):
            # each coefficient is the correctly rounded float of its exact quotient
            assert a[r] == np.float32(shares[r] / Bg[group_of[r]])
            assert w[r] == np.float32(shares[r] / B)
            exact = Fraction(shares[r], B)
            two_level = Fraction(float(a[r])) * Fraction(float(W[group_of[r]]))
            assert abs(two_level - exact) <= exact * Fraction(2, 2 ** 23)
        for g in range(G):
            assert W[g] == np.float32(Bg[g] / B)
        assert abs(float(np.sum(W.astype(np.float64))) - 1.0) < 1e-6


def test_weights_of_named_configs(oracle):
    a, W, w = oracle.coefficients([0, 0, 1, 1], [64, 64, 32, 32], 2)
    assert a.tolist() == [0.5, 0.5, 0.5, 0.5]
    assert W.tolist() == [np.float32(2 / 3), np.float32(1 / 3)]
    assert w.tolist() == [np.float32(1 / 3)] * 2 + [np.float32(1 / 6)] * 2
    a, W, w = oracle.coefficients([0] * 4 + [1] * 4, [48] * 4 + [32] * 4, 2)
    assert a.tolist() == [0.25] * 8
    assert W.tolist() == [np.float32(3 / 5), np.float32(2 / 5)]
    assert w.tolist() == [np.float32(3 / 20)] * 4 + [np.float32(1 / 10)] * 4


@pytest.mark.parametrize("group_of,shares,G", [([0, 2], [1, 1], 3), ([0, 1], [1, 0], 2),
                                               ([0, -1], [1, 1], 2), ([0, 0], [1, 1], 3)])
def test_weights_invalid(oracle, group_of, shares, G):
    with pytest.raises(ValueError):
        oracle.coefficients(group_of, shares, G)


# ----------------------------------------------------------------------------- dispatch decision (Section III-B)
def test_route_decision_against_set_arithmetic_and_the_library(oracle):
    """Pin: Python set arithmetic on the paper's testbed shapes (2 GPUs + 2 MLUs and the other
    five configurations of Section IV-C) and on random layouts; the library's kt_route must
    give the same answer and the list of groups involved."""
    import random
    from paper_2505_10183_b200 import binding as kt
    # the paper's configurations: G = GPU group 0, M = MLU group 1
    for group_of, parts, want in (([0, 0], [0, 1], 0), ([1, 1], [0, 1], 0), ([0, 1], [0, 1], 1),
                                  ([0, 0, 1], [0, 1, 2], 1), ([0, 1, 1], [1, 2], 0), ([0, 0, 1, 1], [0, 1, 2, 3], 1),
                                  ([0, 0, 1, 1], [2, 3], 0), ([0, 0, 1, 1], [1], 0)):
        assert oracle.route(group_of, parts) == want
    rnd = random.Random(8)
    for _ in range(300):
        K = rnd.randint(1, 20)
        G = rnd.randint(1, min(K, 6))
        group_of = list(range(G)) + [rnd.randrange(G) for _ in range(K - G)]
        rnd.shuffle(group_of)
        parts = rnd.sample(range(K), rnd.randint(1, K))
        groups = sorted({group_of[r] for r in parts})
        want = 0 if len(groups) == 1 else 1
        assert oracle.route(group_of, parts) == want
        assert kt.kt_route(group_of, parts, G) == (want, groups)
    for bad in ([], [0, 0], [5], [-1]):
        with pytest.raises(oracle.OracleError):
            oracle.route([0, 1, 1], bad)
    for bad in ([], [0, 0], [5], [-1]):
        with pytest.raises(kt.KtError) as e:
            kt.kt_route([0, 1, 1], bad, 2)
        assert e.value.status == kt.KT_ERR_INVALID
