"""Pins for the oracle's load-adaptive sampler (paper Section III-C "Dynamic Data
Allocation", Section IV-A sampler) and online adaptation (Section III-C "Online
Adaptation"), and host-side parity of the library's kt_adapt_* against the oracle.

The sampler is pinned to brute force over Python sets written from the text, to counting
identities, and, for equal shares, to torch.utils.data.DistributedSampler; the adaptation to
the closed form of an exponential moving average, to the fixed point schedule(tau) and to
its no-thrash property."""
import math
import random

import numpy as np
import pytest
import torch


# ----------------------------------------------------------------------------- sampler
def brute_force_sampler(lst, D, shares, drop_last):
    """Written from the text, position by position, nothing shared with the oracle's loops."""
    B = sum(shares)
    S = D // B if drop_last else -(-D // B)
    out = [[] for _ in shares]
    for p in range(S * B):
        s, w = divmod(p, B)
        r, c = 0, 0
        while w >= c + shares[r]:
            c += shares[r]
            r += 1
        out[r].append(lst[p % D])
    return out, S


@pytest.mark.parametrize("drop_last", [False, True])
def test_sampler_brute_force_and_partition(oracle, drop_last):
    rnd = random.Random(3)
    for _ in range(60):
        K = rnd.randint(1, 9)
        shares = [rnd.randint(1, 40) for _ in range(K)]
        B = sum(shares)
        D = rnd.choice([B, 2 * B, 7 * B + rnd.randint(0, B - 1), rnd.randint(1, 5000)])
        perm = list(range(D))
        rnd.shuffle(perm)
        got = oracle.sampler_indices(np.array(perm), D, shares, drop_last)
        want, S = brute_force_sampler(perm, D, shares, drop_last)
        assert oracle.sampler_steps(D, B, drop_last) == S
        for r in range(K):
            assert got[r].tolist() == want[r]
            assert got[r].size == S * shares[r]          # load is proportional to the share, exactly
        # every step's slices together are exactly that step's positions of the list
        for s in range(S):
            step = sorted(v for r in range(K) for v in got[r][s * shares[r]:(s + 1) * shares[r]].tolist())
            assert step == sorted(perm[p % D] for p in range(s * B, (s + 1) * B))
        # whole epochs: nothing is lost when nothing is dropped, nothing repeats when D divides
        allv = np.concatenate(got) if S else np.zeros(0, np.int64)
        if not drop_last:
            assert set(allv.tolist()) == set(range(D))
        if D % B == 0:
            assert sorted(allv.tolist()) == list(range(D))


def test_sampler_identity_list_single_rank_and_wraparound(oracle):
    got = oracle.sampler_indices(None, 10, [4], False)          # K = 1: the list itself, continued from its start
    assert got[0].tolist() == [0, 1, 2, 3, 4, 5, 6, 7, 8, 9, 0, 1]
    assert oracle.sampler_indices(None, 10, [4], True)[0].tolist() == list(range(8))
    got = oracle.sampler_indices(None, 12, [3, 2, 1], False)     # worked by hand: c = 0, 3, 5; B = 6
    assert got[0].tolist() == [0, 1, 2, 6, 7, 8]
    assert got[1].tolist() == [3, 4, 9, 10]
    assert got[2].tolist() == [5, 11]
    with pytest.raises(oracle.OracleError):
        oracle.sampler_indices(None, 10, [4, 0], False)
    with pytest.raises(oracle.OracleError):
        oracle.sampler_indices(None, 0, [4], False)


def test_sampler_equal_shares_cover_the_same_steps_as_the_library_sampler(oracle):
    """With equal shares, every step's global mini-batch (the union over ranks) must be the one
    torch.utils.data.DistributedSampler + a per-rank batch of b produce; the library hands the
    positions of a step to ranks in a different order (strided), so sets are compared."""
    from torch.utils.data import DistributedSampler
    K, b = 4, 8
    D = 10 * K * b + K * 3          # a multiple of K, so that both pad alike; last step incomplete
    data = list(range(D))
    per_rank = [list(iter(DistributedSampler(data, num_replicas=K, rank=r, shuffle=False))) for r in range(K)]
    got = oracle.sampler_indices(None, D, [b] * K, False)
    full_steps = D // (K * b)
    for s in range(full_steps):
        lib_step = sorted(v for r in range(K) for v in per_rank[r][s * b:(s + 1) * b])
        our_step = sorted(v for r in range(K) for v in got[r][s * b:(s + 1) * b].tolist())
        assert our_step == lib_step
    # the incomplete last step: the library pads up to a multiple of K from the start of the list,
    # this sampler up to a multiple of B; the library's tail is a prefix of ours as a multiset
    lib_tail = sorted(v for r in range(K) for v in per_rank[r][full_steps * b:])
    our_tail = sorted(v for r in range(K) for v in got[r][full_steps * b:].tolist())
    assert all(our_tail.count(v) >= lib_tail.count(v) for v in set(lib_tail))


# ----------------------------------------------------------------------------- online adaptation
def test_adapt_moving_average_closed_form(oracle):
    """Constant shares (period never reached): ema_n = tau + (tau_0 - tau) (1 - alpha)^n."""
    shares, alpha = [10, 30], 0.25
    ad = oracle.Adapter(shares, 40, alpha, 10 ** 6, 0.0)
    tau0, tau = np.array([0.02, 0.05]), np.array([0.03, 0.04])
    ad.observe(tau0 * shares)
    for n in range(1, 40):
        assert not ad.observe(tau * shares)
        want = tau + (tau0 - tau) * (1.0 - alpha) ** n
        assert np.allclose(ad.ema, want, rtol=1e-13, atol=0)
    assert ad.shares.tolist() == shares


def test_adapt_reaches_the_schedule_of_the_true_speeds_and_stays(oracle):
    rnd = random.Random(5)
    for _ in range(40):
        K = rnd.randint(2, 8)
        B = rnd.choice([64, 256, 500])
        tau = [rnd.choice([1.0, 1.25, 1.5, 2.0, 3.0]) / 64.0 for _ in range(K)]     # exact in binary
        start = oracle.schedule([1.0] * K, B).tolist()
        ad = oracle.Adapter(start, B, 1.0, 1, 0.0)
        changes = 0
        for _ in range(6):
            changes += ad.observe([t * b for t, b in zip(tau, ad.shares)])
            assert int(ad.shares.sum()) == B and int(ad.shares.min()) >= 1
        target = oracle.schedule(tau, B).tolist()
        predicted = lambda b: max(t * x for t, x in zip(tau, b))
        # the fixed point is the schedule of the true per-sample times unless the start was already as good
        assert ad.shares.tolist() == target or predicted(ad.shares) <= predicted(target)
        assert changes <= 1
        assert predicted(ad.shares) <= predicted(start)


def test_adapt_hysteresis_keeps_shares_under_noise_and_follows_a_real_slowdown(oracle):
    rng = np.random.default_rng(9)
    tau = np.array([1.0, 1.0, 1.6, 1.6]) / 64.0
    ad = oracle.Adapter([64] * 4, 256, 0.3, 5, 0.05)
    history = []
    for step in range(200):
        noise = 1.0 + rng.uniform(-0.01, 0.01, size=4)
        history.append(ad.observe(tau * ad.shares * noise))
    assert sum(history) == 1 and ad.shares.tolist() == [79, 79, 49, 49]      # one move, then quiet
    # rank 0 throttles to half speed: the shares follow within a few periods, and settle again
    tau2 = tau.copy()
    tau2[0] *= 2.0
    moves = [ad.observe(tau2 * ad.shares * (1.0 + rng.uniform(-0.01, 0.01, size=4))) for _ in range(200)]
    assert 1 <= sum(moves) <= 6 and not any(moves[100:])
    want = oracle.schedule(tau2, 256)
    assert np.abs(ad.shares - want).max() <= 2
    assert ad.shares[0] < 79 / 1.5


def test_adapt_hysteresis_threshold_worked_by_hand(oracle):
    """Two ranks at 50 / 50 of 100 samples, every observation adopted into the average at once
    (alpha = 1, period = 1).  Per-sample times 1 and 1.5 (in 1/64 s): the step now takes
    max(50, 75) = 75; the schedule of those times is 60 / 40 and predicts max(60, 60) = 60, that is
    0.8 of 75.  New shares are taken only if they predict less than (1 - hysteresis) of the
    present step: at 0.25 they are not, at 0.15 they are.  With times 1 and 3 the candidate 75 / 25
    predicts 75 of 150, exactly one half: a hysteresis of one half keeps the old shares (the
    comparison is strict), a quarter lets them go."""
    def after_one(x, h):
        ad = oracle.Adapter([50, 50], 100, 1.0, 1, h)
        changed = ad.observe([50 * 1.0 / 64.0, 50 * x / 64.0])
        return bool(changed), ad.shares.tolist()
    assert after_one(1.5, 0.25) == (False, [50, 50])
    assert after_one(1.5, 0.15) == (True, [60, 40])
    assert after_one(1.5, 0.0) == (True, [60, 40])
    assert after_one(3.0, 0.5) == (False, [50, 50])
    assert after_one(3.0, 0.25) == (True, [75, 25])
    # equal speeds: the candidate is the present split, nothing to adopt whatever the threshold
    assert after_one(1.0, 0.0) == (False, [50, 50])


def test_adapt_rejects_bad_input(oracle):
    for alpha, period, h in ((0.0, 1, 0.0), (1.5, 1, 0.0), (0.5, 0, 0.0), (0.5, 1, 1.0), (0.5, 1, -0.1)):
        with pytest.raises(oracle.OracleError):
            oracle.Adapter([1, 1], 2, alpha, period, h).observe([1.0, 1.0])
    for times in ([1.0, 0.0], [1.0, -1.0], [float("nan"), 1.0], [float("inf"), 1.0]):
        with pytest.raises(oracle.OracleError):
            oracle.Adapter([1, 1], 2, 0.5, 1, 0.0).observe(times)


# ----------------------------------------------------------------------------- library vs oracle (host functions, no GPU)
@pytest.fixture(scope="module")
def kt():
    from paper_2505_10183_b200 import binding
    return binding


def test_library_adaptation_matches_oracle_bit_for_bit(kt, oracle):
    rnd = random.Random(21)
    for _ in range(60):
        K = rnd.randint(1, 12)
        B = rnd.randint(K, 600)
        start = oracle.schedule([rnd.uniform(0.5, 2.0) for _ in range(K)], B).tolist()
        alpha, period, h = rnd.choice([0.1, 0.5, 1.0]), rnd.randint(1, 4), rnd.choice([0.0, 0.02, 0.2])
        ad = oracle.Adapter(start, B, alpha, period, h)
        st = kt.kt_adapt_create(start, B, alpha, period, h)
        tau = [rnd.uniform(0.5, 3.0) for _ in range(K)]
        for step in range(30):
            if step == 15:
                tau[rnd.randrange(K)] *= rnd.choice([0.5, 2.0, 3.0])
            times = [t * b * rnd.uniform(0.97, 1.03) for t, b in zip(tau, ad.shares)]
            changed_o = ad.observe(times)
            shares, changed = kt.kt_adapt_observe(st, times)
            assert shares == ad.shares.tolist() and changed == changed_o
            ema, b2, n = kt.kt_adapt_state(st)
            assert ema == ad.ema.tolist() and b2 == shares and n == step + 1       # doubles, bit for bit
        kt.kt_adapt_destroy(st)


def test_library_adaptation_and_sampler_argument_checks(kt):
    for args in (([1, 1], 3, 0.5, 1, 0.0), ([1, 0], 1, 0.5, 1, 0.0), ([1, 1], 2, 0.0, 1, 0.0),
                 ([1, 1], 2, 0.5, 0, 0.0), ([1, 1], 2, 0.5, 1, 1.0)):
        with pytest.raises(kt.KtError) as e:
            kt.kt_adapt_create(*args)
        assert e.value.status == kt.KT_ERR_INVALID
    st = kt.kt_adapt_create([1, 1], 2, 0.5, 1, 0.0)
    for times in ([1.0, 0.0], [float("nan"), 1.0]):
        with pytest.raises(kt.KtError) as e:
            kt.kt_adapt_observe(st, times)
        assert e.value.status == kt.KT_ERR_INVALID
    assert kt.kt_sampler_steps(50000, 256, False) == 196 and kt.kt_sampler_steps(50000, 256, True) == 195
    with pytest.raises(kt.KtError):
        kt.kt_sampler_steps(0, 256, False)
    with pytest.raises(kt.KtError) as e:        # validated on the host before anything is launched
        kt.kt_sampler_indices(None, 100, [0, 4], [torch.zeros(0, dtype=torch.int64)] * 2, stream=0)
    assert e.value.status == kt.KT_ERR_INVALID
