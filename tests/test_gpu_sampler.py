"""GPU parity of the load-adaptive sampler kernel (kt_sampler_indices) against the CPU
oracle: integer index work, so every entry must match exactly."""
import random

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def kt():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    from paper_2505_10183_b200 import binding
    torch.cuda.set_device(0)
    return binding


def run(kt, oracle, D, shares, drop_last, shuffled=True, seed=0):
    perm = None
    if shuffled:
        g = torch.Generator().manual_seed(seed)
        perm = torch.randperm(D, generator=g)
    steps = kt.kt_sampler_steps(D, sum(shares), drop_last)
    guard = 16
    bufs = [torch.full((steps * b + 2 * guard,), -7, dtype=torch.int64, device="cuda") for b in shares]
    out = [buf[guard:guard + steps * b] for buf, b in zip(bufs, shares)]
    kt.kt_sampler_indices(perm.cuda() if perm is not None else None, D, shares, out, drop_last=drop_last)
    torch.cuda.synchronize()
    want = oracle.sampler_indices(perm.numpy() if perm is not None else None, D, shares, drop_last)
    assert steps == oracle.sampler_steps(D, sum(shares), drop_last)
    for r in range(len(shares)):
        assert np.array_equal(out[r].cpu().numpy(), want[r]), "rank %d" % r
        assert bool((bufs[r][:guard] == -7).all()) and bool((bufs[r][guard + steps * shares[r]:] == -7).all())


def test_paper_training_setup(kt, oracle):
    """50 000 training images, global batch 256 (Section IV-B), shares of the 2G+2M-like
    schedule; with and without the incomplete last batch, shuffled and not."""
    for drop_last in (False, True):
        for shuffled in (True, False):
            run(kt, oracle, 50000, [79, 79, 49, 49], drop_last, shuffled)
    run(kt, oracle, 1281167, [40, 40, 40, 40, 29, 29, 19, 19], False)     # an ImageNet-sized epoch


@pytest.mark.parametrize("seed", range(3))
def test_random_cases(kt, oracle, seed):
    rnd = random.Random(300 + seed)
    for _ in range(30):
        K = rnd.randint(1, 16)
        shares = [rnd.randint(1, 64) for _ in range(K)]
        B = sum(shares)
        D = rnd.choice([1, B - 1 if B > 1 else 1, B, B + 1, 3 * B, rnd.randint(1, 20000)])
        run(kt, oracle, D, shares, rnd.random() < 0.5, rnd.random() < 0.7, seed=rnd.randint(0, 99))


def test_degenerate_and_maximum(kt, oracle):
    run(kt, oracle, 5, [8], True)                      # fewer samples than one batch, dropped: no steps
    run(kt, oracle, 5, [8], False)                     # ... kept: one step that wraps around
    run(kt, oracle, 10007, [1] * 64, False)            # the maximum rank count
    with pytest.raises(kt.KtError) as e:
        kt.kt_sampler_indices(None, 100, [1] * 65, [torch.zeros(2, dtype=torch.int64, device="cuda")] * 65)
    assert e.value.status == kt.KT_ERR_INVALID
