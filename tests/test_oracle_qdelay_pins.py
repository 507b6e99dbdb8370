"""Pins of the oracle's recent average queueing delay q_k (paper Sec. 4.2: a
sliding window, by default a 5 s linear weighted one) against closed forms of
the linearly weighted moving average, hand-worked cases and exact fractions."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import oracle

W = 5_000_000          # the paper's default window: 5 s


def q1(now, times, delays, window=W):
    t = np.asarray(times, dtype=np.int64).reshape(1, 1, -1)
    d = np.asarray(delays, dtype=np.int32).reshape(1, 1, -1)
    return int(oracle.queue_delay(np.array([now], np.int64), t, d, window)[0, 0])


def test_constant_delay_is_returned_whatever_the_weights():
    rng = np.random.default_rng(1)
    now = 10**9
    t = now - rng.integers(0, W, size=200)
    assert q1(now, t, np.full(200, 1234)) == 1234


def test_single_and_two_samples_by_hand():
    now = 7_000_000
    assert q1(now, [now - 100], [500]) == 500
    # ages 1 s and 4 s in a 5 s window: weights 4 and 1 (in seconds) -> (4*100 + 1*600) / 5 = 200
    assert q1(now, [now - 1_000_000, now - 4_000_000], [100, 600]) == 200
    # the newer sample dominates: swapping the delays gives (4*600 + 1*100) / 5 = 500
    assert q1(now, [now - 1_000_000, now - 4_000_000], [600, 100]) == 500
    # floor of a non-integer mean: weights 5 (age 0) and 2 (age 3 s): (5*1 + 2*2) / 7 = 1.28..
    assert q1(now, [now, now - 3_000_000], [1, 2]) == 1


def test_textbook_linearly_weighted_moving_average():
    """n samples one step apart, the newest at age 0 in a window of n steps:
    weights n, n-1, .., 1 and LWMA = sum (n-i) x_i / (n (n+1) / 2)."""
    rng = np.random.default_rng(2)
    for n in (1, 2, 5, 50):
        step = 1000
        x = rng.integers(0, 10_000, size=n)                 # x[0] newest
        now = 10**7
        t = now - step * np.arange(n)
        want = sum((n - i) * int(x[i]) for i in range(n)) // (n * (n + 1) // 2)
        assert q1(now, t, x, window=n * step) == want
        # the order of the slots does not matter
        perm = rng.permutation(n)
        assert q1(now, t[perm], x[perm], window=n * step) == want


def test_window_edges_empty_slots_and_future_samples():
    now = 10**8
    assert q1(now, [], []) == 0
    assert q1(now, [-1, -5], [77, 99]) == 0                  # empty slots
    assert q1(now, [now - W], [900]) == 0                    # exactly one window old: weight 0
    assert q1(now, [now - W + 1, now - W], [900, 5]) == 900  # weight 1 vs weight 0
    assert q1(now, [now + 1, now], [10**6, 40]) == 40        # a sample from after the snapshot is ignored
    assert q1(now, [now - 10, -1, now - 2 * W], [30, 10**6, 10**6]) == 30
    assert q1(100, [90, -1], [30, 10**6]) == 30              # early in the clock an empty slot is still empty


def test_older_samples_weigh_less():
    now = 10**8
    prev = None
    for age in range(0, W, W // 10):
        q = q1(now, [now - 1000, now - age], [0, 10_000])
        if prev is not None:
            assert q <= prev                                 # ageing the large sample lowers the average
        prev = q


@pytest.mark.parametrize("seed", range(8))
def test_exact_fractions(seed):
    rng = np.random.default_rng(300 + seed)
    n_ctx, S, M = 3, 4, int(rng.integers(1, 300))
    big = seed % 2 == 0
    window = (1 << 24) if big else int(rng.integers(1, 10**6))
    now = rng.integers(10**9, 2 * 10**9, size=n_ctx)
    t = now[:, None, None] - rng.integers(-window // 4, 2 * window, size=(n_ctx, S, M))
    t[rng.random(size=t.shape) < 0.1] = -1
    d = rng.integers((1 << 24) - 1000 if big else 0, 1 << 24, size=(n_ctx, S, M)).astype(np.int32)
    got = oracle.queue_delay(now, t, d, window)
    for c in range(n_ctx):
        for k in range(S):
            num, den = 0, 0
            for j in range(M):
                tj = int(t[c, k, j])
                age = int(now[c]) - tj
                if tj < 0 or age < 0 or age >= window:
                    continue
                num += (window - age) * int(d[c, k, j])
                den += window - age
            want = 0 if den == 0 else int(Fraction(num, den).__floor__())
            assert got[c, k] == want


def test_rejects_bad_arguments():
    t = np.zeros((1, 1, 2), np.int64)
    with pytest.raises(ValueError):
        oracle.queue_delay(np.zeros(1, np.int64), t, np.array([[[1, -1]]], np.int32), W)
    with pytest.raises(ValueError):
        oracle.queue_delay(np.zeros(1, np.int64), t, np.zeros((1, 1, 2), np.int32), 0)
