"""Parity of pard_update_queue_delay (the State Planner's sliding-window
average queueing delay, paper Sec. 4.2) with the CPU oracle, bit for bit."""
import numpy as np
import pytest

from oracle import oracle
from paper_2602_08747_b200 import binding as pb
from tests.gpu_util import run_queue_delay

pytestmark = pytest.mark.gpu


def draw(rng, n_ctx, S, M, window, big=False):
    now = rng.integers(10**9, 2 * 10**9, size=n_ctx)
    t = now[:, None, None] - rng.integers(-window // 4, 2 * window + 1, size=(n_ctx, S, M))
    t[rng.random(size=t.shape) < 0.1] = -1
    lo = (1 << 24) - 1000 if big else 0
    d = rng.integers(lo, 1 << 24, size=(n_ctx, S, M)).astype(np.int32)
    return now, t, d


@pytest.mark.parametrize("M", [0, 1, 2, 31, 64, 65, 1000, 4097, 1 << 15])
@pytest.mark.parametrize("window", [1, 5_000_000, 1 << 24])
def test_matches_the_oracle(M, window):
    rng = np.random.default_rng(M * 3 + window % 1000)
    n_ctx, S = 21, 5
    now, t, d = draw(rng, n_ctx, S, M, window, big=(window == 1 << 24))
    if M >= 31:
        t[0, 0, :] = now[0] - rng.integers(0, max(1, window // 2), size=M)   # a row with every sample in the window
        t[1, 1, :] = -1                                                   # an empty row
    want = oracle.queue_delay(now, t, d, window)
    rc, got = run_queue_delay(now, t, d, window)
    assert rc == 0
    assert np.array_equal(got, want)
    if M >= 31 and window > 1:
        assert (got > 0).any() and got[1, 1] == 0


def test_many_rows():
    rng = np.random.default_rng(5)
    now, t, d = draw(rng, 4096, 8, 50, 5_000_000)
    want = oracle.queue_delay(now, t, d, 5_000_000)
    rc, got = run_queue_delay(now, t, d, 5_000_000)
    assert rc == 0 and np.array_equal(got, want)


def test_largest_sums_do_not_overflow():
    """Every sample at age 0 with the largest delay and the longest window."""
    M, window = 1 << 15, 1 << 24
    now = np.array([10**12], np.int64)
    t = np.full((1, 1, M), 10**12, np.int64)
    d = np.full((1, 1, M), (1 << 24) - 1, np.int32)
    rc, got = run_queue_delay(now, t, d, window)
    assert rc == 0 and got[0, 0] == (1 << 24) - 1 == oracle.queue_delay(now, t, d, window)[0, 0]


def test_reports_a_delay_out_of_range():
    now = np.array([1000], np.int64)
    t = np.full((1, 2, 4), 900, np.int64)
    d = np.full((1, 2, 4), 5, np.int32)
    assert run_queue_delay(now, t, d, 1000)[0] == 0
    d[0, 1, 2] = 1 << 24
    assert run_queue_delay(now, t, d, 1000, check=False)[0] == pb.PARD_EDATA
    d[0, 1, 2] = -3
    assert run_queue_delay(now, t, d, 1000, check=False)[0] == pb.PARD_EDATA
    t[0, 1, 2] = -1                                          # an empty slot's delay is never looked at
    assert run_queue_delay(now, t, d, 1000, check=False)[0] == 0
