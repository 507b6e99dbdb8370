"""Pins of the oracle's batch-wait estimate w = F^{-1}(lambda) (Sec. 4.2, Batch
wait estimation) against the paper's worked example, the Irwin-Hall closed
form, exact special cases and an exhaustive enumeration on tiny inputs."""
import math

import numpy as np
import pytest

from oracle import oracle
from paper_2602_08747_b200 import inputs
from tests import util

M_PAPER = 10_000           # sample count of the paper's Overheads paragraph


def uniform_grid(n_ctx, S, M, d):
    """Recorded batch waits spread evenly over [0, d): the arrival process of the
    worked example (a request is equally likely to arrive anywhere in a batch)."""
    return np.tile((np.arange(M, dtype=np.int64) * d // M).astype(np.int32), (n_ctx, S, 1))


def irwin_hall_cdf(n, x):
    return sum((-1) ** k * math.comb(n, k) * (x - k) ** n for k in range(int(math.floor(x)) + 1)) / math.factorial(n)


def irwin_hall_quantile(n, lam):
    lo, hi = 0.0, float(n)
    for _ in range(80):
        mid = 0.5 * (lo + hi)
        if irwin_hall_cdf(n, mid) < lam:
            lo = mid
        else:
            hi = mid
    return 0.5 * (lo + hi)


def test_worked_example_values():
    """Sec. 4.2 worked example: lambda = 0.1, equal durations d; the estimate over
    4, 3, 2, 1 subsequent modules is 1.24d, 0.84d, 0.44d, 0.10d."""
    d = 100_000
    rows = util.read_golden("w_worked_example.txt")
    p = util.pipeline(inputs.chain_edges(5), 5, [d] * 5)
    w = oracle.estimate_w([p], None, 1, 5, 4, uniform_grid(1, 5, M_PAPER, d), 1, 10, seed=2602)
    for k in range(4):
        covered, _, val = rows[k]
        assert int(covered) == 4 - k
        # the paper prints two decimals; the Monte Carlo error at M = 10,000 is below 0.01 d per module
        assert abs(w[0, k] / d - float(val)) < 0.005 + 0.012 * int(covered), (k, w[0, k])


@pytest.mark.parametrize("lam_num", [1, 3, 5, 9])
def test_quantiles_follow_irwin_hall(lam_num):
    """The sum of n independent uniform batch waits is Irwin-Hall distributed."""
    d = 1_000_000
    p = util.pipeline(inputs.chain_edges(7), 7, [d] * 7)
    w = oracle.estimate_w([p], None, 1, 7, 6, uniform_grid(1, 7, M_PAPER, d), lam_num, 10, seed=lam_num)
    for k in range(6):
        n = 6 - k
        sd = math.sqrt(n / 12.0)
        assert abs(w[0, k] / d - irwin_hall_quantile(n, lam_num / 10)) < 0.05 * sd + 0.01, (k, n)


def test_lambda_bounds():
    """lambda = 0 gives (nearly) no wait, lambda = 1 (nearly) the summed durations,
    and the estimate is monotone in lambda (Sec. 4.2)."""
    d = 1000
    p = util.pipeline(inputs.chain_edges(4), 4, [d] * 4)
    ws = uniform_grid(1, 4, 2000, d)
    prev = None
    for num in range(0, 11):
        w = oracle.estimate_w([p], None, 1, 4, 3, ws, num, 10, seed=5)[0]
        if prev is not None:
            assert (w >= prev).all()
        prev = w
    lo = oracle.estimate_w([p], None, 1, 4, 3, ws, 0, 10, seed=5)[0]
    hi = oracle.estimate_w([p], None, 1, 4, 3, ws, 10, 10, seed=5)[0]
    assert (lo >= 0).all() and lo[2] < 0.01 * d and lo[0] < 0.5 * d
    assert hi[2] > 0.99 * d and hi[2] < d and 2.5 * d < hi[0] < 3 * d


def test_constant_waits_are_exact():
    """If every recorded wait of stage i equals v_i, every sample of a path sums
    to the same value and w is that sum whatever the random picks were."""
    rng = np.random.default_rng(3)
    S = 9
    edges = inputs.random_dag_edges(rng, S)
    p = util.pipeline(edges, S, [10] * S)
    R = inputs.n_slots(p)
    v = rng.integers(0, 5000, size=(2, S))
    ws = np.repeat(v[:, :, None], 37, axis=2).astype(np.int32)
    w = oracle.estimate_w([p], None, 2, S, R, ws, 1, 3, seed=11)
    for c in range(2):
        slot = 0
        for k in range(S):
            for path in util.explicit_paths(p, k):
                assert w[c, slot] == sum(int(v[c, i]) for i in path)
                slot += 1
        assert slot == R


def _splitmix64(x):
    mask = (1 << 64) - 1
    z = (x + 0x9E3779B97F4A7C15) & mask
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & mask
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & mask
    return z ^ (z >> 31)


def test_splitmix64_published_vector():
    """First outputs of splitmix64 seeded with 0 (the generator's published test
    vector: the state advances by the golden-ratio constant each draw)."""
    gamma = 0x9E3779B97F4A7C15
    assert [_splitmix64(i * gamma) for i in range(3)] == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]


@pytest.mark.parametrize("seed", range(4))
def test_small_cases_by_enumeration(seed):
    """Tiny M on a random DAG: the samples are written out one by one with an
    independent splitmix64, sorted, and the rank floor(lambda M) element taken."""
    rng = np.random.default_rng(40 + seed)
    S = int(rng.integers(2, 7))
    n_ctx = 3
    M = int(rng.integers(1, 12))
    edges = inputs.random_dag_edges(rng, S)
    p = util.pipeline(edges, S, [10] * S)
    R = inputs.n_slots(p)
    stride_R = R + 2                                     # padded slot stride
    ws = rng.integers(0, 1000, size=(n_ctx, S, M)).astype(np.int32)
    num, den = int(rng.integers(0, 8)), 7
    sd = int(rng.integers(0, 2**63))
    w = oracle.estimate_w([p], None, n_ctx, S, stride_R, ws, num, den, seed=sd)
    rank = min(M - 1, num * M // den)
    for c in range(n_ctx):
        slot = 0
        for k in range(S):
            for path in util.explicit_paths(p, k):
                sums = []
                for m in range(M):
                    tot = 0
                    for j, i in enumerate(path):
                        counter = (sd + (((c * stride_R + slot) * M + m) * 64 + j)) & ((1 << 64) - 1)
                        idx = ((_splitmix64(counter) >> 32) * M) >> 32
                        tot += int(ws[c, i, idx])
                    sums.append(tot)
                assert w[c, slot] == sorted(sums)[rank], (c, k, slot)
                slot += 1


def test_rejects_bad_arguments():
    p = util.pipeline(inputs.chain_edges(2), 2, [5, 5])
    ws = np.zeros((1, 2, 4), np.int32)
    with pytest.raises(ValueError):
        oracle.estimate_w([p], None, 1, 2, 1, ws, 2, 1)          # lambda > 1
    with pytest.raises(ValueError):
        oracle.estimate_w([p], None, 1, 2, 1, ws, 1, 0)          # zero denominator
