"""Pins of the oracle's comparison rules and order variants: requests with a known
downstream path (Sec. 5.2, dynamic-path DAGs), arrival order (Table 1 / Sec. 5.3,
PARD-FCFS), Nexus' window scan and Clipper++'s split budgets (Sec. 5.1, Baseline).

Each rule is pinned to a hand-worked example under tests/golden/ and to a
restatement of the paper's sentence in another form (explicit window search,
fixed point over all keep sets), never to the oracle itself.
"""
import itertools

import numpy as np
import pytest

from oracle import oracle
from paper_2602_08747_b200 import inputs
from tests import util

MASK, FCFS, NEXUS, CLIPPER = oracle.MODE_PATH_MASK, oracle.MODE_FCFS, oracle.MODE_NEXUS, oracle.MODE_CLIPPER


def _one_stage(deadline, d=100, B=1, free_at=0, now=0, workers=None, flags=None):
    p = util.pipeline([], 1, [d], bmax=max(B, 1))
    st = util.state(1, 1, 0, now, B, free_at=free_at, workers=workers)
    r = util.requests(deadline)
    if flags is not None:
        r["flags"] = flags
    return inputs.Workload("pin", [p], r, st, 1)


def plan(wl, mode, arrivals=None):
    return oracle.plan(wl.pipelines, wl.requests, wl.state, wl.n_ctx, mode, arrivals)


# --------------------------------------------------------------------------
# known downstream path (Sec. 5.2)
# --------------------------------------------------------------------------
DIAMOND = dict(edges=[(0, 1), (0, 2), (1, 3), (2, 3)], d=[10, 20, 50, 5], q=[1, 2, 3, 4], w=[100, 7, 11, 13])


def test_masked_lsub_diamond_hand_computed():
    p = util.pipeline(DIAMOND["edges"], 4, DIAMOND["d"])
    for stage, mask, want in util.read_golden("diamond_lsub_masked.txt"):
        got = oracle.lsub_masked(p, int(stage), [1] * 4, DIAMOND["q"], DIAMOND["w"], int(mask))
        assert got == int(want), (stage, mask)


@pytest.mark.parametrize("seed", range(6))
def test_masked_lsub_equals_max_over_the_selected_explicit_paths(seed):
    rng = np.random.default_rng(300 + seed)
    S = int(rng.integers(2, 10))
    p = inputs.make_pipeline(inputs.random_dag_edges(rng, S), S, [3] * S,
                             [rng.integers(1, 900, size=3).astype(np.int64) for _ in range(S)])
    R = max(1, inputs.n_slots(p))
    batch, q, w = rng.integers(1, 4, size=S), rng.integers(0, 300, size=S), rng.integers(0, 2000, size=R)
    base = 0
    for k in range(S):
        paths = util.explicit_paths(p, k)
        sums = [sum(int(q[i]) + p.latency(i, int(batch[i])) for i in path) + int(w[base + j])
                for j, path in enumerate(paths)]
        for mask in [0, 1, 2, 3, 5, 0x8000, 0xffff] + [int(x) for x in rng.integers(1, 1 << 16, size=6)]:
            chosen = [s for j, s in enumerate(sums) if j < 16 and (mask >> j) & 1] if mask else sums
            want = 0 if not paths else (max(chosen) if chosen else -1)
            assert oracle.lsub_masked(p, k, batch, q, w, mask) == want, (k, mask)
        base += len(paths)


def test_mask_of_all_paths_or_zero_is_the_plain_plan():
    rng = np.random.default_rng(5)
    wl = util.random_small_workload(rng, 600, n_ctx=2)
    want = plan(wl, 0)
    for flags in (0, 0xffff):
        wl.requests["flags"] = flags
        got = plan(wl, MASK)
        for key in ("keep", "est_us", "perm", "seg_kept"):
            assert np.array_equal(got[key], want[key]), (flags, key)
    # without the mode bit the flags are not looked at
    wl.requests["flags"] = rng.integers(0, 1 << 16, size=wl.n)
    assert np.array_equal(plan(wl, 0)["keep"], want["keep"])


def test_request_on_the_short_branch_is_kept_where_the_unknown_path_is_dropped():
    """Diamond: from stage 0 the branch through 1 costs 131, through 2 only 69.  Deadline 150
    with d_0 = 10 and an idle stage: est = 10 + Lsub."""
    p = util.pipeline(DIAMOND["edges"], 4, DIAMOND["d"])
    st = util.state(1, 4, 4, 0, 1, q=[DIAMOND["q"]], w=[DIAMOND["w"]])
    r = util.requests([100, 100, 100])
    r["flags"] = [0, 1, 2]                       # unknown, long branch, short branch
    o = oracle.plan([p], r, st, 1, MASK)
    assert list(o["perm"]) == [0, 1, 2]
    assert list(o["est_us"]) == [141, 141, 79]   # the third does not queue behind dropped ones
    assert list(o["keep"]) == [0, 0, 1]
    # a mask naming no path of the stage is an input error
    r["flags"] = [0, 4, 2]
    with pytest.raises(ValueError):
        oracle.plan([p], r, st, 1, MASK)


def _fixed_point_keep_sets(order, deadline, A, d, cap):
    """All keep sets K with  r in K  <=>  A_r + floor(#K ahead of r / cap) * d <= deadline_r."""
    n = len(order)
    sols = []
    for bits in itertools.product([0, 1], repeat=n):
        ahead, ok = 0, True
        for pos in range(n):
            i = order[pos]
            fits = A[i] + (ahead // cap) * d <= deadline[i]
            if fits != bool(bits[pos]):
                ok = False
                break
            ahead += bits[pos]
        if ok:
            sols.append(bits)
    return sols


@pytest.mark.parametrize("seed", range(6))
def test_masked_plan_is_the_unique_fixed_point(seed):
    rng = np.random.default_rng(400 + seed)
    p = util.pipeline(DIAMOND["edges"], 4, DIAMOND["d"], bmax=2)
    B = int(rng.integers(1, 3))
    st = util.state(1, 4, 4, 0, B, q=[DIAMOND["q"]], w=[DIAMOND["w"]])
    n = 9
    dl = rng.integers(60, 260, size=n)
    r = util.requests(dl)                        # all at stage 0
    r["flags"] = rng.integers(0, 4, size=n)
    o = oracle.plan([p], r, st, 1, MASK)
    order = sorted(range(n), key=lambda i: (int(dl[i]), i))
    assert list(o["perm"]) == order
    lsub = {0: 131, 1: 131, 2: 69, 3: 131}
    A = [10 + lsub[int(f)] for f in r["flags"]]
    sols = _fixed_point_keep_sets(order, dl, A, 10, B)
    assert sols == [tuple(int(x) for x in o["keep"])]


# --------------------------------------------------------------------------
# arrival order (Table 1: PARD-FCFS drops by arrival order)
# --------------------------------------------------------------------------
def test_fcfs_serves_in_index_order_whatever_the_deadlines():
    d = 37
    n = 12
    dl = 10**9 - np.arange(n)                     # later arrivals have EARLIER deadlines
    o = plan(_one_stage(dl, d=d, B=1, now=5000, free_at=4000), FCFS)
    assert list(o["perm"]) == list(range(n))
    assert list(o["est_us"]) == [5000 + (i + 1) * d for i in range(n)]   # single-server FIFO
    o = plan(_one_stage(dl, d=d, B=1, now=5000, free_at=4000), 0)
    assert list(o["perm"]) == list(range(n))[::-1]


def test_fcfs_orders_every_queue_by_index():
    rng = np.random.default_rng(7)
    wl = util.random_small_workload(rng, 500, n_ctx=3)
    o = plan(wl, FCFS)
    r = wl.requests
    key = sorted(range(wl.n), key=lambda i: (int(r["ctx"][i]), int(r["stage"][i]), i))
    assert list(o["perm"]) == key


@pytest.mark.parametrize("seed", range(8))
def test_fcfs_plan_is_the_unique_fixed_point(seed):
    """Brute force over all 2^n keep sets in arrival order (thresholds are not monotone there)."""
    rng = np.random.default_rng(500 + seed)
    n = 10
    d, B = 20, int(rng.integers(1, 4))
    dl = rng.integers(10, 140, size=n)
    o = plan(_one_stage(dl, d=d, B=B, free_at=3), FCFS)
    sols = _fixed_point_keep_sets(list(range(n)), dl, [3 + d] * n, d, B)
    assert sols == [tuple(int(x) for x in o["keep"])]
    kept_ahead = np.concatenate([[0], np.cumsum(o["keep"])[:-1]])
    assert list(o["est_us"]) == [3 + d + (int(a) // B) * d for a in kept_ahead]


def test_fcfs_keeps_no_more_than_budget_order_on_one_queue():
    """Why the remaining budget matters (Sec. 5.3): earliest-deadline-first admission is maximal."""
    rng = np.random.default_rng(9)
    for _ in range(30):
        dl = rng.integers(0, 400, size=60)
        wl = _one_stage(dl, d=25, B=2)
        assert plan(wl, FCFS)["n_kept"] <= plan(wl, 0)["n_kept"]


# --------------------------------------------------------------------------
# Nexus (Sec. 5.1 Baseline)
# --------------------------------------------------------------------------
def test_nexus_hand_worked_window_example():
    rows = util.read_golden("nexus_window_example.txt")
    dl = [int(r[1]) for r in rows]
    o = plan(_one_stage(dl, d=100, B=2), NEXUS)
    assert list(o["perm"]) == [int(r[0]) for r in rows]
    assert list(o["keep"]) == [int(r[2]) for r in rows]
    assert list(o["est_us"]) == [int(r[3]) for r in rows]
    assert o["n_kept"] == 3 and list(o["kept_idx"]) == [2, 3, 8]


def _nexus_by_window_search(dl, d, W, base):
    """The rule of Sec. 5.1 written as an explicit search: from the scan position on, try every
    window start in turn until all W requests of the window fit the batch that would start now."""
    n = len(dl)
    keep, est = [0] * n, [0] * n
    t, pos = base, 0
    while pos < n:
        p = pos
        while p < n and not all(t + d <= dl[j] for j in range(p, min(p + W, n))):
            p += 1
        for j in range(pos, min(p + W, n)):
            est[j] = t + d
        for j in range(p, min(p + W, n)):
            keep[j] = 1
        pos = min(p + W, n)
        t += d
    return keep, est


@pytest.mark.parametrize("seed", range(10))
def test_nexus_equals_the_explicit_window_search(seed):
    rng = np.random.default_rng(600 + seed)
    n = int(rng.integers(1, 60))
    d, B, m = int(rng.integers(5, 40)), int(rng.integers(1, 5)), int(rng.integers(1, 3))
    dl = rng.integers(0, 30 * d // B + 50, size=n)
    o = plan(_one_stage(dl, d=d, B=B, free_at=11, workers=m), NEXUS)
    keep, est = _nexus_by_window_search([int(x) for x in dl], d, B * m, 11)
    assert list(o["keep"]) == keep
    # the estimate of a dropped request is that of the batch it was tested against; the explicit
    # search assigns the same instant to everything it passes over
    assert list(o["est_us"]) == est


def test_nexus_with_generous_deadlines_is_plain_batching():
    o = plan(_one_stage(10**9 + np.arange(10), d=100, B=4), NEXUS)
    assert o["keep"].all()
    assert list(o["est_us"]) == [100] * 4 + [200] * 4 + [300] * 2


def test_nexus_ignores_downstream_stages():
    """The reactive rule looks at the current module only (Sec. 3): a request that cannot finish
    the pipeline but can finish this module is kept."""
    p = util.pipeline(inputs.chain_edges(3), 3, [10, 500, 500])
    st = util.state(1, 3, inputs.n_slots(p), 0, 1)
    r = util.requests([15, 15], stage=0)
    assert list(oracle.plan([p], r, st, 1, NEXUS)["keep"]) == [1, 0]      # second batch ends at 20
    assert list(oracle.plan([p], r, st, 1, 0)["keep"]) == [0, 0]


# --------------------------------------------------------------------------
# Clipper++ (Sec. 5.1 Baseline)
# --------------------------------------------------------------------------
def test_clipper_split_hand_worked_example():
    rows = util.read_golden("clipper_split_example.txt")
    p = util.pipeline(inputs.chain_edges(3), 3, [100, 300, 600], bmax=1)
    st = util.state(1, 3, inputs.n_slots(p), 0, 1)
    n = len(rows)
    r = util.requests(np.zeros(n), stage=1)      # deadlines play no role in this rule
    a = util.arrivals([int(x[1]) for x in rows], [int(x[2]) for x in rows])
    o = oracle.plan([p], r, st, 1, CLIPPER, a)
    assert list(o["perm"]) == list(range(n))
    assert list(o["keep"]) == [int(x[3]) for x in rows]
    assert list(o["est_us"]) == [int(x[4]) for x in rows]


def test_clipper_shares_add_up_and_follow_the_durations():
    """SLO_k = SLO * d_k / sum d_i: with one module the share is the whole objective, i.e. the
    single-module Clipper rule (a request goes only when its objective is used up at its start)."""
    o = plan(_one_stage(np.zeros(3), d=50, B=1), CLIPPER, util.arrivals([-1000, -1001, -2000], 1000))
    # the first has spent exactly 1000 at its start 0 (kept); the second starts at 50, behind the
    # first, and has spent 1051 by then; the third is long overdue
    assert list(o["keep"]) == [1, 0, 0]
    # shares of a 3-chain at current batch sizes: the module with the longest duration gets the most
    p = inputs.make_pipeline(inputs.chain_edges(3), 3, [2] * 3,
                             [np.array([100, 200]), np.array([300, 350]), np.array([600, 450])])
    for batch, shares in (([1, 1, 1], [100, 300, 600]), ([2, 2, 2], [200, 350, 450])):
        st = util.state(1, 3, inputs.n_slots(p), 0, [batch])
        for k in range(3):
            r = util.requests([0, 0], stage=k)
            a = util.arrivals([-shares[k], -shares[k] - 1], 1000)
            assert list(oracle.plan([p], r, st, 1, CLIPPER, a)["keep"]) == [1, 0], (batch, k)


@pytest.mark.parametrize("seed", range(6))
def test_clipper_plan_is_the_unique_fixed_point(seed):
    rng = np.random.default_rng(700 + seed)
    n = 10
    p = util.pipeline(inputs.chain_edges(2), 2, [30, 70], bmax=3)
    B = int(rng.integers(1, 4))
    st = util.state(1, 2, inputs.n_slots(p), 0, B, free_at=5)
    arrive = rng.integers(-60, 40, size=n)
    slo = rng.integers(50, 400, size=n)
    o = oracle.plan([p], util.requests(np.zeros(n), stage=0), st, 1, CLIPPER, util.arrivals(arrive, slo))
    # keep iff start - arrive <= floor(slo * 30 / 100)  <=>  start + 30 <= arrive + share + 30
    limit = [int(arrive[i]) + (int(slo[i]) * 30) // 100 + 30 for i in range(n)]
    sols = _fixed_point_keep_sets(list(range(n)), limit, [5 + 30] * n, 30, B)
    assert sols == [tuple(int(x) for x in o["keep"])]


def test_rules_that_exclude_each_other_are_rejected():
    wl = _one_stage([100, 200])
    a = util.arrivals([0, 0], 100)
    for mode in (NEXUS | CLIPPER, NEXUS | MASK, CLIPPER | MASK, NEXUS | 1, CLIPPER | 1):
        with pytest.raises(ValueError):
            plan(wl, mode, a)
    with pytest.raises(ValueError):
        plan(wl, CLIPPER, None)
