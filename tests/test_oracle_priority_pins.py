"""Pins of the oracle's adaptive request priority (paper Sec. 4.3): the high
budget first decision order in the planner, and the load factor / fluctuation
bound / delayed transition that choose between the two orders.  Every check
compares the oracle with something other than itself: the paper's two-request
example, hand-computed values (tests/golden), closed forms, brute force over
all keep sets, and exact rational arithmetic with Python fractions."""
from __future__ import annotations

import itertools
from fractions import Fraction

import numpy as np
import pytest

from oracle import oracle
from paper_2602_08747_b200 import inputs
from tests import util


def golden(name):
    rows = util.read_golden(name)
    return rows


# --------------------------------------------------------------------------
# high budget first as a decision order
# --------------------------------------------------------------------------
def test_paper_two_request_example():
    g = {r[0]: r[1:] for r in golden("priority_order_example.txt")}
    d = int(g["d"][0])
    p = util.pipeline([], 1, [d], bmax=1)
    dl = [int(g["deadline_R4"][0]), int(g["deadline_R5"][0])]      # index 0 = R4, index 1 = R5
    for prio, want_kept in ((0, int(g["kept_low_budget_first"][0])), (1, int(g["kept_high_budget_first"][0]))):
        st = util.state(1, 1, 0, 0, 1)
        st.priority = np.array([[prio]], dtype=np.uint8)
        o = oracle.plan([p], util.requests(dl), st, 1)
        assert o["n_kept"] == want_kept
        if prio == 1:
            assert list(o["perm"]) == [1, 0]                       # R5 is served first
            assert list(o["keep"]) == [1, 0]                       # and R4 is the one dropped
            assert g["dropped_high_budget_first"][0] == "R4"
        else:
            assert list(o["perm"]) == [0, 1]


@pytest.mark.parametrize("seed", range(6))
def test_high_budget_first_order_is_rank_by_counting(seed):
    """Position = number of requests of the same queue with a larger deadline,
    or an equal deadline and a smaller index."""
    rng = np.random.default_rng(900 + seed)
    n, S, n_ctx = 60, 3, 2
    p = util.pipeline(inputs.chain_edges(S), S, [7, 5, 3], bmax=2)
    st = util.state(n_ctx, S, 2, 100, 2)
    st.priority = rng.integers(0, 2, size=(n_ctx, S)).astype(np.uint8)
    st.priority[0, 0] = 1
    r = util.requests(rng.integers(90, 130, size=n), stage=rng.integers(0, S, size=n),
                      ctx=rng.integers(0, n_ctx, size=n))
    o = oracle.plan([p], r, st, n_ctx)
    pos = np.empty(n, dtype=np.int64)
    pos[o["perm"]] = np.arange(n)
    for i in range(n):
        seg = int(r["ctx"][i]) * S + int(r["stage"][i])
        hi = st.priority.reshape(-1)[seg] != 0
        ahead = 0
        for j in range(n):
            if int(r["ctx"][j]) * S + int(r["stage"][j]) != seg:
                continue
            dj, di = int(r["deadline_us"][j]), int(r["deadline_us"][i])
            first = dj > di if hi else dj < di
            if first or (dj == di and j < i):
                ahead += 1
        assert pos[i] - o["seg_offsets"][seg] == ahead


def test_high_budget_first_single_server_closed_form():
    """One stage, one request per batch, nothing downstream: served largest
    deadline first, the request at position r completes at now + (r+1)*d while
    every earlier one was kept; the first late request and all after it are
    dropped (their deadlines are no larger, their batch no earlier)."""
    d, now = 10, 1000
    p = util.pipeline([], 1, [d], bmax=1)
    st = util.state(1, 1, 0, now, 1)
    st.priority = np.array([[1]], dtype=np.uint8)
    dl = np.array([1055, 1012, 1031, 1030, 1100, 1005, 1049])
    o = oracle.plan([p], util.requests(dl), st, 1)
    order = sorted(range(len(dl)), key=lambda i: (-dl[i], i))
    assert list(o["perm"]) == order
    kept = 0
    for r, i in enumerate(order):
        on_time = now + (kept + 1) * d <= dl[i]
        assert o["keep"][r] == (1 if on_time else 0)
        assert o["est_us"][r] == now + (kept + 1) * d
        kept += on_time
    keep = list(o["keep"])
    assert keep == sorted(keep, reverse=True)                      # a prefix of the queue


@pytest.mark.parametrize("seed", range(8))
def test_high_budget_first_kept_set_is_the_unique_fixed_point(seed):
    """Brute force over all 2^n keep sets: exactly one set K satisfies
    'r in K <=> the estimate with |K ahead of r| admitted requests meets r's
    deadline', visiting the queue largest deadline first; and no queue keeps
    more under high budget first than under low budget first (earliest
    deadline first admits a largest feasible set)."""
    rng = np.random.default_rng(940 + seed)
    n = int(rng.integers(1, 10))
    d = int(rng.integers(5, 30))
    B = int(rng.integers(1, 4))
    m = int(rng.integers(1, 3))
    p = util.pipeline(inputs.chain_edges(2), 2, [d, 9], bmax=B)
    now, free_at, q1, w0 = 100, int(rng.integers(80, 130)), int(rng.integers(0, 9)), int(rng.integers(0, 9))
    st = util.state(1, 2, 1, now, [[B, 1]], free_at=[[free_at, 0]], q=[[0, q1]], w=[[w0]], workers=[[m, 1]])
    dl = rng.integers(100, 100 + 12 * d, size=n)
    low = oracle.plan([p], util.requests(dl, stage=0), st, 1)
    st.priority = np.array([[1, 0]], dtype=np.uint8)
    o = oracle.plan([p], util.requests(dl, stage=0), st, 1)
    order = sorted(range(n), key=lambda i: (-int(dl[i]), i))
    base, lsub = max(now, free_at), q1 + 9 + w0

    def est(ahead):
        return base + (ahead // (B * m)) * d + d + lsub

    consistent = []
    for bits in itertools.product([0, 1], repeat=n):
        ahead, ok = 0, True
        for r in range(n):
            if bool(bits[r]) != (est(ahead) <= dl[order[r]]):
                ok = False
                break
            ahead += bits[r]
        if ok:
            consistent.append(bits)
    assert len(consistent) == 1
    assert list(consistent[0]) == list(o["keep"])
    assert list(o["perm"]) == order
    assert o["n_kept"] <= low["n_kept"]


def test_priority_is_per_queue_and_null_means_low_budget_first():
    rng = np.random.default_rng(7)
    wl = util.random_small_workload(rng, 200, n_ctx=3)
    a = oracle.plan(wl.pipelines, wl.requests, wl.state, wl.n_ctx)
    wl.state.priority = np.zeros((wl.n_ctx, wl.state.stage_stride), dtype=np.uint8)
    b = oracle.plan(wl.pipelines, wl.requests, wl.state, wl.n_ctx)
    for k in ("keep", "est_us", "perm", "kept_idx"):
        assert np.array_equal(a[k], b[k])
    # flipping one queue changes only that queue's rows
    wl.state.priority[1, 0] = 1
    c = oracle.plan(wl.pipelines, wl.requests, wl.state, wl.n_ctx)
    seg = 1 * wl.state.stage_stride + 0
    lo, hi = int(a["seg_offsets"][seg]), int(a["seg_offsets"][seg + 1])
    assert np.array_equal(a["perm"][:lo], c["perm"][:lo]) and np.array_equal(a["perm"][hi:], c["perm"][hi:])
    assert np.array_equal(a["keep"][:lo], c["keep"][:lo]) and np.array_equal(a["keep"][hi:], c["keep"][hi:])
    assert sorted(a["perm"][lo:hi]) == sorted(c["perm"][lo:hi])


# --------------------------------------------------------------------------
# load factor, fluctuation bound, delayed transition
# --------------------------------------------------------------------------
def _one_queue(d, B=1, bmax=4):
    return util.pipeline([], 1, [d], bmax=bmax)


def _update(p, x, window, interval, B, prev, workers=None, n_ctx=1, S=1, poc=None, pipes=None):
    x = np.asarray(x, dtype=np.uint32).reshape(n_ctx, S, -1)
    return oracle.update_priority(pipes or [p], poc, n_ctx, S, np.full((n_ctx, S), B, np.int32)
                                  if np.isscalar(B) else B, workers, x, window, interval,
                                  np.full((n_ctx, S), prev, np.uint8) if np.isscalar(prev) else prev)


def test_hand_computed_eps_example():
    rows = golden("priority_eps_example.txt")
    g = {r[0]: r[1:] for r in rows if r[0] != "case"}
    x = [int(v) for v in g["arrivals"]]
    W, tau = int(g["window"][0]), int(g["interval_us"][0])
    # the fixture's own arithmetic
    ts = [Fraction(sum(x[j - W + 1:j + 1]), W) for j in range(W - 1, len(x))]
    dev = sum(abs(x[j] - ts[j - W + 1]) for j in range(W - 1, len(x)))
    assert dev / sum(x[W - 1:]) == Fraction(int(g["eps_num"][0]), int(g["eps_den"][0]))
    for r in rows:
        if r[0] != "case":
            continue
        d, want0, want1 = int(r[1]), int(r[3]), int(r[4])
        p = _one_queue(d)
        assert _update(p, x, W, tau, 1, 0)[0, 0] == want0, r
        assert _update(p, x, W, tau, 1, 1)[0, 0] == want1, r


@pytest.mark.parametrize("B,m", [(1, 1), (4, 1), (2, 3)])
def test_steady_workload_has_no_band(B, m):
    """Constant input: T_s = T_in, eps = 0, so the priority follows mu > 1 / mu < 1
    and only mu == 1 exactly keeps the old one.  mu = a*d / (B*m*tau)."""
    d, tau = 50, 1000
    p = _one_queue(d, bmax=4)
    workers = np.full((1, 1), m, np.int32)
    for a in range(1, 200):
        num, den = a * d, B * m * tau
        for prev in (0, 1):
            got = _update(p, [a] * 6, 3, tau, B, prev, workers=workers)[0, 0]
            want = 1 if num > den else (0 if num < den else prev)
            assert got == want, (a, prev)


def test_no_arrivals_is_low_budget_first_and_padding_is_untouched():
    p = _one_queue(10)
    assert _update(p, [0, 0, 0, 0], 2, 1000, 1, 1)[0, 0] == 0
    # samples before the first full window do not count: 9 arrives only there
    assert _update(p, [9, 0, 0], 2, 1000, 1, 1)[0, 0] == 0
    # a stage column the pipeline lacks keeps whatever was there
    x = np.zeros((1, 3, 4), np.uint32)
    out = oracle.update_priority([p], None, 1, 3, np.ones((1, 3), np.int32), None, x, 2, 1000,
                                 np.array([[1, 7, 9]], np.uint8))
    assert list(out[0]) == [0, 7, 9]


def test_delayed_transition_follows_a_ramp():
    """A slowly rising then falling load: the order flips to high budget first
    only above 1 + eps and back only below 1 - eps (never at the crossing of 1)."""
    d, tau, W, H = 100, 1000, 4, 12
    p = _one_queue(d)
    rng = np.random.default_rng(5)
    load = np.concatenate([np.linspace(4, 16, 60), np.linspace(16, 4, 60)])
    series = np.maximum(0, np.rint(load + rng.normal(0, 1.5, size=load.size))).astype(np.int64)
    prio, flips = 0, []
    for t in range(H, len(series)):
        x = series[t - H:t]
        ts = [Fraction(int(sum(x[j - W + 1:j + 1])), W) for j in range(W - 1, H)]
        sx = int(sum(x[W - 1:]))
        eps = sum(abs(int(x[j]) - ts[j - W + 1]) for j in range(W - 1, H)) / sx
        mu = Fraction(int(x[-1]) * d, tau)
        want = 1 if mu > 1 + eps else (0 if mu < 1 - eps else prio)
        got = int(_update(p, x, W, tau, 1, prio)[0, 0])
        assert got == want
        if got != prio:
            flips.append((t, got, float(mu), float(eps)))
            assert (mu > 1) == (got == 1)
        prio = got
    assert [f[1] for f in flips][:1] == [1] and 0 in [f[1] for f in flips]   # it went up and came back


@pytest.mark.parametrize("seed", range(12))
def test_exact_rational_arithmetic(seed):
    """The definition evaluated with Python fractions, including values at the
    top of the allowed ranges (no overflow in the cross-multiplied form)."""
    rng = np.random.default_rng(1200 + seed)
    big = seed % 3 == 0
    S, n_ctx = 3, 4
    H = int(rng.integers(1, 40))
    W = int(rng.integers(1, H + 1))
    bmax = 4096 if big else 8
    tables = [rng.integers((1 << 39) if big else 1, (1 << 40) if big else 400, size=bmax).astype(np.int64)
              for _ in range(S)]
    p = inputs.make_pipeline(inputs.chain_edges(S), S, [bmax] * S, tables)
    B = rng.integers(1, bmax + 1, size=(n_ctx, S)).astype(np.int32)
    m = rng.integers(1, (1 << 18) if big else 4, size=(n_ctx, S)).astype(np.int32)
    tau = int(rng.integers(1 << 30, 1 << 31)) if big else int(rng.integers(1, 5000))
    hi = (1 << 24) if big else 50
    x = rng.integers(0, hi, size=(n_ctx, S, H)).astype(np.uint32)
    if not big:
        x[0, 0] = 0
    prev = rng.integers(0, 2, size=(n_ctx, S)).astype(np.uint8)
    got = oracle.update_priority([p], None, n_ctx, S, B, m, x, W, tau, prev)
    for c in range(n_ctx):
        for k in range(S):
            xs = [int(v) for v in x[c, k]]
            sx = sum(xs[W - 1:])
            if sx == 0:
                want = 0
            else:
                ts = {j: Fraction(sum(xs[j - W + 1:j + 1]), W) for j in range(W - 1, H)}
                eps = sum(abs(xs[j] - ts[j]) for j in range(W - 1, H)) / sx
                t_m = Fraction(int(B[c, k]) * int(m[c, k]), p.latency(k, int(B[c, k])))
                mu = Fraction(xs[-1], tau) / t_m
                want = 1 if mu > 1 + eps else (0 if mu < 1 - eps else int(prev[c, k]))
            assert got[c, k] == want, (c, k)


def test_update_priority_rejects_bad_arguments():
    p = _one_queue(10)
    x = np.ones((1, 1, 4), np.uint32)
    ok = dict(pipelines=[p], pipeline_of_ctx=None, n_ctx=1, stage_stride=1, batch=np.ones((1, 1), np.int32),
              workers=None, arrivals=x, window=2, interval_us=1000, priority=np.zeros((1, 1), np.uint8))
    oracle.update_priority(**ok)
    for bad in (dict(window=0), dict(window=5), dict(interval_us=0), dict(batch=np.full((1, 1), 9, np.int32)),
                dict(workers=np.zeros((1, 1), np.int32)), dict(pipeline_of_ctx=np.array([1], np.int32))):
        with pytest.raises(ValueError):
            oracle.update_priority(**{**ok, **bad})
