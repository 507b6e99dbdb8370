"""Pins of the CPU oracle against what the paper and the mathematics fix.

Each test names the passage or fact it pins.  None of them compares the oracle
with itself or with the CUDA library.
"""
import itertools

import numpy as np
import pytest

from oracle import oracle
from paper_2602_08747_b200 import inputs
from tests import util


def plan(wl, mode=0):
    return oracle.plan(wl.pipelines, wl.requests, wl.state, wl.n_ctx, mode)


# --------------------------------------------------------------------------
# order (Sec. 4.3: smallest remaining budget first; ties by index)
# --------------------------------------------------------------------------
@pytest.mark.parametrize("seed", range(5))
def test_order_is_rank_by_counting(seed):
    rng = np.random.default_rng(seed)
    n = 64
    p = util.pipeline(inputs.chain_edges(3), 3, [5, 6, 7])
    st = util.state(2, 3, inputs.n_slots(p), 100, 2)
    r = util.requests(rng.integers(0, 12, size=n), stage=rng.integers(0, 3, size=n),
                      ctx=rng.integers(0, 2, size=n))
    o = oracle.plan([p], r, st, 2)
    # position of request i = number of requests that must come before it
    key = [(int(r["ctx"][i]), int(r["stage"][i]), int(r["deadline_us"][i]), i) for i in range(n)]
    for i in range(n):
        rank = sum(1 for j in range(n) if key[j] < key[i])
        assert o["perm"][rank] == i
    # segment offsets are the counts of smaller (ctx, stage)
    for c in range(2):
        for k in range(3):
            want = sum(1 for j in range(n) if (key[j][0], key[j][1]) < (c, k))
            assert o["seg_offsets"][c * 3 + k] == want
    assert o["seg_offsets"][-1] == n


# --------------------------------------------------------------------------
# L_sub (Eq. 3 State Planner part; DAG: max over subsequent paths)
# --------------------------------------------------------------------------
def test_lsub_diamond_hand_computed():
    p = util.pipeline([(0, 1), (0, 2), (1, 3), (2, 3)], 4, [10, 20, 50, 5])
    batch = [1, 1, 1, 1]
    q = [1, 2, 3, 4]
    w = [100, 7, 11, 13]
    for stage, want in util.read_golden("diamond_lsub.txt"):
        assert oracle.lsub(p, int(stage), batch, q, w) == int(want)
    assert [oracle.count_paths(p, k) for k in range(4)] == [2, 1, 1, 0]
    assert [oracle.slot_base(p, k) for k in range(4)] == [0, 2, 3, 4]


def test_lsub_chain_uses_paper_w_values():
    """Sec. 4.2 worked example: with equal durations d the estimate over 4, 3,
    2, 1 subsequent modules is 1.24d, 0.84d, 0.44d, 0.10d; for a chain
    L_sub = sum q_i + sum d_i + w_k (Eq. 3)."""
    d = 1000
    rows = util.read_golden("w_worked_example.txt")
    p = util.pipeline(inputs.chain_edges(5), 5, [d] * 5)
    q = [3, 5, 7, 11, 13]
    w = []
    for k in range(4):              # stage k has 4-k modules after it, one path each
        covered, frac, val = rows[k]
        assert int(covered) == 4 - k
        assert abs(float(frac) * int(covered) - float(val)) < 0.011
        w.append(int(round(float(val) * d)))
    assert w == [1240, 840, 440, 100]
    for k in range(5):
        want = 0 if k == 4 else sum(q[k + 1:]) + d * (4 - k) + w[k]
        assert oracle.lsub(p, k, [1] * 5, q, w) == want


@pytest.mark.parametrize("seed", range(8))
def test_lsub_equals_max_over_explicit_paths(seed):
    rng = np.random.default_rng(100 + seed)
    S = int(rng.integers(2, 13))
    edges = inputs.random_dag_edges(rng, S)
    bmax = 6
    tables = [rng.integers(1, 1000, size=bmax).astype(np.int64) for _ in range(S)]
    p = inputs.make_pipeline(edges, S, [bmax] * S, tables)
    R = inputs.n_slots(p)
    batch = rng.integers(1, bmax + 1, size=S)
    q = rng.integers(0, 500, size=S)
    w = rng.integers(0, 2000, size=max(R, 1))
    base = 0
    for k in range(S):
        paths = util.explicit_paths(p, k)
        assert oracle.count_paths(p, k) == len(paths)
        assert oracle.slot_base(p, k) == base
        want = 0
        if paths:
            want = max(sum(int(q[i]) + p.latency(i, int(batch[i])) for i in path) + int(w[base + j])
                       for j, path in enumerate(paths))
        assert oracle.lsub(p, k, batch, q, w) == want
        base += len(paths)
    assert base == R


def test_lsub_single_path_is_chain_sum_and_sink_is_zero():
    p = inputs.make_pipeline(inputs.chain_edges(4), 4, [3] * 4,
                             [np.array([10, 20, 30]), np.array([1, 2, 3]),
                              np.array([100, 200, 300]), np.array([7, 8, 9])])
    batch = [1, 2, 3, 1]
    q = [1000, 2000, 3000, 4000]
    assert oracle.lsub(p, 3, batch, q, None) == 0
    assert oracle.lsub(p, 2, batch, q, None) == 4000 + 7
    assert oracle.lsub(p, 1, batch, q, None) == (3000 + 300) + (4000 + 7)
    assert oracle.lsub(p, 0, batch, q, None) == (2000 + 2) + (3000 + 300) + (4000 + 7)
    # the profile is read at the CURRENT batch size of each stage
    assert oracle.lsub(p, 0, [1, 3, 1, 3], q, None) == (2000 + 3) + (3000 + 100) + (4000 + 9)


# --------------------------------------------------------------------------
# wait / estimate (Sec. 4.2 Request Broker: t_e, W_k, D_k)
# --------------------------------------------------------------------------
def test_fifo_single_server_completion_times():
    """One stage, batch 1, idle server, generous deadlines: the request at
    position p completes at now + (p+1)*d (deterministic single-server FIFO)."""
    d = 37
    p = util.pipeline([], 1, [d], bmax=1)
    now = 5000
    st = util.state(1, 1, 0, now, 1, free_at=now - 10)
    n = 20
    r = util.requests(10**9 + np.arange(n))
    o = oracle.plan([p], r, st, 1)
    assert o["keep"].all()
    assert list(o["est_us"]) == [now + (i + 1) * d for i in range(n)]
    # busy server: everything shifts by the remaining time of the running batch
    st = util.state(1, 1, 0, now, 1, free_at=now + 11)
    o = oracle.plan([p], r, st, 1)
    assert list(o["est_us"]) == [now + 11 + (i + 1) * d for i in range(n)]


def test_batches_of_B_share_a_start_time():
    d, B = 100, 4
    p = util.pipeline([], 1, [d], bmax=B)
    st = util.state(1, 1, 0, 0, B, free_at=0)
    r = util.requests(10**6 + np.arange(10))
    o = oracle.plan([p], r, st, 1)
    assert list(o["est_us"]) == [100] * 4 + [200] * 4 + [300] * 2
    # two identical workers: a round starts 2*B requests
    st = util.state(1, 1, 0, 0, B, free_at=0, workers=2)
    o = oracle.plan([p], r, st, 1)
    assert list(o["est_us"]) == [100] * 8 + [200] * 2


def test_duration_is_the_profile_at_the_current_batch_size():
    """D_k = d_k at the current batch size (Sec. 4.2 Request Broker, third
    bullet), for the stage itself as well as downstream."""
    p = inputs.make_pipeline([], 1, [4], [np.array([100, 150, 200, 250])])
    r = util.requests(10**6 + np.arange(7))
    for B, d in ((1, 100), (3, 200), (4, 250)):
        st = util.state(1, 1, 0, 0, B, free_at=0)
        o = oracle.plan([p], r, st, 1)
        assert list(o["est_us"]) == [d * (i // B + 1) for i in range(7)]


def test_drop_wrong_set_example():
    """Sec. 3.2 Observation #2: W = t_e - t_b; and a dropped request takes no
    batch slot, so dropping R1..R4 lets R5..R8 ride the first batch."""
    g = {k: float(v) for k, v in util.read_golden("drop_wrong_set.txt")}
    d = 8000
    B = int(g["batch_size"])
    n = int(g["n_requests"])
    arrival = np.array([(i + 0.5) / n * d for i in range(n)]).astype(np.int64)
    assert abs(arrival[:4].mean() / d - g["mean_arrival_R1_4"]) < 1e-9
    assert abs(arrival[4:].mean() / d - g["mean_arrival_R5_8"]) < 1e-9
    p = util.pipeline([], 1, [d], bmax=B)
    t_e = int(g["t_e"] * d)
    st = util.state(1, 1, 0, 0, B, free_at=t_e)
    slo = 10 * d
    # arrival order == deadline order (equal SLO): R1..R4 form the first batch
    o = oracle.plan([p], util.requests(arrival + slo), st, 1)
    start = o["est_us"] - d                       # est = t_e + d_k
    wait = start - arrival[o["perm"]]
    assert list(o["perm"]) == list(range(n))
    assert abs(wait[:4].mean() / d - g["mean_wait_R1_4"]) < 1e-9
    # R1..R4 cannot make it (deadline already behind t_e + d): they are dropped
    # and R5..R8 start at t_e, waiting 0.25 d on average
    deadline = arrival + slo
    deadline[:4] = t_e + d - 1
    o = oracle.plan([p], util.requests(deadline), st, 1)
    assert list(o["keep"]) == [0] * 4 + [1] * 4
    start = o["est_us"] - d
    wait = (start - arrival[o["perm"]])[4:]
    assert abs(wait.mean() / d - g["mean_wait_R5_8"]) < 1e-9


# --------------------------------------------------------------------------
# drop rule (Sec. 5.3: compare the estimate with the overall objective)
# --------------------------------------------------------------------------
def test_empty_system_keeps_any_request_with_slack():
    """One request, idle stages, q = w = 0: kept iff now + d_k + (longest
    downstream path of durations) <= deadline; equality is kept."""
    p = util.pipeline([(0, 1), (0, 2), (1, 3), (2, 3)], 4, [10, 20, 50, 5])
    now = 1000
    st = util.state(1, 4, inputs.n_slots(p), now, 1, free_at=0)
    longest = {0: 10 + 50 + 5, 1: 20 + 5, 2: 50 + 5, 3: 5}
    for k in range(4):
        for slack in (-1, 0, 1, 1000):
            r = util.requests([now + longest[k] + slack], stage=k)
            o = oracle.plan([p], r, st, 1)
            assert o["est_us"][0] == now + longest[k]
            assert bool(o["keep"][0]) == (slack >= 0)


def test_sink_stage_is_the_reactive_rule():
    """L_sub = 0 at the last stage: drop iff the remaining budget at batch
    start is below the execution duration (Sec. 2, reactive policies)."""
    d = 40
    p = util.pipeline(inputs.chain_edges(2), 2, [999, d], bmax=2)
    now = 500
    st = util.state(1, 2, 1, now, 2, free_at=[[0, 520]], q=[[77, 88]], w=[[55]])
    dl = np.array([555, 559, 560, 561, 600, 601, 640])
    o = oracle.plan([p], util.requests(dl, stage=1), st, 1)
    kept = 0
    for j in range(len(dl)):
        t_e = 520 + (kept // 2) * d
        remaining = dl[j] - t_e
        assert bool(o["keep"][j]) == (remaining >= d)
        kept += int(o["keep"][j])


def _kept_ahead(o):
    """Kept requests ahead of each position inside its own queue."""
    so = o["seg_offsets"].astype(np.int64)
    out = np.zeros(len(o["keep"]), dtype=np.int64)
    for s in range(len(so) - 1):
        k = o["keep"][so[s]:so[s + 1]].astype(np.int64)
        out[so[s]:so[s + 1]] = np.cumsum(k) - k
    return out


@pytest.mark.parametrize("seed", range(6))
def test_monotonicity(seed):
    """The number of requests admitted among the first r of a queue can only
    grow when every deadline of the queue grows, and can only shrink when the
    clock, the running batch, or a downstream q / w estimate grows.  (A single
    request may still flip the other way: an earlier request that is now kept
    takes a batch slot.)"""
    rng = np.random.default_rng(200 + seed)
    wl = util.random_small_workload(rng, 200, n_ctx=2)
    o = plan(wl)
    so = o["seg_offsets"]
    for s in range(len(so) - 1):       # est never decreases along a queue
        e = o["est_us"][so[s]:so[s + 1]]
        assert (np.diff(e) >= 0).all()
    wl2 = inputs.Workload("x", wl.pipelines, wl.requests.copy(), wl.state, wl.n_ctx)
    wl2.requests["deadline_us"] += 25
    o2 = plan(wl2)
    assert (o2["perm"] == o["perm"]).all()
    assert (_kept_ahead(o2) >= _kept_ahead(o)).all()
    assert (o2["seg_kept"] >= o["seg_kept"]).all()
    for field in ("now_us", "free_at_us", "q_us", "w_us"):
        st = wl.state
        bumped = inputs.QueueState(st.stage_stride, st.slot_stride, st.now_us.copy(),
                                   st.batch, st.free_at_us.copy(), st.q_us.copy(),
                                   st.w_us.copy(), st.workers, st.pipeline_of_ctx)
        getattr(bumped, field)[...] += rng.integers(0, 30, size=getattr(bumped, field).shape)
        o3 = oracle.plan(wl.pipelines, wl.requests, bumped, wl.n_ctx)
        assert (_kept_ahead(o3) <= _kept_ahead(o)).all(), field
        assert (o3["seg_kept"] <= o["seg_kept"]).all(), field


@pytest.mark.parametrize("seed", range(6))
def test_raw_position_mode_is_never_more_lenient(seed):
    rng = np.random.default_rng(300 + seed)
    wl = util.random_small_workload(rng, 300, n_ctx=2)
    a, r = plan(wl, 0), plan(wl, 1)
    assert (a["perm"] == r["perm"]).all()
    assert (r["keep"] <= a["keep"]).all()
    assert (a["est_us"] <= r["est_us"]).all()


@pytest.mark.parametrize("seed", range(12))
def test_kept_set_is_the_unique_fixed_point_and_maximal(seed):
    """Brute force over all 2^n keep-sets of one queue.  A set K is consistent
    when r in K <=> the estimate of r, with the members of K ahead of it taking
    the batch slots, meets r's deadline.  Exactly one set is consistent, it is
    the oracle's, and no feasible set (all members on time when only members
    are served, in deadline order) is larger."""
    rng = np.random.default_rng(400 + seed)
    n = int(rng.integers(1, 11))
    d = int(rng.integers(5, 30))
    B = int(rng.integers(1, 4))
    m = int(rng.integers(1, 3))
    p = util.pipeline(inputs.chain_edges(2), 2, [d, 9], bmax=B)
    now, free_at, q1, w0 = 100, int(rng.integers(80, 130)), int(rng.integers(0, 9)), int(rng.integers(0, 9))
    st = util.state(1, 2, 1, now, [[B, 1]], free_at=[[free_at, 0]], q=[[0, q1]], w=[[w0]],
                    workers=[[m, 1]])
    dl = np.sort(rng.integers(100, 100 + 12 * d, size=n))
    o = oracle.plan([p], util.requests(dl, stage=0), st, 1)
    lsub = q1 + 9 + w0
    base = max(now, free_at)

    def est(ahead):
        return base + (ahead // (B * m)) * d + d + lsub

    consistent, best_feasible = [], 0
    for bits in itertools.product([0, 1], repeat=n):
        ahead, ok, feas = 0, True, True
        for r in range(n):
            on_time = est(ahead) <= dl[r]
            if bool(bits[r]) != on_time:
                ok = False
            if bits[r] and not on_time:
                feas = False
            ahead += bits[r]
        if ok:
            consistent.append(bits)
        if feas:
            best_feasible = max(best_feasible, sum(bits))
    assert len(consistent) == 1
    assert list(consistent[0]) == list(o["keep"])
    assert best_feasible == o["n_kept"]


# --------------------------------------------------------------------------
# the scan form of the broker loop (used by a parallel implementation)
# --------------------------------------------------------------------------
@pytest.mark.parametrize("seed", range(10))
def test_prefix_min_form_equals_the_loop(seed):
    """With thresholds u_r = 0 if D_r < A else cap*(floor((D_r-A)/d)+1),
    A = base + d + L_sub, the admitted position is
    c_r = min(r, r-1 + min_{t<r}(u_t - t)) and keep_r <=> c_r < u_r."""
    rng = np.random.default_rng(500 + seed)
    n = 500
    d = int(rng.integers(3, 40))
    B = int(rng.integers(1, 5))
    p = util.pipeline([], 1, [d], bmax=B)
    now = 1000
    st = util.state(1, 1, 0, now, B, free_at=now + 3)
    dl = np.sort(rng.integers(900, 1000 + 60 * d, size=n))
    o = oracle.plan([p], util.requests(dl), st, 1)
    A = now + 3 + d
    X = dl - A
    u = np.where(X < 0, 0, B * (np.maximum(X, 0) // d + 1))
    t = np.arange(n)
    v = u - t
    pm = np.minimum.accumulate(v)
    c = np.zeros(n, dtype=np.int64)
    c[1:] = np.minimum(t[1:], t[1:] - 1 + pm[:-1])
    assert (o["keep"] == (c < u)).all()
    assert (o["est_us"] == A + (c // B) * d).all()


# --------------------------------------------------------------------------
# compaction and counters (Sec. 5.1 Metrics)
# --------------------------------------------------------------------------
@pytest.mark.parametrize("name", ["C1", "C1b"])
def test_counters_and_compaction_are_consistent(name):
    wl = inputs.make(name)
    o = plan(wl)
    assert o["n_kept"] == int(o["keep"].sum())
    assert (o["kept_idx"] == o["perm"][o["keep"] == 1]).all()
    assert sorted(o["perm"]) == list(range(wl.n))
    S = wl.state.stage_stride
    counts = np.bincount(wl.requests["ctx"].astype(np.int64) * S + wl.requests["stage"],
                         minlength=wl.n_ctx * S)
    assert (np.diff(o["seg_offsets"]) == counts).all()
    assert (o["ctx_total"] == counts.reshape(wl.n_ctx, S).sum(axis=1)).all()
    assert (o["ctx_kept"] == o["seg_kept"].reshape(wl.n_ctx, S).sum(axis=1)).all()
    kept_by_seg = np.add.reduceat(np.concatenate([o["keep"], [0]]).astype(np.int64),
                                  np.minimum(o["seg_offsets"][:-1], wl.n))
    kept_by_seg[np.diff(o["seg_offsets"]) == 0] = 0
    assert (kept_by_seg == o["seg_kept"]).all()


def test_empty_inputs():
    p = util.pipeline(inputs.chain_edges(2), 2, [5, 6])
    st = util.state(3, 2, 1, 10, 1)
    o = oracle.plan([p], util.requests([]), st, 3)
    assert o["n_kept"] == 0 and (o["seg_offsets"] == 0).all() and (o["ctx_total"] == 0).all()
    # requests only in the last ctx
    o = oracle.plan([p], util.requests([100, 5], stage=1, ctx=2), st, 3)
    assert list(o["ctx_total"]) == [0, 0, 2]
    assert list(o["perm"]) == [1, 0]
    assert list(o["keep"]) == [0, 1]


def test_out_of_range_inputs_are_rejected():
    p = util.pipeline(inputs.chain_edges(2), 2, [5, 6])
    st = util.state(1, 2, 1, 10, 1)
    with pytest.raises(ValueError):
        oracle.plan([p], util.requests([1], stage=2), st, 1)
    with pytest.raises(ValueError):
        oracle.plan([p], util.requests([1], ctx=1), st, 1)
    st = util.state(1, 2, 1, 10, 5)
    with pytest.raises(ValueError):
        oracle.plan([p], util.requests([1]), st, 1)
