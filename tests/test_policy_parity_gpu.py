"""Parity of the comparison rules and order variants (requests with a known downstream path,
arrival order, Nexus' window scan, Clipper++'s split budgets) with the CPU oracle, bit for bit,
through the C ABI."""
import numpy as np
import pytest

from oracle import oracle
from paper_2602_08747_b200 import binding as pb
from paper_2602_08747_b200 import inputs
from tests import util
from tests.gpu_util import assert_identical, run_library

pytestmark = pytest.mark.gpu

MASK, FCFS, NEXUS, CLIPPER = pb.PARD_MODE_PATH_MASK, pb.PARD_MODE_FCFS, pb.PARD_MODE_NEXUS, pb.PARD_MODE_CLIPPER
assert (MASK, FCFS, NEXUS, CLIPPER) == (oracle.MODE_PATH_MASK, oracle.MODE_FCFS, oracle.MODE_NEXUS, oracle.MODE_CLIPPER)


def check(wl, mode, arrivals=None):
    want = oracle.plan(wl.pipelines, wl.requests, wl.state, wl.n_ctx, mode, arrivals)
    rc, got = run_library(wl, mode, arrivals=arrivals)
    assert rc == 0
    assert_identical(got, want)
    return got


def paths_per_stage(wl):
    """[n_ctx, S] number of downstream paths of every (ctx, stage)."""
    S = wl.state.stage_stride
    per_pipe = [[oracle.count_paths(p, k) if k < p.n_stages else 0 for k in range(S)] for p in wl.pipelines]
    poc = wl.state.pipeline_of_ctx
    poc = np.zeros(wl.n_ctx, np.int64) if poc is None else np.asarray(poc)
    return np.asarray(per_pipe, dtype=np.int64)[poc]


def draw_masks(wl, rng, unknown=0.2):
    """Every request names a random non-empty subset of its stage's first 16 downstream paths;
    a share of them (and every request at a sink) leaves the path unknown (0)."""
    r = wl.requests
    npaths = paths_per_stage(wl)[r["ctx"], r["stage"]]
    width = np.minimum(npaths, 16)
    m = rng.integers(1, 1 << 16, size=wl.n) & ((1 << width) - 1)
    m = np.where(m == 0, 1, m)                     # non-empty where the stage has a path at all
    m = np.where((width == 0) | (rng.random(wl.n) < unknown), 0, m)
    r["flags"] = m.astype(np.uint16)


def draw_arrivals(wl, rng):
    """Arrival at the module some time before `now`; objectives of a few hundred milliseconds."""
    now = wl.state.now_us[wl.requests["ctx"]]
    span = int(max(1, (wl.requests["deadline_us"].max() - wl.requests["deadline_us"].min()) // 2 + 1))
    arrive = np.maximum(0, now - rng.integers(0, span, size=wl.n))
    return util.arrivals(arrive, rng.integers(1, 1 << 20, size=wl.n))


# --------------------------------------------------------------------------
# the hand-worked examples, through the library
# --------------------------------------------------------------------------
def test_nexus_window_example_on_the_gpu():
    rows = util.read_golden("nexus_window_example.txt")
    p = util.pipeline([], 1, [100], bmax=2)
    st = util.state(1, 1, 0, 1000, 2, free_at=1000)              # the example's time 0 is 1000 here
    wl = inputs.Workload("nexus", [p], util.requests([1000 + int(r[1]) for r in rows]), st, 1)
    got = check(wl, NEXUS)
    assert list(got["keep"]) == [int(r[2]) for r in rows]
    assert list(got["est_us"]) == [1000 + int(r[3]) for r in rows]


def test_clipper_split_example_on_the_gpu():
    rows = util.read_golden("clipper_split_example.txt")
    p = util.pipeline(inputs.chain_edges(3), 3, [100, 300, 600], bmax=1)
    st = util.state(1, 3, inputs.n_slots(p), 1000, 1, free_at=1000)
    wl = inputs.Workload("clipper", [p], util.requests(np.zeros(len(rows)), stage=1), st, 1)
    a = util.arrivals([1000 + int(r[1]) for r in rows], [int(r[2]) for r in rows])
    got = check(wl, CLIPPER, a)
    assert list(got["keep"]) == [int(r[3]) for r in rows]
    assert list(got["est_us"]) == [1000 + int(r[4]) for r in rows]


def test_masked_diamond_on_the_gpu():
    p = util.pipeline([(0, 1), (0, 2), (1, 3), (2, 3)], 4, [10, 20, 50, 5])
    st = util.state(1, 4, 4, 0, 1, q=[[1, 2, 3, 4]], w=[[100, 7, 11, 13]])
    r = util.requests([100, 100, 100, 400, 30, 30], stage=[0, 0, 0, 0, 1, 3])
    r["flags"] = [0, 1, 2, 3, 1, 9]
    got = check(inputs.Workload("diamond", [p], r, st, 1), MASK)
    assert list(got["keep"][:3]) == [0, 0, 1]                    # only the request on the short branch makes 100


# --------------------------------------------------------------------------
# seeded workloads
# --------------------------------------------------------------------------
REDUCED = [("C1", {}), ("C1b", {}), ("C1", {"n": 1}), ("C1b", {"n": 2049}),
           ("C2b", {"n": 100_003}), ("C3", {"n": 70_001}), ("C3b", {"n": 300_007}),
           ("C4b", {"n_epochs": 64, "per_epoch": 8192}), ("C4", {"n_epochs": 37, "per_epoch": 1000}),
           ("C5b", {"n_inst": 16, "per_inst": 65536}), ("C5", {"n_inst": 9, "per_inst": 5001}),
           ("C4b", {"n_epochs": 1100, "per_epoch": 200})]


@pytest.mark.parametrize("name,kw", REDUCED)
def test_known_paths_on_the_configs(name, kw):
    wl = inputs.make(name, **kw)
    draw_masks(wl, np.random.default_rng(21))
    check(wl, MASK)
    check(wl, MASK | FCFS)


@pytest.mark.parametrize("name,kw", REDUCED)
def test_arrival_order_rules_on_the_configs(name, kw):
    wl = inputs.make(name, **kw)
    check(wl, FCFS)
    check(wl, NEXUS)
    check(wl, CLIPPER, draw_arrivals(wl, np.random.default_rng(22)))


@pytest.mark.parametrize("seed", range(12))
def test_random_small_workloads_under_every_rule(seed):
    rng = np.random.default_rng(1300 + seed)
    wl = util.random_small_workload(rng, int(rng.integers(1, 9000)), n_ctx=int(rng.integers(1, 6)))
    draw_masks(wl, rng)
    a = util.arrivals(rng.integers(900, 2000, size=wl.n), rng.integers(0, 600, size=wl.n))
    for mode, arr in ((MASK, None), (FCFS, None), (MASK | FCFS, None), (NEXUS, None), (CLIPPER, a)):
        check(wl, mode, arr)


def test_known_paths_with_queues_served_high_budget_first():
    wl = inputs.make("C3b", n=200_003)
    rng = np.random.default_rng(23)
    draw_masks(wl, rng)
    wl.state.priority = rng.integers(0, 2, size=(wl.n_ctx, wl.state.stage_stride)).astype(np.uint8)
    check(wl, MASK)


def test_grouped_promise_does_not_change_the_rules():
    """PARD_MODE_GROUPED is a performance promise for the planner's own rule; the comparison rules
    take their own path with or without it."""
    wl = inputs.make("C4b", n_epochs=20, per_epoch=3000)
    draw_masks(wl, np.random.default_rng(26))
    for mode in (MASK, FCFS, NEXUS):
        want = oracle.plan(wl.pipelines, wl.requests, wl.state, wl.n_ctx, mode)
        rc, got = run_library(wl, mode | pb.PARD_MODE_GROUPED)
        assert rc == 0
        assert_identical(got, want)


def test_mask_of_zero_is_the_default_plan():
    wl = inputs.make("C2b", n=50_001)
    rc, plain = run_library(wl, 0)
    rc2, masked = run_library(wl, MASK)
    assert rc == 0 and rc2 == 0
    assert_identical(masked, plain)


def _one_stage(deadline, d=10, B=2, free_at=0, now=0, workers=None):
    p = util.pipeline([], 1, [d], bmax=max(B, 1))
    st = util.state(1, 1, 0, now, B, free_at=free_at, workers=workers)
    return inputs.Workload("edge", [p], util.requests(deadline), st, 1)


def test_nexus_window_sizes_against_step_and_queue_lengths():
    """Windows of 1 (a batch completes at every lane), of exactly one 32-request step, across
    steps, and wider than the whole queue (one partly filled batch)."""
    rng = np.random.default_rng(24)
    n = 5000
    for B, m in ((1, 1), (32, 1), (16, 2), (33, 1), (4096, 1), (4096, 3), (7, 5)):
        d = 13
        dl = rng.integers(0, (n // (B * m) + 3) * d * 2, size=n)
        check(_one_stage(dl, d=d, B=B, workers=m), NEXUS)
        check(_one_stage(np.full(n, 10**9), d=d, B=B, workers=m), NEXUS)          # nothing is ever dropped
        check(_one_stage(np.zeros(n), d=d, B=B, workers=m, now=5), NEXUS)         # everything is


def test_long_runs_broken_late():
    """A run of fitting requests far longer than a step, broken by its last request: every
    provisional keep of the run has to be taken back."""
    n = 3000
    dl = np.full(n, 10**6)
    dl[2500] = 0
    got = check(_one_stage(dl, d=10, B=4096), NEXUS)
    assert got["n_kept"] == n - 2501


def test_walk_converges_on_adversarial_thresholds():
    """Thresholds that fall by one per request make every lane's decision depend on all lanes
    below it (the fixed-point iteration needs its full 32 rounds)."""
    n = 4096
    d = 10
    for dl in (np.arange(n)[::-1] * d + d, (np.arange(n) % 64)[::-1] * d + d, np.arange(n) % 3 * d + d):
        check(_one_stage(dl, d=d, B=1), FCFS)
        check(_one_stage(dl, d=d, B=3), FCFS)


def test_zero_requests_and_empty_queues():
    p = util.pipeline(inputs.chain_edges(2), 2, [5, 6])
    st = util.state(3, 2, 1, 10, 1)
    for mode in (MASK, FCFS, NEXUS):
        check(inputs.Workload("edge", [p], util.requests([]), st, 3), mode)
        check(inputs.Workload("edge", [p], util.requests([100, 5, 100], stage=1, ctx=2), st, 3), mode)


def test_errors_of_the_rules():
    import torch
    wl = inputs.make("C1")
    a = util.arrivals(np.zeros(wl.n), 1000)
    for mode, arr in ((NEXUS | CLIPPER, a), (NEXUS | MASK, None), (CLIPPER | MASK, a), (FCFS | 1, None),
                      (MASK | 1, None), (CLIPPER, None)):
        rc, _ = run_library(wl, mode, check=False, arrivals=arr)
        assert rc == pb.PARD_EINVAL, mode
    wl.state.priority = np.zeros((1, 3), np.uint8)
    rc, _ = run_library(wl, FCFS, check=False)
    assert rc == pb.PARD_EINVAL
    wl.state.priority = None
    # a mask that names no path of the request's stage (stage 0 of the chain has one path: bit 0)
    wl.requests["flags"] = 0
    wl.requests["flags"][17] = 2
    wl.requests["stage"][17] = 0
    rc, _ = run_library(wl, MASK, check=False)
    assert rc == pb.PARD_EDATA
    # an objective beyond the documented range
    wl.requests["flags"] = 0
    a["slo_us"][5] = 1 << 31
    rc, _ = run_library(wl, CLIPPER, check=False, arrivals=a)
    assert rc == pb.PARD_EDATA
    torch.cuda.synchronize()
    check(inputs.make("C1"), FCFS)                              # the context still works


# full sizes: one configuration per rule
@pytest.mark.parametrize("name,mode", [("C3b", MASK), ("C3", FCFS), ("C4", NEXUS), ("C5", CLIPPER)])
def test_rules_full_size(name, mode):
    wl = inputs.make(name)
    rng = np.random.default_rng(25)
    if mode & MASK:
        draw_masks(wl, rng)
    check(wl, mode, draw_arrivals(wl, rng) if mode & CLIPPER else None)
