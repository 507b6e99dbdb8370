"""Parity of the CUDA library with the CPU oracle for the adaptive request
priority (paper Sec. 4.3): queues served high budget first inside the planner,
and the load-factor / delayed-transition update that picks each queue's order.
All outputs are integers and are compared bit for bit."""
import numpy as np
import pytest

from oracle import oracle
from paper_2602_08747_b200 import binding as pb
from paper_2602_08747_b200 import inputs
from tests import util
from tests.gpu_util import assert_identical, run_library, run_update_priority

pytestmark = pytest.mark.gpu


def both(wl, mode=0):
    want = oracle.plan(wl.pipelines, wl.requests, wl.state, wl.n_ctx, mode & 1)
    for m in (mode, mode | pb.PARD_MODE_SCAN):
        rc, got = run_library(wl, m)
        assert rc == 0
        assert_identical(got, want)
    return want


def with_priority(wl, rng=None, value=None):
    S = wl.state.stage_stride
    if value is not None:
        wl.state.priority = np.full((wl.n_ctx, S), value, dtype=np.uint8)
    else:
        wl.state.priority = (rng.integers(0, 3, size=(wl.n_ctx, S)) % 2 * rng.integers(1, 200)).astype(np.uint8)
    return wl


@pytest.mark.parametrize("name,kw", [
    ("C1", {}), ("C1b", {}), ("C1b", {"n": 12345}),
    ("C2b", {"n": 100_003}), ("C3b", {"n": 300_007}),
    ("C4b", {"n_epochs": 64, "per_epoch": 8192}), ("C5b", {"n_inst": 16, "per_inst": 65536}),
    ("C4b", {"n_epochs": 1100, "per_epoch": 200}), ("C5b", {"n_inst": 600, "per_inst": 301}),
])
@pytest.mark.parametrize("mode", [0, 1])
def test_configs_reduced_with_mixed_priorities(name, kw, mode):
    rng = np.random.default_rng(17)
    want = both(with_priority(inputs.make(name, **kw), rng), mode)
    if name.endswith("b") and mode == 0:
        assert 0 < want["n_kept"] < len(want["keep"])             # keeps and drops are both exercised


@pytest.mark.parametrize("name,kw", [("C1b", {}), ("C3b", {"n": 200_001}), ("C5b", {"n_inst": 5, "per_inst": 30_000})])
def test_every_queue_high_budget_first(name, kw):
    both(with_priority(inputs.make(name, **kw), value=1))
    both(with_priority(inputs.make(name, **kw), value=255), mode=1)


@pytest.mark.parametrize("seed", range(20))
def test_random_small_workloads_with_priorities(seed):
    rng = np.random.default_rng(1900 + seed)
    n = int(rng.integers(1, 9000))
    wl = util.random_small_workload(rng, n, n_ctx=int(rng.integers(1, 6)))
    both(with_priority(wl, rng), mode=seed & 1)


def _one_stage(deadline, d=10, B=2, prio=1, now=0, free_at=0, workers=None):
    p = util.pipeline([], 1, [d], bmax=max(B, 1))
    st = util.state(1, 1, 0, now, B, free_at=free_at, workers=workers)
    st.priority = np.array([[prio]], dtype=np.uint8)
    return inputs.Workload("edge", [p], util.requests(deadline), st, 1)


def test_high_budget_first_edge_cases():
    rng = np.random.default_rng(3)
    both(_one_stage(np.full(5000, 1000)))                         # all deadlines equal: index order, a prefix kept
    both(_one_stage(np.full(5000, 5)))                            # nothing can be kept
    both(_one_stage(np.full(3000, 10**9)))                        # everything is kept
    both(_one_stage([50]))                                        # one request
    both(_one_stage(rng.integers(0, 40_000, size=70_000), d=7, B=3))          # a long queue: warp-wide searches
    both(_one_stage(rng.integers(0, 40_000, size=70_000), d=7, B=3), mode=1)
    both(_one_stage(rng.integers(0, 2_000_000, size=30_000), d=1, B=1))       # d = 1: no reciprocal
    both(_one_stage(rng.integers(1 << 40, (1 << 40) + (1 << 34), size=20_000), d=(1 << 33) + 5, B=2,
                    now=1 << 40))                                 # operands beyond 32 bits
    both(_one_stage(rng.integers(0, 5000, size=9000), d=7, B=3, workers=2**31 - 1))


def test_high_and_low_budget_first_queues_side_by_side_across_tiles():
    """Queues of both kinds, with boundaries that fall inside and on the edges of
    the decision pass's tiles, and one queue whose window count forces the scan."""
    rng = np.random.default_rng(23)
    S = 6
    p = util.pipeline(inputs.chain_edges(S), S, [9, 7, 5, 11, 3, 8], bmax=4)
    sizes = [2048, 1, 4095, 0, 6000, 8]
    stage = np.repeat(np.arange(S), sizes)
    dl = rng.integers(900, 9000, size=stage.size)
    st = util.state(1, S, 5, 1000, 2, free_at=990, q=4, w=3)
    st.priority = np.array([[1, 0, 1, 1, 0, 1]], dtype=np.uint8)
    perm = rng.permutation(stage.size)
    both(inputs.Workload("mix", [p], util.requests(dl[perm], stage=stage[perm]), st, 1))
    dl[:2048] = rng.integers(900, 900 + 5000 * 9, size=2048)     # > 4096 windows in a low-budget-first queue
    st.priority = np.array([[0, 1, 1, 1, 0, 1]], dtype=np.uint8)
    both(inputs.Workload("mix2", [p], util.requests(dl[perm], stage=stage[perm]), st, 1))


def test_full_size_with_mixed_priorities():
    rng = np.random.default_rng(29)
    both(with_priority(inputs.make("C3b"), rng))
    both(with_priority(inputs.make("C5b"), rng))


# --------------------------------------------------------------------------
# the priority update
# --------------------------------------------------------------------------
def _draw_update_case(rng, n_ctx, S, H, W, big=False, n_pipes=1):
    pipes, poc = [], None
    bmax = 4096 if big else 8
    for _ in range(n_pipes):
        s = int(rng.integers(1, S + 1)) if n_pipes > 1 else S
        tables = [rng.integers((1 << 39) if big else 1, (1 << 40) if big else 400, size=bmax).astype(np.int64)
                  for _ in range(s)]
        pipes.append(inputs.make_pipeline(inputs.chain_edges(s), s, [bmax] * s, tables))
    if n_pipes > 1:
        poc = rng.integers(0, n_pipes, size=n_ctx).astype(np.int32)
    B = rng.integers(1, bmax + 1, size=(n_ctx, S)).astype(np.int32)
    m = rng.integers(1, (1 << 18) if big else 4, size=(n_ctx, S)).astype(np.int32)
    tau = int(rng.integers(1 << 30, 1 << 31)) if big else int(rng.integers(1, 5000))
    # rates around the module throughput, so that all three outcomes occur
    x = np.zeros((n_ctx, S, H), dtype=np.uint32)
    for c in range(n_ctx):
        p = pipes[int(poc[c]) if poc is not None else 0]
        for k in range(S):
            kk = min(k, p.n_stages - 1)
            cap_rate = int(B[c, k]) * int(m[c, k]) * tau / p.latency(kk, min(int(B[c, k]), bmax))
            level = max(1.0, min(cap_rate, float((1 << 24) - 2))) * rng.uniform(0.3, 1.7)
            noise = rng.uniform(0.0, 0.6)
            x[c, k] = np.clip(np.rint(level * (1 + noise * rng.uniform(-1, 1, size=H))), 0, (1 << 24) - 1)
    x[0, 0] = 0
    prev = rng.integers(0, 2, size=(n_ctx, S)).astype(np.uint8)
    return pipes, poc, B, m, x, tau, prev


@pytest.mark.parametrize("H,W", [(1, 1), (5, 5), (12, 5), (32, 1), (33, 32), (64, 7), (100, 33), (4096, 300),
                                 (4096, 4096)])
@pytest.mark.parametrize("big", [False, True])
def test_update_priority_matches_the_oracle(H, W, big):
    rng = np.random.default_rng(H * 7 + W + (1000 if big else 0))
    n_ctx, S = 37, 5
    pipes, poc, B, m, x, tau, prev = _draw_update_case(rng, n_ctx, S, H, W, big)
    want = oracle.update_priority(pipes, poc, n_ctx, S, B, m, x, W, tau, prev)
    rc, got = run_update_priority(pipes, poc, n_ctx, S, B, m, x, W, tau, prev)
    assert rc == 0
    assert np.array_equal(got, want)
    if H >= 12 and not big:
        changed = got != prev
        assert changed.any() and (~changed).any()                 # both a switch and a kept priority occur


def test_update_priority_several_pipelines_padded_rows_and_default_workers():
    rng = np.random.default_rng(77)
    n_ctx, S, H, W = 50, 6, 40, 5
    pipes, poc, B, m, x, tau, prev = _draw_update_case(rng, n_ctx, S, H, W, n_pipes=4)
    for c in range(n_ctx):                                        # batch sizes of padding columns are arbitrary
        B[c, pipes[int(poc[c])].n_stages:] = -5
    prev = rng.integers(0, 256, size=(n_ctx, S)).astype(np.uint8)
    want = oracle.update_priority(pipes, poc, n_ctx, S, B, None, x, W, tau, prev)
    rc, got = run_update_priority(pipes, poc, n_ctx, S, B, None, x, W, tau, prev)
    assert rc == 0
    assert np.array_equal(got, want)
    for c in range(n_ctx):
        ns = pipes[int(poc[c])].n_stages
        assert np.array_equal(got[c, ns:], prev[c, ns:])


def test_update_priority_reports_bad_device_data():
    p = util.pipeline([], 1, [10], bmax=4)
    x = np.ones((1, 1, 8), np.uint32)
    ok = dict(pipelines=[p], pipeline_of_ctx=None, n_ctx=1, S=1, batch=np.array([[2]], np.int32), workers=None,
              arrivals=x, window=3, interval_us=100, priority=np.zeros((1, 1), np.uint8))
    assert run_update_priority(**ok)[0] == 0
    xb = x.copy()
    xb[0, 0, 3] = 1 << 24
    for bad in (dict(batch=np.array([[5]], np.int32)), dict(batch=np.array([[0]], np.int32)),
                dict(workers=np.array([[0]], np.int32)), dict(workers=np.array([[1 << 30]], np.int32)),
                dict(arrivals=xb)):
        assert run_update_priority(**{**ok, **bad}, check=False)[0] == pb.PARD_EDATA


def test_updated_priorities_feed_the_planner():
    """The two entry points chained on the device, as a State Planner would:
    update the priorities from the arrival history, then plan with them."""
    import torch
    rng = np.random.default_rng(41)
    wl = inputs.make("C5b", n_inst=12, per_inst=20_000)
    S, H, W, tau = wl.state.stage_stride, 30, 5, 1_000_000
    st = wl.state
    x = np.zeros((wl.n_ctx, S, H), dtype=np.uint32)
    for c in range(wl.n_ctx):
        p = wl.pipelines[int(st.pipeline_of_ctx[c])]
        for k in range(p.n_stages):
            rate = int(st.batch[c, k]) * int(st.workers[c, k]) * tau / p.latency(k, int(st.batch[c, k]))
            x[c, k] = np.clip(np.rint(rate * rng.uniform(0.5, 1.5) * (1 + 0.2 * rng.uniform(-1, 1, size=H))), 0,
                              (1 << 24) - 1)
    prev = rng.integers(0, 2, size=(wl.n_ctx, S)).astype(np.uint8)
    prio = oracle.update_priority(wl.pipelines, st.pipeline_of_ctx, wl.n_ctx, S, st.batch, st.workers, x, W, tau, prev)
    assert 0 < int((prio != 0).sum()) < prio.size
    st.priority = prio
    want = oracle.plan(wl.pipelines, wl.requests, st, wl.n_ctx)

    dev = "cuda:0"
    pipes = [pb.pard_load_pipeline(p) for p in wl.pipelines]
    d_state = pb.device_state(st, dev)
    d_state.priority = torch.from_numpy(prev).to(dev)             # the device array starts from the old priorities
    d_x = torch.from_numpy(x.view(np.int32)).to(dev)
    ws_p = pb.alloc_workspace(pb.pard_update_priority_workspace_bytes(len(pipes)), dev)
    stream = torch.cuda.current_stream().cuda_stream
    pb.pard_update_priority(pipes, d_state.pipeline_of_ctx, wl.n_ctx, S, d_state.batch, d_state.workers, d_x, H, W,
                            tau, 0, d_state.priority, ws_p, stream=stream)
    out = pb.alloc_out(wl.n, wl.n_ctx * S, dev)
    ws = pb.alloc_workspace(pb.pard_plan_workspace_bytes(wl.n, wl.n_ctx, S), dev)
    pb.pard_plan(pipes, pb.device_requests(wl.requests, dev), wl.n, d_state, wl.n_ctx, 0, out, ws, stream=stream)
    torch.cuda.synchronize()
    got = pb.out_to_numpy(out, wl.n)
    for key in ("keep", "est_us", "perm", "kept_idx", "seg_offsets", "seg_kept"):
        assert np.array_equal(got[key], want[key]), key
    assert got["n_kept"] == want["n_kept"]
