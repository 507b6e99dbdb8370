"""Parity of the CUDA library (through the C ABI) with the CPU oracle, element
by element and bit for bit, on the same seeded inputs."""
import numpy as np
import pytest

from oracle import oracle
from paper_2602_08747_b200 import binding as pb
from paper_2602_08747_b200 import inputs
from tests import util
from tests.gpu_util import assert_identical, run_library

pytestmark = pytest.mark.gpu


def both(wl, mode=0):
    """Oracle vs library, with the decision taken from the batch-window tables
    (default) and by the scan kernels (PARD_MODE_SCAN)."""
    want = oracle.plan(wl.pipelines, wl.requests, wl.state, wl.n_ctx, mode & 1)
    rc, got = run_library(wl, mode)
    assert rc == 0
    assert_identical(got, want)
    rc, got2 = run_library(wl, mode | pb.PARD_MODE_SCAN)
    assert rc == 0
    assert_identical(got2, want)
    return got


# sizes chosen to span several tiles of both the sort (4096) and the decision
# pass (2048) and to leave a ragged tail
@pytest.mark.parametrize("name,kw", [
    ("C1", {}), ("C1b", {}),
    ("C1", {"n": 1}), ("C1", {"n": 2047}), ("C1", {"n": 2049}), ("C1b", {"n": 12345}),
    ("C2", {"n": 100_003}), ("C2b", {"n": 100_003}),
    ("C3", {"n": 70_001}), ("C3b", {"n": 300_007}),
    ("C4", {"n_epochs": 37, "per_epoch": 1000}), ("C4b", {"n_epochs": 64, "per_epoch": 8192}),
    ("C5", {"n_inst": 9, "per_inst": 5001}), ("C5b", {"n_inst": 16, "per_inst": 65536}),
    # thousands of queues: the lane-per-queue form of the segment search
    ("C4b", {"n_epochs": 1100, "per_epoch": 200}), ("C5b", {"n_inst": 600, "per_inst": 301}),
])
@pytest.mark.parametrize("mode", [0, 1])
def test_configs_reduced(name, kw, mode):
    both(inputs.make(name, **kw), mode)


@pytest.mark.parametrize("seed", range(20))
def test_random_small_workloads(seed):
    rng = np.random.default_rng(900 + seed)
    n = int(rng.integers(1, 9000))
    wl = util.random_small_workload(rng, n, n_ctx=int(rng.integers(1, 6)))
    both(wl, mode=seed & 1)


def _one_stage(n, deadline, d=10, B=2, free_at=0, now=0, workers=None):
    p = util.pipeline([], 1, [d], bmax=max(B, 1))
    st = util.state(1, 1, 0, now, B, free_at=free_at, workers=workers)
    return inputs.Workload("edge", [p], util.requests(deadline), st, 1)


def test_all_deadlines_equal():
    both(_one_stage(5000, np.full(5000, 1000)))
    both(_one_stage(5000, np.full(5000, 10_000)))


def test_all_expired_and_all_kept():
    got = both(_one_stage(6000, np.arange(6000) % 7, now=10_000))
    assert got["n_kept"] == 0
    got = both(_one_stage(6000, 10**12 + np.arange(6000)[::-1]))
    assert got["n_kept"] == 6000


def test_batch_one_and_batch_max_and_many_workers():
    rng = np.random.default_rng(5)
    dl = rng.integers(0, 40_000, size=9000)
    both(_one_stage(9000, dl, B=1, d=7))
    both(_one_stage(9000, dl, B=4096, d=7))
    both(_one_stage(9000, dl, B=3, d=7, workers=2**31 - 1))


def test_threshold_exactly_at_tile_and_warp_boundaries():
    # u jumps by cap at positions that land on 32, 256, 2048 and 4096
    for B in (32, 256, 2048, 4096):
        dl = np.repeat(np.arange(1, 6) * 100, B)     # B requests per batch deadline
        both(_one_stage(len(dl), dl, d=100, B=B))
        both(_one_stage(len(dl), dl - 1, d=100, B=B))


def test_segment_boundaries_on_tile_boundaries_and_empty_segments():
    p = util.pipeline(inputs.chain_edges(5), 5, [3, 4, 5, 6, 7], bmax=4)
    st = util.state(3, 5, inputs.n_slots(p), [100, 200, 300], 2, q=1, w=2)
    rng = np.random.default_rng(6)
    # queue lengths that are multiples of the tile sizes, with empty queues and an empty ctx
    lens = {(0, 0): 2048, (0, 1): 4096, (0, 3): 2048, (2, 0): 6144, (2, 4): 1}
    dl, stg, ctx = [], [], []
    for (c, k), m in lens.items():
        dl.append(rng.integers(0, 4000, size=m)); stg.append(np.full(m, k)); ctx.append(np.full(m, c))
    order = rng.permutation(sum(lens.values()))
    r = util.requests(np.concatenate(dl)[order], stage=np.concatenate(stg)[order],
                      ctx=np.concatenate(ctx)[order])
    got = both(inputs.Workload("edge", [p], r, st, 3))
    assert list(got["ctx_total"]) == [8192, 0, 6145]


def test_zero_requests():
    p = util.pipeline(inputs.chain_edges(2), 2, [5, 6])
    st = util.state(3, 2, 1, 10, 1)
    got = both(inputs.Workload("edge", [p], util.requests([]), st, 3))
    assert got["n_kept"] == 0


def test_large_times_use_the_64_bit_division():
    # deadlines and durations beyond 2^32 us
    d = (1 << 35) + 12345
    p = util.pipeline([], 1, [d], bmax=2)
    now = 1 << 50
    st = util.state(1, 1, 0, now, 2, free_at=now + 17)
    rng = np.random.default_rng(7)
    dl = now + rng.integers(0, 40 * d, size=7000)
    both(inputs.Workload("edge", [p], util.requests(dl), st, 1))


def test_wide_deadline_span():
    # 2^44 us between the earliest and the latest deadline: 6 radix passes
    rng = np.random.default_rng(8)
    dl = rng.integers(0, 1 << 44, size=20_000)
    both(_one_stage(20_000, dl, d=1 << 30, B=4, now=0))


def test_top_digit_of_one_and_two_bits():
    """Keys of 8k + 1 and 8k + 2 bits: the top radix pass ranks by ballots instead of through
    shared memory (full tiles) and by the generic code (the ragged last tile)."""
    rng = np.random.default_rng(14)
    for span_bits in (9, 10, 17, 18):
        n = 50_001
        dl = rng.integers(0, 1 << span_bits, size=n)
        dl[0], dl[1] = 0, (1 << span_bits) - 1              # the span is exactly span_bits wide
        both(_one_stage(n, dl, d=3, B=2))


def test_multiple_pipelines_and_padded_rows():
    rng = np.random.default_rng(9)
    pa = util.pipeline(inputs.chain_edges(2), 2, [30, 40])
    pbig = util.pipeline([(0, 1), (0, 2), (1, 3), (2, 3)], 4, [10, 20, 50, 5])
    n_ctx = 5
    poc = [1, 0, 1, 1, 0]
    S, R = 6, 9                                    # wider rows than any pipeline needs
    st = util.state(n_ctx, S, R, rng.integers(100, 200, size=n_ctx), 2,
                    free_at=rng.integers(100, 300, size=(n_ctx, S)),
                    q=rng.integers(0, 9, size=(n_ctx, S)), w=rng.integers(0, 30, size=(n_ctx, R)), poc=poc)
    n = 30_000
    ctx = rng.integers(0, n_ctx, size=n)
    stage = np.where(np.asarray(poc)[ctx] == 0, rng.integers(0, 2, size=n), rng.integers(0, 4, size=n))
    r = util.requests(rng.integers(100, 3000, size=n), stage=stage, ctx=ctx)
    both(inputs.Workload("edge", [pa, pbig], r, st, n_ctx))


@pytest.mark.parametrize("n", [3000, 9000])     # planned by one block / by the kernels of the general path
def test_device_detected_errors(n):
    p = util.pipeline(inputs.chain_edges(2), 2, [5, 6])
    good = util.requests(np.arange(n) + 100)
    st = util.state(1, 2, 1, 10, 1)
    for bad_field, bad_val in (("stage", 2), ("ctx", 1), ("deadline_us", -5), ("deadline_us", 1 << 60)):
        r = good.copy()
        r[bad_field][1234] = bad_val
        rc, _ = run_library(inputs.Workload("bad", [p], r, st, 1), check=False)
        assert rc == pb.PARD_EDATA, bad_field
    rc, _ = run_library(inputs.Workload("bad", [p], good, util.state(1, 2, 1, 10, 5), 1), check=False)
    assert rc == pb.PARD_EDATA
    rc, _ = run_library(inputs.Workload("bad", [p], good, util.state(1, 2, 1, 10, 1, workers=0), 1), check=False)
    assert rc == pb.PARD_EDATA
    # a request queued at a stage its pipeline does not have (row is wider than the pipeline)
    r = good.copy()
    r["stage"][7] = 2
    rc, _ = run_library(inputs.Workload("bad", [p], r, util.state(1, 3, 1, 10, 1), 1), check=False)
    assert rc == pb.PARD_EDATA
    # the same with a deadline far from the queue's start: the request's batch window (offset 2,500
    # with the default duration of 1) lies beyond the queue's window table; it must be
    # reported, not looked up (the offset stays below n, i.e. inside the caller's workspace)
    r = good.copy()
    r["stage"][2500] = 2
    rc, _ = run_library(inputs.Workload("bad", [p], r, util.state(1, 3, 1, 10, 1), 1), check=False)
    assert rc == pb.PARD_EDATA
    # the context still works afterwards
    both(inputs.Workload("ok", [p], good, st, 1))


def test_bounded_wait_runs_out_and_is_reported():
    """Failure detection without a fault: with the stall aid the tiles of the first
    sort pass wait for a word that never comes; each wait is bounded, the call
    returns PARD_ETIMEOUT, nothing hangs and the next call is correct."""
    wl = inputs.make("C3", n=300_000)
    rc, _ = run_library(wl, mode=pb.PARD_MODE_TEST_STALL, check=False)
    assert rc == pb.PARD_ETIMEOUT
    both(wl)


def test_bounded_grid_barrier_runs_out_and_is_reported():
    """The scan path's blocks meet at counters; a block that never arrives (stall aid) makes every
    other block's bounded wait run out: PARD_ETIMEOUT, nothing hangs, the next call is correct.
    The call is sorted block by block, so the sort itself has no wait to run out first."""
    wl, _ = _grouped(n_epochs=40, seed=7)
    rc, _ = run_library(wl, mode=pb.PARD_MODE_SCAN | pb.PARD_MODE_TEST_STALL, check=False)
    assert rc == pb.PARD_ETIMEOUT
    both(wl)


def test_key_wider_than_64_bits_is_sorted_in_chunks():
    """Segment, deadline and index bits beyond one 64-bit sort element: the key is sorted in
    chunks and the queues are walked; same plan as the oracle's."""
    # 2^59 span * 2^14 requests * 64 segments
    p = util.pipeline(inputs.chain_edges(2), 2, [5, 6])
    n = 10_000
    rng = np.random.default_rng(12)
    dl = rng.integers(0, 200, size=n).astype(np.int64)
    dl[-1] = (1 << 59)
    dl[17] = (1 << 59) - 3
    st = util.state(32, 2, 1, 10, 1)
    r = util.requests(dl, stage=rng.integers(0, 2, size=n), ctx=rng.integers(0, 32, size=n))
    wl = inputs.Workload("wide", [p], r, st, 32)
    for mode in (0, 1):
        want = oracle.plan(wl.pipelines, wl.requests, wl.state, wl.n_ctx, mode)
        rc, got = run_library(wl, mode)
        assert rc == 0
        assert_identical(got, want)
    # deadlines spread over the whole span, several super-passes, some queues served high budget first
    n = 60_001
    dl = rng.integers(0, 1 << 59, size=n)
    dl[:5000] = rng.integers(0, 400, size=5000)                  # and a cluster that the planner keeps part of
    st = util.state(700, 2, 1, 10, 2)
    st.priority = rng.integers(0, 2, size=(700, 2)).astype(np.uint8)
    r = util.requests(dl, stage=rng.integers(0, 2, size=n), ctx=rng.integers(0, 700, size=n))
    wl = inputs.Workload("wide", [p], r, st, 700)
    want = oracle.plan(wl.pipelines, wl.requests, wl.state, wl.n_ctx, 0)
    rc, got = run_library(wl, 0)
    assert rc == 0
    assert_identical(got, want)
    # one small ctx (the one-block path finds the width and hands over)
    p1 = util.pipeline(inputs.chain_edges(40), 40, [3] * 40)
    dl = rng.integers(0, 1 << 59, size=5000)
    dl[:2000] = rng.integers(0, 300, size=2000)
    wl = inputs.Workload("wide", [p1], util.requests(dl, stage=rng.integers(0, 40, size=5000)),
                         util.state(1, 40, inputs.n_slots(p1), 10, 2), 1)
    assert 6 + 59 + 13 > 64
    want = oracle.plan(wl.pipelines, wl.requests, wl.state, wl.n_ctx, 0)
    rc, got = run_library(wl, 0)
    assert rc == 0
    assert_identical(got, want)


def test_wide_key_without_waiting_is_reported():
    """With PARD_MODE_NOWAIT nothing is read back, so the chunked sort cannot be started: the
    width is reported by pard_plan_status."""
    import torch
    p = util.pipeline(inputs.chain_edges(2), 2, [5, 6])
    dl = np.arange(10_000, dtype=np.int64)
    dl[-1] = 1 << 59
    wl = inputs.Workload("wide", [p], util.requests(dl), util.state(32, 2, 1, 10, 1), 32)
    pipes = [pb.pard_load_pipeline(q) for q in wl.pipelines]
    ws = pb.alloc_workspace(pb.pard_plan_workspace_bytes(wl.n, 32, 2))
    out = pb.alloc_out(wl.n, 64)
    stream = torch.cuda.current_stream().cuda_stream
    assert pb.pard_plan(pipes, pb.device_requests(wl.requests), wl.n, pb.device_state(wl.state), 32, pb.PARD_MODE_NOWAIT,
                        out, ws, stream=stream, check=False) == pb.PARD_OK
    assert pb.pard_plan_status(ws, stream, check=False) == pb.PARD_ERANGE


def test_workspace_too_small_and_foreign_handle():
    import torch
    wl = inputs.make("C1")
    pipes = [pb.pard_load_pipeline(p) for p in wl.pipelines]
    need = pb.pard_plan_workspace_bytes(wl.n, 1, 3)
    ws = pb.alloc_workspace(need)
    out = pb.alloc_out(wl.n, 3)
    d_req, d_st = pb.device_requests(wl.requests), pb.device_state(wl.state)
    assert pb.pard_plan(pipes, d_req, wl.n, d_st, 1, 0, out, ws, workspace_bytes=need - 1,
                        check=False) == pb.PARD_EWORKSPACE
    host_only = pb.pard_load_pipeline(wl.pipelines[0], host_only=True)
    assert pb.pard_plan([host_only], d_req, wl.n, d_st, 1, 0, out, ws, check=False) == pb.PARD_EINVAL
    torch.cuda.synchronize()


def test_host_buffer_entry_point_matches():
    import torch
    wl = inputs.make("C2b", n=150_001)
    wl.state.priority = np.random.default_rng(5).integers(0, 2, size=(wl.n_ctx, wl.state.stage_stride)).astype(np.uint8)
    want = oracle.plan(wl.pipelines, wl.requests, wl.state, wl.n_ctx)
    pipes = [pb.pard_load_pipeline(p) for p in wl.pipelines]
    st = wl.state
    S, R = st.stage_stride, st.slot_stride
    n_seg = wl.n_ctx * S
    hs = pb.QueueStateArrays(S, R, st.now_us, st.batch, st.free_at_us, st.q_us, st.w_us, st.workers,
                             st.pipeline_of_ctx, st.priority)
    out = pb.PlanOut(np.zeros(wl.n, np.uint8), np.zeros(wl.n, np.int64), np.zeros(wl.n, np.uint32),
                     np.zeros(wl.n, np.uint32), np.zeros(1, np.uint64),
                     np.zeros(n_seg + 1, np.uint32), np.zeros(n_seg, np.uint32))
    ws = pb.alloc_workspace(pb.pard_plan_host_workspace_bytes(wl.n, wl.n_ctx, S, R))
    req = np.ascontiguousarray(wl.requests)
    pb.pard_plan_host(pipes, req, wl.n, hs, wl.n_ctx, 0, out, ws,
                      stream=torch.cuda.current_stream().cuda_stream)
    nk = int(out.n_kept[0])
    assert nk == want["n_kept"]
    assert np.array_equal(out.keep, want["keep"])
    assert np.array_equal(out.est_us, want["est_us"])
    assert np.array_equal(out.perm, want["perm"])
    assert np.array_equal(out.kept_idx[:nk], want["kept_idx"])
    assert np.array_equal(out.seg_offsets, want["seg_offsets"])
    assert np.array_equal(out.seg_kept, want["seg_kept"])


def test_sharded_plans_concatenate_to_the_whole_job():
    """Sharding by ctx (the multi-GPU path) needs no exchange: the shards'
    outputs, planned one after the other on this GPU, concatenate to the oracle's
    plan of the whole job."""
    from paper_2602_08747_b200 import sharding
    wl = inputs.make("C4b", n_epochs=12, per_epoch=3000)
    whole = oracle.plan(wl.pipelines, wl.requests, wl.state, wl.n_ctx)
    parts = []
    for rank in range(3):
        rc, got = run_library(sharding.shard_workload(wl, 3, rank))
        assert rc == 0
        parts.append(got)
    for key in ("keep", "est_us", "ctx_total", "ctx_kept", "seg_kept"):
        assert np.array_equal(np.concatenate([p[key] for p in parts]), whole[key]), key
    assert sum(p["n_kept"] for p in parts) == whole["n_kept"]


# full sizes, in the launch configuration the benchmark times
@pytest.mark.parametrize("name", ["C2", "C3", "C3b", "C4", "C5"])
def test_configs_full_size(name):
    both(inputs.make(name))


def test_window_count_limits():
    """4,094 batch windows in one queue still use the window tables, 4,097 do not;
    both sides of the limit give the oracle's plan."""
    rng = np.random.default_rng(11)
    for span_windows in (4094, 4097):
        d = 10
        dl = rng.integers(0, span_windows * d, size=50_000)
        dl[0] = span_windows * d - 1                      # the last window is occupied
        both(_one_stage(len(dl), dl, d=d, B=3))


# --------------------------------------------------------------------------
# requests grouped by ctx, every ctx within one sort tile: the block-local sort
# --------------------------------------------------------------------------
def _grouped(n_epochs=40, seed=0, keep_lo=0.3):
    """C4b with a random share of every epoch's requests removed (order kept):
    contexts of ragged sizes, still grouped by ascending ctx."""
    rng = np.random.default_rng(seed)
    wl = inputs.make("C4b", n_epochs=n_epochs, per_epoch=8192)
    share = rng.uniform(keep_lo, 1.0, size=wl.n_ctx)
    share[rng.integers(0, wl.n_ctx)] = 1.0                       # one ctx fills its tile exactly
    keep = rng.random(wl.n) < share[wl.requests["ctx"]]
    wl.requests = np.ascontiguousarray(wl.requests[keep])
    return wl, rng


def grouped(wl, mode=0):
    """The same through PARD_MODE_GROUPED: one thread block plans each ctx from start to end."""
    want = oracle.plan(wl.pipelines, wl.requests, wl.state, wl.n_ctx, mode & 1)
    rc, got = run_library(wl, mode | pb.PARD_MODE_GROUPED)
    assert rc == 0
    assert_identical(got, want)


@pytest.mark.parametrize("mode", [0, 1])
def test_grouped_contexts_take_the_local_sort(mode):
    wl, rng = _grouped(seed=1)
    both(wl, mode)
    grouped(wl, mode)
    # some contexts empty, one with a single request
    wl, rng = _grouped(seed=2, keep_lo=0.5)
    r = wl.requests
    drop = np.isin(r["ctx"], [3, 4, 17]) | ((r["ctx"] == 9) & (np.arange(wl.n) != np.flatnonzero(r["ctx"] == 9)[0]))
    wl.requests = np.ascontiguousarray(r[~drop])
    both(wl, mode)
    grouped(wl, mode)
    # queues served high budget first among them
    wl, rng = _grouped(seed=3)
    wl.state.priority = rng.integers(0, 2, size=(wl.n_ctx, wl.state.stage_stride)).astype(np.uint8)
    both(wl, mode)
    grouped(wl, mode)


@pytest.mark.parametrize("name,kw", [("C4", {"n_epochs": 37, "per_epoch": 1000}), ("C4b", {"n_epochs": 64, "per_epoch": 8192}),
                                     ("C5b", {"n_inst": 600, "per_inst": 301}), ("C5", {"n_inst": 9, "per_inst": 5001}),
                                     ("C4b", {"n_epochs": 1100, "per_epoch": 200})])
@pytest.mark.parametrize("mode", [0, 1])
def test_block_per_ctx_on_the_grouped_configs(name, kw, mode):
    grouped(inputs.make(name, **kw), mode)


def test_grouped_contexts_larger_than_a_tile_sort_inside_their_ranges():
    """PARD_MODE_GROUPED with contexts of more than a sort tile on average: the radix passes stay
    inside every ctx's range and leave the ctx bits alone."""
    for mode in (0, 1):
        grouped(inputs.make("C5b", n_inst=16, per_inst=65536), mode)
    grouped(inputs.make("C5", n_inst=9, per_inst=20_001))
    # ragged: contexts far below a tile, one empty, several of many tiles; priorities
    rng = np.random.default_rng(15)
    wl = inputs.make("C5b", n_inst=12, per_inst=30_000)
    share = rng.uniform(0.05, 1.0, size=wl.n_ctx)
    share[3] = 0.0
    share[7] = 1.0
    keep = rng.random(wl.n) < share[wl.requests["ctx"]]
    wl.requests = np.ascontiguousarray(wl.requests[keep])
    assert wl.n > wl.n_ctx * 8192
    grouped(wl)
    wl.state.priority = rng.integers(0, 2, size=(wl.n_ctx, wl.state.stage_stride)).astype(np.uint8)
    grouped(wl)
    grouped(wl, 1)
    # a broken promise is reported
    r = wl.requests.copy()
    r[[5, wl.n - 7]] = r[[wl.n - 7, 5]]
    wl.requests = r
    rc, _ = run_library(wl, pb.PARD_MODE_GROUPED, check=False)
    assert rc == pb.PARD_EDATA
    # a stage stride that is not a power of two: the promise is not used, the result is the same
    p = util.pipeline(inputs.chain_edges(3), 3, [30, 40, 50])
    n = 60_000
    ctx = np.sort(rng.integers(0, 3, size=n))
    st = util.state(3, 3, inputs.n_slots(p), 100, 2)
    wl3 = inputs.Workload("odd", [p], util.requests(rng.integers(100, 5000, size=n), stage=rng.integers(0, 3, size=n), ctx=ctx), st, 3)
    grouped(wl3)


def test_grouped_contexts_larger_than_a_tile_full_size():
    grouped(inputs.make("C5"))


def test_block_per_ctx_full_size():
    grouped(inputs.make("C4"))


def test_single_small_ctx_is_one_block():
    """One ctx of at most a sort tile: the whole call is one kernel; sizes around the limit."""
    for n in (1, 2, 31, 33, 4097, 8191, 8192, 8193):
        both(inputs.make("C1b", n=n))
        both(inputs.make("C1", n=n), mode=1)
    # many stages, a DAG, priorities
    wl = inputs.make("C3b", n=8000)
    wl.state.priority = np.random.default_rng(4).integers(0, 2, size=(1, wl.state.stage_stride)).astype(np.uint8)
    both(wl)
    both(wl, mode=1)


def test_broken_grouping_promise_is_reported():
    wl, rng = _grouped(seed=4)
    r = wl.requests.copy()
    i, j = 5, wl.n - 7
    r[[i, j]] = r[[j, i]]                                        # two requests far from their ctx's group
    wl.requests = r
    rc, _ = run_library(wl, pb.PARD_MODE_GROUPED, check=False)
    assert rc == pb.PARD_EDATA
    wl, rng = _grouped(seed=5, keep_lo=0.9)
    r = wl.requests.copy()
    r["ctx"][r["ctx"] == 21] = 20                                # ctx 20 now holds two epochs: more than a tile
    wl.requests = r
    rc, _ = run_library(wl, pb.PARD_MODE_GROUPED, check=False)
    assert rc == pb.PARD_EDATA
    # the same two breaches in a call of more contexts than the block-per-ctx planner takes on
    # (there a block per ctx only sorts): reported as well, nothing behind the sort runs
    for breach in ("order", "size"):
        wl = inputs.make("C4b", n_epochs=700, per_epoch=600)
        r = wl.requests.copy()
        if breach == "order":
            r[[5, wl.n - 7]] = r[[wl.n - 7, 5]]
        else:
            r["ctx"][(r["ctx"] >= 100) & (r["ctx"] < 120)] = 100      # 20 epochs in one ctx: 12,000 requests
        wl.requests = r
        rc, _ = run_library(wl, pb.PARD_MODE_GROUPED, check=False)
        assert rc == pb.PARD_EDATA, breach
    grouped(inputs.make("C4b", n_epochs=700, per_epoch=600))
    # input errors inside a block-planned ctx
    wl = inputs.make("C1b")
    wl.requests["stage"][100] = 7
    rc, _ = run_library(wl, 0, check=False)
    assert rc == pb.PARD_EDATA
    wl = inputs.make("C1b")
    wl.requests["ctx"][100] = 3
    rc, _ = run_library(wl, 0, check=False)
    assert rc == pb.PARD_EDATA
    both(inputs.make("C1b"))                                     # the context still works


def test_grouped_contexts_fall_back_when_the_device_says_no():
    """Same sizes, but the device finds a reason against the local sort: requests
    out of ctx order, or one ctx larger than a tile.  Results are the oracle's
    either way."""
    wl, rng = _grouped(seed=4)
    r = wl.requests.copy()
    i, j = 5, wl.n - 7
    r[[i, j]] = r[[j, i]]                                        # two requests far from their ctx's group
    wl.requests = r
    both(wl)
    wl, rng = _grouped(seed=5, keep_lo=0.9)
    r = wl.requests.copy()
    r["ctx"][r["ctx"] == 21] = 20                                # ctx 20 now holds two epochs, ctx 21 none
    wl.requests = r
    both(wl)
    # shuffled completely
    wl, rng = _grouped(seed=6)
    wl.requests = np.ascontiguousarray(wl.requests[rng.permutation(wl.n)])
    both(wl)


def test_grouped_contexts_with_equal_deadlines_and_one_stage():
    """No bit differs inside a ctx (one stage, all deadlines of a ctx equal): index order stands."""
    p = util.pipeline([], 1, [10], bmax=2)
    n_ctx, per = 6, 3000
    ctx = np.repeat(np.arange(n_ctx), per)
    dl = 1000 + 50 * ctx
    st = util.state(n_ctx, 1, 0, 900, 2)
    both(inputs.Workload("flat", [p], util.requests(dl, stage=0, ctx=ctx), st, n_ctx))
