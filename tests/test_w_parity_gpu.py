"""Parity of pard_estimate_w (CUDA, through the C ABI) with the oracle's
batch-wait estimate (Sec. 4.2, Batch wait estimation): bit-exact, the result
is an integer number of microseconds picked from integer sums."""
import numpy as np
import pytest

from oracle import oracle
from paper_2602_08747_b200 import binding as pb
from paper_2602_08747_b200 import inputs
from tests import gpu_util, util

pytestmark = pytest.mark.gpu


def oracle_w(wl, samples, num, den, seed, R=None):
    st = wl.state
    return oracle.estimate_w(wl.pipelines, st.pipeline_of_ctx, wl.n_ctx, st.stage_stride,
                             R or st.slot_stride, samples, num, den, seed)


def compare(wl, samples, num, den, seed, R=None):
    rc, got = gpu_util.run_estimate_w(wl, samples, num, den, seed, slot_stride=R, fill=0)
    assert rc == pb.PARD_OK
    want = oracle_w(wl, samples, num, den, seed, R)
    bad = np.argwhere(got != want)
    assert bad.size == 0, (bad[:4], got[tuple(bad[0])], want[tuple(bad[0])])
    return got


@pytest.mark.parametrize("name,M", [("C1", 10_000), ("C2", 1000), ("C5", 257)])
def test_workload_dags(name, M):
    """The chain, the 8-stage DAG and the random 16-stage DAG instances; M = 10,000
    is the paper's sample count (several rounds per thread and a ragged tail)."""
    kw = {"C1": {}, "C2": {"n": 1 << 12}, "C5": {"n_inst": 24, "per_inst": 16}}[name]
    wl = inputs.make(name, **kw)
    rng = np.random.default_rng(77)
    samples = inputs.draw_wait_samples(rng, wl, M)
    compare(wl, samples, 1, 10, seed=12345)


@pytest.mark.parametrize("num,den", [(0, 1), (1, 1), (1, 2), (9, 10), (3, 7), (999, 1000)])
def test_quantile_levels(num, den):
    wl = inputs.make("C5", n_inst=3, per_inst=16)
    samples = inputs.draw_wait_samples(np.random.default_rng(num * 31 + den), wl, 4099)
    compare(wl, samples, num, den, seed=2**64 - 5)


@pytest.mark.parametrize("M", [1, 2, 31, 255, 256, 257, 32768])
def test_sample_counts(M):
    """Fewer samples than threads, exactly one round, and the largest allowed count."""
    rng = np.random.default_rng(M)
    p = util.pipeline(inputs.random_dag_edges(rng, 6), 6, [900] * 6)
    R = max(1, inputs.n_slots(p))
    st = util.state(2, 6, R, 0, 1)
    wl = inputs.Workload("w", [p], util.requests([]), st, 2)
    samples = rng.integers(0, 900, size=(2, 6, M)).astype(np.int32)
    compare(wl, samples, 1, 10, seed=M)


def test_largest_waits_and_longest_path():
    """64 stages in a chain with every wait near the upper limit: the sums reach
    just under 2^30, the top of the select's range."""
    S = 64
    p = util.pipeline(inputs.chain_edges(S), S, [1] * S)
    R = inputs.n_slots(p)
    st = util.state(1, S, R, 0, 1)
    wl = inputs.Workload("w", [p], util.requests([]), st, 1)
    rng = np.random.default_rng(5)
    samples = rng.integers(pb.PARD_WAIT_LIMIT_US - 1000, pb.PARD_WAIT_LIMIT_US, size=(1, S, 300)).astype(np.int32)
    got = compare(wl, samples, 1, 2, seed=99)
    assert got[0, 0] > 63 * (pb.PARD_WAIT_LIMIT_US - 1000)


def test_mixed_pipelines_padding_left_untouched():
    rng = np.random.default_rng(8)
    p0 = util.pipeline(inputs.chain_edges(3), 3, [50] * 3)
    p1 = util.pipeline(inputs.DAG8_EDGES, 8, [70] * 8)
    R = inputs.n_slots(p1) + 3
    poc = np.array([1, 0, 0, 1, 1], dtype=np.int32)
    st = util.state(5, 8, R, 0, 1, poc=poc)
    wl = inputs.Workload("w", [p0, p1], util.requests([]), st, 5)
    samples = rng.integers(0, 70, size=(5, 8, 500)).astype(np.int32)
    rc, got = gpu_util.run_estimate_w(wl, samples, 1, 10, 3, fill=-7)
    assert rc == pb.PARD_OK
    want = oracle_w(wl, samples, 1, 10, 3)
    for c in range(5):
        ns = inputs.n_slots(wl.pipelines[poc[c]])
        assert np.array_equal(got[c, :ns], want[c, :ns])
        assert (got[c, ns:] == -7).all()


def test_sink_only_pipeline_writes_nothing():
    p = util.pipeline([], 1, [10])
    st = util.state(2, 1, 1, 0, 1)
    wl = inputs.Workload("w", [p], util.requests([]), st, 2)
    rc, got = gpu_util.run_estimate_w(wl, np.zeros((2, 1, 10), np.int32), 1, 10, 0, fill=-7)
    assert rc == pb.PARD_OK and (got == -7).all()


def test_device_detected_errors():
    p = util.pipeline(inputs.chain_edges(3), 3, [50] * 3)
    st = util.state(2, 3, 2, 0, 1)
    wl = inputs.Workload("w", [p], util.requests([]), st, 2)
    samples = np.full((2, 3, 64), 5, np.int32)
    samples[1, 2, :] = pb.PARD_WAIT_LIMIT_US               # every draw of stage 2 is out of range
    rc, _ = gpu_util.run_estimate_w(wl, samples, 1, 10, 0, check=False)
    assert rc == pb.PARD_EDATA
    samples[1, 2, :] = -1
    rc, _ = gpu_util.run_estimate_w(wl, samples, 1, 10, 0, check=False)
    assert rc == pb.PARD_EDATA
    samples[1, 2, :] = 5
    st.pipeline_of_ctx = np.array([0, 4], dtype=np.int32)   # pipeline id out of range
    rc, _ = gpu_util.run_estimate_w(wl, samples, 1, 10, 0, check=False)
    assert rc == pb.PARD_EDATA
    # the context is still usable
    st.pipeline_of_ctx = None
    compare(wl, samples, 1, 10, 0)


def test_estimate_feeds_the_planner():
    """w from pard_estimate_w used as pard_queue_state_t.d_w_us gives the plan the
    oracle computes from the oracle's w."""
    wl = inputs.make("C2", n=1 << 14)
    samples = inputs.draw_wait_samples(np.random.default_rng(1), wl, 2000)
    rc, w = gpu_util.run_estimate_w(wl, samples, 1, 10, 42)
    assert rc == pb.PARD_OK
    w_or = oracle_w(wl, samples, 1, 10, 42)
    ns = inputs.n_slots(wl.pipelines[0])
    assert np.array_equal(w[:, :ns], w_or[:, :ns])
    wl.state.w_us = np.where(w < 0, 0, w)
    _, got = gpu_util.run_library(wl)
    wl.state.w_us = np.where(w_or < 0, 0, w_or)
    want = oracle.plan(wl.pipelines, wl.requests, wl.state, wl.n_ctx, 0)
    for k in ("keep", "est_us", "perm", "seg_kept"):
        assert np.array_equal(got[k], want[k]), k


@pytest.mark.parametrize("name,kw", [("C1", {}), ("C1b", {}), ("C2b", {"n": 60_001}), ("C3b", {"n": 200_003}),
                                     ("C4b", {"n_epochs": 12, "per_epoch": 4000}), ("C5b", {"n_inst": 7, "per_inst": 9001})])
def test_configs_with_w_from_the_estimator(name, kw):
    """The five workloads with their batch-wait estimates produced by the State Planner's own
    estimator instead of being drawn: M = 10,000 recorded waits per stage, uniform on [0, d) (Sec. 3.2,
    Fig. 3b), lambda = 0.1 (Sec. 4.2).  Each side estimates w itself and plans with its own w."""
    wl = inputs.make(name, **kw)
    samples = inputs.draw_wait_samples(np.random.default_rng(3), wl, 10_000)
    rc, w = gpu_util.run_estimate_w(wl, samples, 1, 10, 7)
    assert rc == pb.PARD_OK
    w_or = oracle_w(wl, samples, 1, 10, 7)
    wl.state.w_us = np.where(w < 0, 0, w)
    rc, got = gpu_util.run_library(wl)
    assert rc == 0
    wl.state.w_us = np.where(w_or < 0, 0, w_or)
    want = oracle.plan(wl.pipelines, wl.requests, wl.state, wl.n_ctx, 0)
    gpu_util.assert_identical(got, want)
