"""Pins of the oracle's epoch-to-epoch state carry (closed-loop replay): busy
period closed forms, agreement with the planner's own estimate of when the last
admitted request completes, and the recorded queueing-delay samples."""
import numpy as np
import pytest

from oracle import oracle
from paper_2602_08747_b200 import inputs
from tests import util


def advance(p, now, B, kept, free_at, workers=None, M=0, slot=0, S=None, poc=None, pipes=None):
    S = S or p.n_stages
    fa = np.array(free_at, dtype=np.int64).reshape(1, S).copy()
    t = np.full((1, S, M), -1, np.int64) if M else None
    d = np.zeros((1, S, M), np.int32) if M else None
    oracle.advance_state(pipes or [p], poc, 1, S, np.array([now], np.int64),
                         np.array(B, np.int32).reshape(1, S),
                         None if workers is None else np.array(workers, np.int32).reshape(1, S),
                         np.array(kept, np.uint32).reshape(1, S), fa, t, d, slot)
    return fa[0], t, d


def test_single_server_busy_period():
    """One request per batch: n admitted requests keep the server busy for n*d
    from the moment it is free (the later of now and free_at)."""
    p = util.pipeline([], 1, [10], bmax=4)
    assert advance(p, 1000, [1], [7], [1030])[0][0] == 1030 + 70      # still busy: continues from free_at
    assert advance(p, 1000, [1], [7], [400])[0][0] == 1000 + 70       # idle: starts now
    assert advance(p, 1000, [1], [0], [400])[0][0] == 1000            # nothing admitted: free from now on
    assert advance(p, 1000, [1], [0], [1030])[0][0] == 1030


def test_rounds_of_batch_times_workers():
    p = util.pipeline([], 1, [10], bmax=4)
    for kept, rounds in ((1, 1), (6, 1), (7, 2), (12, 2), (13, 3)):
        assert advance(p, 0, [3], [kept], [5], workers=[2])[0][0] == 5 + rounds * 10
    # the duration is the profile at the current batch size
    q = inputs.make_pipeline([], 1, [4], [np.array([10, 20, 30, 40], np.int64)])
    assert advance(q, 0, [3], [4], [0])[0][0] == 2 * 30


def test_recorded_sample_is_the_delay_met_now():
    p = util.pipeline(inputs.chain_edges(2), 2, [10, 20], bmax=2)
    fa, t, d = advance(p, 1000, [1, 2], [3, 0], [1250, 900], M=4, slot=2)
    assert list(t[0, 0]) == [-1, -1, 1000, -1] and list(d[0, 0]) == [0, 0, 250, 0]
    assert list(t[0, 1]) == [-1, -1, 1000, -1] and list(d[0, 1]) == [0, 0, 0, 0]     # idle stage: no delay
    fa, t, d = advance(p, 1000, [1, 2], [0, 0], [1000 + (1 << 30), 0], M=1, slot=0)
    assert d[0, 0, 0] == (1 << 24) - 1                                # capped to the sample range


@pytest.mark.parametrize("seed", range(10))
def test_new_free_at_is_when_the_planner_expects_the_last_admitted_request_to_finish_here(seed):
    """est of the last admitted request of a queue = its stage completion time + L_sub, and that
    completion time is where the stage becomes free."""
    rng = np.random.default_rng(2100 + seed)
    wl = util.random_small_workload(rng, int(rng.integers(50, 3000)), n_ctx=3)
    st, p = wl.state, wl.pipelines[0]
    S = st.stage_stride
    o = oracle.plan(wl.pipelines, wl.requests, st, wl.n_ctx, mode=0)
    fa = st.free_at_us.copy()
    oracle.advance_state(wl.pipelines, st.pipeline_of_ctx, wl.n_ctx, S, st.now_us, st.batch, st.workers,
                         o["seg_kept"], fa, None, None, 0)
    seen = 0
    for c in range(wl.n_ctx):
        for k in range(p.n_stages):
            seg = c * S + k
            lo, hi = int(o["seg_offsets"][seg]), int(o["seg_offsets"][seg + 1])
            kept_pos = [j for j in range(lo, hi) if o["keep"][j]]
            if not kept_pos:
                assert fa[c, k] == max(int(st.now_us[c]), int(st.free_at_us[c, k]))
                continue
            lsub = oracle.lsub(p, k, st.batch[c], st.q_us[c], st.w_us[c])
            assert fa[c, k] == int(o["est_us"][kept_pos[-1]]) - lsub
            seen += 1
    assert seen > 0


def test_padding_columns_and_bad_input():
    p = util.pipeline([], 1, [10], bmax=2)
    fa, _, _ = advance(p, 50, [1, 9, 9], [2, 5, 5], [0, 77, 88], S=3)
    assert list(fa) == [70, 77, 88]
    with pytest.raises(ValueError):
        advance(p, 0, [3], [1], [0])                                  # batch size beyond the profile
    with pytest.raises(ValueError):
        advance(p, 0, [1], [1], [0], workers=[0])
    with pytest.raises(ValueError):
        advance(p, 0, [1], [1], [0], M=2, slot=2)


@pytest.mark.parametrize("seed", range(3))
def test_replay_series_properties(seed):
    """The composed loop (queue delay -> plan -> advance): counts add up, time
    never runs backwards, and an overloaded stage starts dropping once its
    backlog has eaten the slack."""
    rng = np.random.default_rng(2200 + seed)
    job = util.small_replay_job(rng, n_inst=3, n_epochs=12, per_epoch=400)
    out = util.replay_with_oracle(job)
    assert out["total"].shape == (12, 3) and (out["kept"] <= out["total"]).all()
    assert (out["total"].sum(axis=1) == 400).all()
    assert (np.diff(out["free_at_series"], axis=0) >= 0).all()
    assert out["kept"].sum() < out["total"].sum() and out["kept"].sum() > 0
