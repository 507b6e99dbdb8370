"""Parity of the closed-loop replay on the GPU (pard_update_queue_delay ->
pard_plan -> pard_goodput -> pard_advance_state, chained on one stream for every
epoch) with the same loop composed of oracle calls: the goodput series, the
final state and the recorded samples, bit for bit."""
import numpy as np
import pytest

from oracle import oracle
from paper_2602_08747_b200 import binding as pb
from paper_2602_08747_b200 import inputs, replay
from tests import util

pytestmark = pytest.mark.gpu


def run_gpu(job, max_req):
    pipes = [pb.pard_load_pipeline(p) for p in job["pipelines"]]
    rp = replay.Replay(pipes, job["pipeline_of_ctx"], job["n_ctx"], job["S"], job["R"], job["batch"],
                       job["workers"], job["free_at0"], job["w"], job["priority"], job["n_samples"],
                       job["window_us"], max_req, "cuda:0")
    res = replay.run(rp, job["epochs"])
    for p in pipes:
        p.free()
    return res


@pytest.mark.parametrize("seed,n_inst,n_epochs,per_epoch", [(0, 3, 12, 400), (1, 1, 30, 2500), (2, 16, 20, 9000)])
def test_replay_matches_the_oracle_loop(seed, n_inst, n_epochs, per_epoch):
    rng = np.random.default_rng(3100 + seed)
    job = util.small_replay_job(rng, n_inst, n_epochs, per_epoch)
    if seed == 2:
        job["priority"] = rng.integers(0, 2, size=(n_inst, job["S"])).astype(np.uint8)
    want = util.replay_with_oracle(job)
    got = run_gpu(job, per_epoch)
    assert got.status == 0
    assert np.array_equal(got.total, want["total"])
    assert np.array_equal(got.kept, want["kept"])
    assert np.array_equal(got.free_at_us, want["free_at"])
    assert np.array_equal(got.sample_time_us, want["sample_time"])
    assert np.array_equal(got.sample_delay_us, want["sample_delay"])
    assert 0 < want["kept"].sum() < want["total"].sum()


def test_advance_state_alone_and_its_device_checks():
    import torch
    rng = np.random.default_rng(9)
    wl = inputs.make("C5b", n_inst=20, per_inst=3000)
    st = wl.state
    S, M = st.stage_stride, 5
    kept = rng.integers(0, 5000, size=(wl.n_ctx, S)).astype(np.uint32)
    fa = st.free_at_us.copy()
    t = np.full((wl.n_ctx, S, M), -1, np.int64)
    d = np.zeros((wl.n_ctx, S, M), np.int32)
    oracle.advance_state(wl.pipelines, st.pipeline_of_ctx, wl.n_ctx, S, st.now_us, st.batch, st.workers, kept, fa,
                         t, d, 3)
    dev = "cuda:0"
    pipes = [pb.pard_load_pipeline(p) for p in wl.pipelines]
    ds = pb.device_state(st, dev)
    d_kept = torch.from_numpy(kept.view(np.int32)).to(dev)
    d_t = torch.full((wl.n_ctx, S, M), -1, dtype=torch.int64, device=dev)
    d_d = torch.zeros((wl.n_ctx, S, M), dtype=torch.int32, device=dev)
    ws = pb.alloc_workspace(pb.pard_advance_state_workspace_bytes(len(pipes)), dev)
    pb.pard_advance_state(pipes, ds.pipeline_of_ctx, wl.n_ctx, S, ds.now_us, ds.batch, ds.workers, d_kept,
                          ds.free_at_us, d_t, d_d, M, 3, 0, ws)
    assert np.array_equal(ds.free_at_us.cpu().numpy(), fa)
    assert np.array_equal(d_t.cpu().numpy(), t) and np.array_equal(d_d.cpu().numpy(), d)
    # without a sample ring only free_at moves
    fa2 = fa.copy()
    oracle.advance_state(wl.pipelines, st.pipeline_of_ctx, wl.n_ctx, S, st.now_us, st.batch, st.workers, kept, fa2,
                         None, None, 0)
    pb.pard_advance_state(pipes, ds.pipeline_of_ctx, wl.n_ctx, S, ds.now_us, ds.batch, ds.workers, d_kept,
                          ds.free_at_us, None, None, 0, 0, 0, ws)
    assert np.array_equal(ds.free_at_us.cpu().numpy(), fa2)
    # a batch size outside the profile is reported, the context stays usable
    ds.batch[0, 0] = 10**6
    rc = pb.pard_advance_state(pipes, ds.pipeline_of_ctx, wl.n_ctx, S, ds.now_us, ds.batch, ds.workers, d_kept,
                               ds.free_at_us, None, None, 0, 0, 0, ws, check=False)
    assert rc == pb.PARD_EDATA
    for p in pipes:
        p.free()
