"""pard_plan_static: the planner variant that allocates no device memory.

An inference server's control loop usually cannot call cudaMalloc: the serving
runtime owns all device memory, and an allocation from that loop may stall the
kernels that are serving requests.  For such callers the library keeps a fixed
scratch array inside its own image and offers pard_plan_static, which takes no
workspace.  This test drives it through the C ABI and requires the same bits as
pard_plan (with a caller-allocated workspace) on two consecutive calls, so that
whatever the first call leaves in the shared scratch is shown not to leak into
the second; both are also held against the CPU oracle, and the device's free
memory is read before and after a call to see that nothing was allocated.
Collected last on purpose: a failure here cannot hide other tests.
"""
import numpy as np
import pytest

from oracle import oracle
from paper_2602_08747_b200 import binding as pb
from paper_2602_08747_b200 import build as pbuild
from paper_2602_08747_b200 import inputs

pytestmark = pytest.mark.gpu

KEYS = ("keep", "est_us", "perm", "kept_idx", "seg_offsets", "seg_kept")


def _setup(wl):
    import torch
    pbuild.build()
    S = wl.state.stage_stride
    pipes = [pb.pard_load_pipeline(p) for p in wl.pipelines]
    d_req = pb.device_requests(wl.requests)
    d_state = pb.device_state(wl.state)
    stream = torch.cuda.current_stream().cuda_stream
    return S, pipes, d_req, d_state, stream


def _with_workspace(wl, mode):
    import torch
    S, pipes, d_req, d_state, stream = _setup(wl)
    out = pb.alloc_out(wl.n, wl.n_ctx * S)
    ws = pb.alloc_workspace(pb.pard_plan_workspace_bytes(wl.n, wl.n_ctx, S))
    pb.pard_plan(pipes, d_req, wl.n, d_state, wl.n_ctx, mode, out, ws, stream=stream)
    torch.cuda.synchronize()
    return pb.out_to_numpy(out, wl.n)


def _static(wl, mode):
    import torch
    S, pipes, d_req, d_state, stream = _setup(wl)
    out = pb.alloc_out(wl.n, wl.n_ctx * S)      # outputs are still the caller's
    for t in (out.keep, out.est_us, out.perm, out.kept_idx, out.seg_kept, out.seg_offsets):
        t.fill_(-1 if t.dtype != torch.uint8 else 255)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    pb.pard_plan_static(pipes, d_req, wl.n, d_state, wl.n_ctx, mode, out, stream=stream)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    res = pb.out_to_numpy(out, wl.n)
    res["free_bytes"] = (free_before, free_after)
    return res


def _same(got, want):
    assert got["n_kept"] == want["n_kept"]
    for k in KEYS:
        assert np.array_equal(got[k], want[k]), k


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    # first a multi-ctx problem that fills much of the scratch, then a small one
    # with a different shape: stale look-back words, histograms or sort buffers
    # of the first call would corrupt the second
    first = inputs.make("C5b", n_inst=12, per_inst=20_001)
    second = inputs.make("C1b")
    want_first, want_second = _with_workspace(first, 0), _with_workspace(second, 0)
    _same(_static(first, 0), want_first)
    got_second = _static(second, 0)
    _same(got_second, want_second)
    # the device had as much free memory after the call as before it (the very first call on a
    # device may load the library's kernels, so the second call is the one looked at)
    before, after = got_second["free_bytes"]
    assert after >= before
    # and the same problem twice, in the other position mode
    want = _with_workspace(first, 1)
    _same(_static(first, 1), want)
    again = _static(first, 1)
    _same(again, want)
    assert again["free_bytes"][1] >= again["free_bytes"][0]
    # the reference results themselves are the oracle's
    for wl, mode, got in ((first, 0, want_first), (second, 0, want_second), (first, 1, want)):
        _same(got, oracle.plan(wl.pipelines, wl.requests, wl.state, wl.n_ctx, mode))


def test_problem_larger_than_the_scratch_is_refused():
    import torch
    wl = inputs.make("C3", n=600_000)
    S, pipes, d_req, d_state, stream = _setup(wl)
    assert pb.pard_plan_workspace_bytes(wl.n, wl.n_ctx, S) > pb.PARD_STATIC_SCRATCH_BYTES
    out = pb.alloc_out(wl.n, wl.n_ctx * S)
    rc = pb.pard_plan_static(pipes, d_req, wl.n, d_state, wl.n_ctx, 0, out, stream=stream, check=False)
    assert rc == pb.PARD_ESTATIC
    torch.cuda.synchronize()
    # a problem that fits still runs afterwards
    small = inputs.make("C1")
    _same(_static(small, 0), _with_workspace(small, 0))
