"""Runs a workload through the C-ABI CUDA library and returns numpy outputs."""
from __future__ import annotations

import numpy as np

from paper_2602_08747_b200 import binding as pb
from paper_2602_08747_b200 import build as pbuild


def run_library(wl, mode=0, check=True, arrivals=None):
    import torch
    pbuild.build()
    assert torch.cuda.is_available()
    dev = "cuda:0"
    pipes = [pb.pard_load_pipeline(p) for p in wl.pipelines]
    S = wl.state.stage_stride
    n_seg = wl.n_ctx * S
    d_req = pb.device_requests(wl.requests, dev)
    d_state = pb.device_state(wl.state, dev)
    out = pb.alloc_out(wl.n, n_seg, dev)
    ws = pb.alloc_workspace(pb.pard_plan_workspace_bytes(wl.n, wl.n_ctx, S), dev)
    stream = torch.cuda.current_stream().cuda_stream
    if arrivals is not None or mode & (pb.PARD_MODE_PATH_MASK | pb.PARD_MODE_FCFS | pb.PARD_MODE_NEXUS | pb.PARD_MODE_CLIPPER):
        d_arr = None if arrivals is None else pb.device_requests(arrivals, dev)      # 16-byte records as well
        rc = pb.pard_plan_policy(pipes, d_req, d_arr, wl.n, d_state, wl.n_ctx, mode, out, ws, stream=stream,
                                 check=check)
    else:
        rc = pb.pard_plan(pipes, d_req, wl.n, d_state, wl.n_ctx, mode, out, ws, stream=stream, check=check)
    if rc != pb.PARD_OK:
        return rc, None
    total = torch.empty(wl.n_ctx, dtype=torch.int64, device=dev)
    kept = torch.empty(wl.n_ctx, dtype=torch.int64, device=dev)
    # the counters both ways: from the per-queue kept counts, and by counting the keep flags
    pb.pard_goodput(None, out.seg_offsets, out.seg_kept, wl.n, wl.n_ctx, S, total, kept, stream=stream)
    total2, kept2 = torch.empty_like(total), torch.empty_like(kept)
    pb.pard_goodput(out.keep, out.seg_offsets, None, wl.n, wl.n_ctx, S, total2, kept2, stream=stream)
    torch.cuda.synchronize()
    res = pb.out_to_numpy(out, wl.n)
    res["ctx_total"] = total.cpu().numpy()
    res["ctx_kept"] = kept.cpu().numpy()
    res["ctx_total_from_flags"] = total2.cpu().numpy()
    res["ctx_kept_from_flags"] = kept2.cpu().numpy()
    for p in pipes:
        p.free()
    return rc, res


KEYS = ["seg_offsets", "perm", "keep", "est_us", "n_kept", "kept_idx", "seg_kept", "ctx_total", "ctx_kept"]


def assert_identical(got, want):
    """Bit-exact comparison of every output (all of them are integers)."""
    for k in ("ctx_total", "ctx_kept"):           # the second way of counting, against the oracle too
        if k + "_from_flags" in got:
            assert np.array_equal(got[k + "_from_flags"], want[k]), k + "_from_flags"
    for k in KEYS:
        g, w = got[k], want[k]
        if isinstance(w, (int, np.integer)):
            assert int(g) == int(w), k
        else:
            assert g.shape == w.shape, (k, g.shape, w.shape)
            if not np.array_equal(g, w):
                bad = np.flatnonzero(g != w)
                raise AssertionError("%s differs at %d positions, first %d: got %s want %s"
                                     % (k, bad.size, bad[0], g[bad[0]], w[bad[0]]))


def run_estimate_w(wl, samples, lambda_num, lambda_den, seed, slot_stride=None, check=True, fill=-7):
    """pard_estimate_w on cuda:0; returns (status, w [n_ctx, slot_stride] as numpy).
    The output buffer is pre-filled with `fill` so that untouched entries show."""
    import torch
    pbuild.build()
    dev = "cuda:0"
    pipes = [pb.pard_load_pipeline(p) for p in wl.pipelines]
    st = wl.state
    R = slot_stride or st.slot_stride
    d_samples = torch.from_numpy(np.ascontiguousarray(samples, dtype=np.int32)).to(dev)
    d_poc = None if st.pipeline_of_ctx is None else torch.from_numpy(st.pipeline_of_ctx.astype(np.int32)).to(dev)
    d_w = torch.full((wl.n_ctx, R), fill, dtype=torch.int64, device=dev)
    ws = pb.alloc_workspace(pb.pard_estimate_w_workspace_bytes(len(pipes)), dev)
    stream = torch.cuda.current_stream().cuda_stream
    rc = pb.pard_estimate_w(pipes, d_poc, wl.n_ctx, st.stage_stride, R, d_samples, int(samples.shape[2]),
                            lambda_num, lambda_den, seed, 0, d_w, ws, stream=stream, check=check)
    torch.cuda.synchronize()
    w = d_w.cpu().numpy()
    for p in pipes:
        p.free()
    return rc, w


def run_update_priority(pipelines, pipeline_of_ctx, n_ctx, S, batch, workers, arrivals, window, interval_us,
                        priority, check=True):
    """pard_update_priority on cuda:0; returns (status, new priorities [n_ctx, S] as numpy)."""
    import torch
    pbuild.build()
    dev = "cuda:0"
    pipes = [pb.pard_load_pipeline(p) for p in pipelines]

    def mv(a, dt):
        return None if a is None else torch.from_numpy(np.ascontiguousarray(a, dtype=dt)).to(dev)

    x = np.ascontiguousarray(arrivals, dtype=np.uint32)
    d_prio = mv(np.asarray(priority, dtype=np.uint8).reshape(n_ctx, S), np.uint8)
    ws = pb.alloc_workspace(pb.pard_update_priority_workspace_bytes(len(pipes)), dev)
    stream = torch.cuda.current_stream().cuda_stream
    rc = pb.pard_update_priority(pipes, mv(pipeline_of_ctx, np.int32), n_ctx, S, mv(batch, np.int32),
                                 mv(workers, np.int32), mv(x.view(np.int32), np.int32), int(x.shape[2]), window,
                                 interval_us, 0, d_prio, ws, stream=stream, check=check)
    torch.cuda.synchronize()
    out = d_prio.cpu().numpy()
    for p in pipes:
        p.free()
    return rc, out


def run_queue_delay(now_us, sample_time_us, sample_delay_us, window_us, check=True):
    """pard_update_queue_delay on cuda:0; returns (status, q [n_ctx, S] as numpy)."""
    import torch
    pbuild.build()
    dev = "cuda:0"
    t = np.ascontiguousarray(sample_time_us, dtype=np.int64)
    d = np.ascontiguousarray(sample_delay_us, dtype=np.int32)
    n_ctx, S, M = t.shape
    d_t = torch.from_numpy(t).to(dev) if M else None
    d_d = torch.from_numpy(d).to(dev) if M else None
    d_now = torch.from_numpy(np.ascontiguousarray(now_us, dtype=np.int64)).to(dev)
    d_q = torch.full((n_ctx, S), -7, dtype=torch.int64, device=dev)
    ws = pb.alloc_workspace(pb.pard_update_queue_delay_workspace_bytes(), dev)
    rc = pb.pard_update_queue_delay(n_ctx, S, d_now, d_t, d_d, M, window_us, 0, d_q, ws,
                                    stream=torch.cuda.current_stream().cuda_stream, check=check)
    torch.cuda.synchronize()
    return rc, d_q.cpu().numpy()
