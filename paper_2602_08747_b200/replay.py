"""Closed-loop replay of a workload over many decision epochs, on the device.

Every epoch chains four C-ABI calls on one stream, with no host round trip in
between: pard_update_queue_delay (q from the recorded delays), pard_plan (the
drop decisions of the epoch's queued requests), pard_goodput (the epoch's row of
the goodput series) and pard_advance_state (free_at and the delay samples for
the next epoch).  This module only owns device buffers and issues the calls; it
computes nothing itself."""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np

from . import binding as pb


@dataclass
class ReplayResult:
    total: np.ndarray          # int64 [n_epochs, n_ctx] queued requests
    kept: np.ndarray           # int64 [n_epochs, n_ctx] requests predicted to finish within their SLO
    free_at_us: np.ndarray     # int64 [n_ctx, S] state after the last epoch
    sample_time_us: np.ndarray
    sample_delay_us: np.ndarray
    status: int


class Replay:
    """Device-resident state of a replay of n_ctx independent pipeline instances."""

    def __init__(self, pipelines: Sequence[pb.Pipeline], pipeline_of_ctx, n_ctx: int, stage_stride: int,
                 slot_stride: int, batch, workers, free_at_us, w_us, priority=None, n_samples: int = 64,
                 window_us: int = 5_000_000, max_requests_per_epoch: int = 1 << 20, device="cuda"):
        import torch
        self.torch = torch
        self.dev = device
        self.pipes = list(pipelines)
        self.n_ctx, self.S, self.R, self.M, self.window = n_ctx, stage_stride, slot_stride, n_samples, window_us

        def mv(a, dt):
            return None if a is None else torch.from_numpy(np.ascontiguousarray(a, dtype=dt)).to(device)

        self.poc = mv(pipeline_of_ctx, np.int32)
        self.state = pb.QueueStateArrays(stage_stride, slot_stride,
                                         torch.zeros(n_ctx, dtype=torch.int64, device=device),
                                         mv(batch, np.int32), mv(free_at_us, np.int64),
                                         torch.zeros((n_ctx, stage_stride), dtype=torch.int64, device=device),
                                         mv(w_us, np.int64), mv(workers, np.int32), self.poc,
                                         mv(priority, np.uint8))
        self.sample_time = torch.full((n_ctx, stage_stride, max(n_samples, 1)), -1, dtype=torch.int64, device=device)
        self.sample_delay = torch.zeros((n_ctx, stage_stride, max(n_samples, 1)), dtype=torch.int32, device=device)
        self.cap = max_requests_per_epoch
        n_seg = n_ctx * stage_stride
        self.out = pb.alloc_out(self.cap, n_seg, device)
        self.ws_plan = pb.alloc_workspace(pb.pard_plan_workspace_bytes(self.cap, n_ctx, stage_stride), device)
        self.ws_q = pb.alloc_workspace(pb.pard_update_queue_delay_workspace_bytes(), device)
        self.ws_adv = pb.alloc_workspace(pb.pard_advance_state_workspace_bytes(len(self.pipes)), device)
        self.stream = torch.cuda.current_stream().cuda_stream
        self.epoch = 0

    def step(self, d_now_us, d_requests, n: int, d_total_row, d_kept_row) -> None:
        """One epoch; everything is enqueued, nothing is waited for."""
        assert n <= self.cap
        st = self.state
        st.now_us = d_now_us
        nw = pb.PARD_MODE_NOWAIT
        pb.pard_update_queue_delay(self.n_ctx, self.S, d_now_us, self.sample_time, self.sample_delay,
                                   self.M, self.window, nw, st.q_us, self.ws_q, stream=self.stream)
        pb.pard_plan(self.pipes, d_requests, n, st, self.n_ctx, nw, self.out, self.ws_plan, stream=self.stream)
        pb.pard_goodput(None, self.out.seg_offsets, self.out.seg_kept, n, self.n_ctx, self.S, d_total_row, d_kept_row,
                        stream=self.stream)
        pb.pard_advance_state(self.pipes, self.poc, self.n_ctx, self.S, d_now_us, st.batch, st.workers,
                              self.out.seg_kept, st.free_at_us, self.sample_time, self.sample_delay, self.M,
                              self.epoch % self.M if self.M else 0, nw, self.ws_adv, stream=self.stream)
        self.epoch += 1

    def statuses(self) -> int:
        """Waits for the stream; the first non-zero status of the last epoch's calls, else 0."""
        for ws in (self.ws_q, self.ws_plan, self.ws_adv):
            rc = pb.pard_plan_status(ws, self.stream)
            if rc != pb.PARD_OK:
                return rc
        return pb.PARD_OK


def run(replay: Replay, epochs: List) -> ReplayResult:
    """epochs: list of (now_us int64 [n_ctx], requests REQUEST_DTYPE [n_e]) host arrays; they are
    copied to the device up front, then all epochs are enqueued back to back."""
    torch = replay.torch
    dev = replay.dev
    E = len(epochs)
    d_now = torch.from_numpy(np.ascontiguousarray(np.stack([e[0] for e in epochs]), dtype=np.int64)).to(dev)
    d_req = [pb.device_requests(e[1], dev) for e in epochs]
    total = torch.zeros((E, replay.n_ctx), dtype=torch.int64, device=dev)
    kept = torch.zeros((E, replay.n_ctx), dtype=torch.int64, device=dev)
    status = pb.PARD_OK
    for i in range(E):
        replay.step(d_now[i], d_req[i], int(epochs[i][1].shape[0]), total[i], kept[i])
        if (i & 63) == 63 or i == E - 1:       # a status word only holds the latest call: look now and then
            status = status or replay.statuses()
    torch.cuda.synchronize()
    return ReplayResult(total.cpu().numpy(), kept.cpu().numpy(), replay.state.free_at_us.cpu().numpy(),
                        replay.sample_time.cpu().numpy(), replay.sample_delay.cpu().numpy(), status)
