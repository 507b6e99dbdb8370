"""The counter exchange of the multi-GPU path over NCCL, on the one GPU there is: a process
group of a single rank gathers and sums the per-ctx goodput counters of a planned shard (the
partitioning itself, and groups of several ranks, are covered on CPU with gloo)."""
import os
import socket

import numpy as np
import pytest

from oracle import oracle
from paper_2602_08747_b200 import binding as pb
from paper_2602_08747_b200 import inputs, sharding

pytestmark = pytest.mark.gpu


def test_counters_over_nccl_with_one_rank():
    import torch
    import torch.distributed as dist
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    os.environ.update({"MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port)})
    torch.cuda.set_device(0)
    try:
        dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda:0"))
    except Exception as e:                      # no usable NCCL set-up on this machine: nothing of ours to test
        pytest.skip("NCCL process group could not be created: %r" % (e,))
    try:
        for wl, mine, combine in (
                (inputs.make("C5b", n_inst=6, per_inst=4000),) * 2 + ("gather",),
                (inputs.make("C3b", n=30_000),) * 2 + ("sum",)):
            mine = sharding.shard_workload(wl, 1, 0) if combine == "gather" else sharding.shard_by_stage(wl, 1, 0)
            S = mine.state.stage_stride
            pipes = [pb.pard_load_pipeline(p) for p in mine.pipelines]
            out = pb.alloc_out(mine.n, mine.n_ctx * S)
            ws = pb.alloc_workspace(pb.pard_plan_workspace_bytes(mine.n, mine.n_ctx, S))
            total = torch.empty(mine.n_ctx, dtype=torch.int64, device="cuda")
            kept = torch.empty(mine.n_ctx, dtype=torch.int64, device="cuda")
            stream = torch.cuda.current_stream().cuda_stream
            pb.pard_plan(pipes, pb.device_requests(mine.requests), mine.n, pb.device_state(mine.state), mine.n_ctx, 0,
                         out, ws, stream=stream)
            pb.pard_goodput(None, out.seg_offsets, out.seg_kept, mine.n, mine.n_ctx, S, total, kept, stream=stream)
            if combine == "gather":
                tot, kp = sharding.gather_counters(total, kept, wl.n_ctx)
            else:
                tot, kp = sharding.sum_counters(total, kept)
            torch.cuda.synchronize()
            want = oracle.plan(wl.pipelines, wl.requests, wl.state, wl.n_ctx)
            assert np.array_equal(tot.cpu().numpy(), want["ctx_total"])
            assert np.array_equal(kp.cpu().numpy(), want["ctx_kept"])
    finally:
        dist.destroy_process_group()
