"""The multi-GPU path on CPU: two gloo ranks shard a job by ctx, plan their
shards independently (the oracle stands in for the GPU planner here) and gather
the goodput counters; the result equals planning the whole job at once."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import oracle
from paper_2602_08747_b200 import inputs, sharding


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = inputs.make("C5b", n_inst=5, per_inst=3000)
    mine = sharding.shard_workload(wl, world, rank)
    o = oracle.plan(mine.pipelines, mine.requests, mine.state, mine.n_ctx)
    tot, kept = sharding.gather_counters(torch.from_numpy(o["ctx_total"]), torch.from_numpy(o["ctx_kept"]),
                                         wl.n_ctx)
    # timing protocol of the benchmark: maximum over ranks
    t = torch.tensor([float(rank + 1)], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    np.savez(os.path.join(out_dir, "rank%d.npz" % rank), total=tot.numpy(), kept=kept.numpy(),
             tmax=t.numpy(), keep=o["keep"], est=o["est_us"], n=mine.n)
    dist.barrier()
    dist.destroy_process_group()


def _stage_worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = inputs.make("C3b", n=40_000)                 # one ctx, 16 stages: sharded by stage
    mine = sharding.shard_by_stage(wl, world, rank)
    o = oracle.plan(mine.pipelines, mine.requests, mine.state, mine.n_ctx)
    tot, kept = sharding.sum_counters(torch.from_numpy(o["ctx_total"]), torch.from_numpy(o["ctx_kept"]))
    # original indices: positions in the whole request array
    orig = np.flatnonzero((wl.requests["stage"] >= sharding.stage_range(16, world, rank)[0]) &
                          (wl.requests["stage"] < sharding.stage_range(16, world, rank)[1]))
    np.savez(os.path.join(out_dir, "rank%d.npz" % rank), total=tot.numpy(), kept=kept.numpy(), keep=o["keep"],
             est=o["est_us"], perm=orig[o["perm"]], kept_idx=orig[o["kept_idx"]], seg_kept=o["seg_kept"], n=mine.n)
    dist.barrier()
    dist.destroy_process_group()


def test_three_ranks_by_stage_equal_the_whole_job(tmp_path):
    world = 3
    mp.spawn(_stage_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    wl = inputs.make("C3b", n=40_000)
    whole = oracle.plan(wl.pipelines, wl.requests, wl.state, wl.n_ctx)
    parts = [np.load(tmp_path / ("rank%d.npz" % r)) for r in range(world)]
    for p in parts:                                   # every rank holds the summed counters
        assert np.array_equal(p["total"], whole["ctx_total"])
        assert np.array_equal(p["kept"], whole["ctx_kept"])
    assert sum(int(p["n"]) for p in parts) == wl.n
    for key, wkey in (("keep", "keep"), ("est", "est_us"), ("perm", "perm"), ("kept_idx", "kept_idx")):
        assert np.array_equal(np.concatenate([p[key] for p in parts]), whole[wkey]), key
    # every queue is planned by exactly one rank
    assert np.array_equal(sum(p["seg_kept"] for p in parts), whole["seg_kept"])


def test_ctx_ranges_partition_the_contexts():
    for n_ctx in (1, 2, 5, 256, 4096):
        for world in (1, 2, 3, 8):
            r = [sharding.ctx_range(n_ctx, world, k) for k in range(world)]
            assert r[0][0] == 0 and r[-1][1] == n_ctx
            assert all(r[k][1] == r[k + 1][0] for k in range(world - 1))
            sizes = [b - a for a, b in r]
            assert max(sizes) - min(sizes) <= 1


def test_two_ranks_equal_the_whole_job(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    wl = inputs.make("C5b", n_inst=5, per_inst=3000)
    whole = oracle.plan(wl.pipelines, wl.requests, wl.state, wl.n_ctx)
    parts = [np.load(tmp_path / ("rank%d.npz" % r)) for r in range(world)]
    for p in parts:                                   # every rank holds the full counters
        assert np.array_equal(p["total"], whole["ctx_total"])
        assert np.array_equal(p["kept"], whole["ctx_kept"])
        assert p["tmax"][0] == float(world)
    # service order is ctx-major, so the shards' outputs concatenate to the whole job's
    assert sum(int(p["n"]) for p in parts) == wl.n
    assert np.array_equal(np.concatenate([p["keep"] for p in parts]), whole["keep"])
    assert np.array_equal(np.concatenate([p["est"] for p in parts]), whole["est_us"])
