"""The benchmark's own launcher (python bench.py --gpus N without torchrun), on CPU: it starts
one process per rank with the rendezvous environment set, the ranks find each other, and a
world size that does not match --gpus is refused."""
import argparse
import json
import os

import pytest
import torch
import torch.distributed as dist

import bench


def _probe(out_dir):
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    assert os.environ["MASTER_ADDR"] == "127.0.0.1" and int(os.environ["LOCAL_RANK"]) == rank
    dist.init_process_group("gloo")
    t = torch.tensor([float(rank + 1)], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)                   # the benchmark's max-over-ranks timing
    with open(os.path.join(out_dir, "rank%d.json" % rank), "w") as f:
        json.dump({"rank": rank, "world": dist.get_world_size(), "n_gpus": world, "tmax": float(t.item())}, f)
    dist.barrier()
    dist.destroy_process_group()


def test_launcher_starts_one_rank_per_gpu(tmp_path):
    bench.spawn_ranks(3, _probe, (str(tmp_path),))
    got = [json.load(open(tmp_path / ("rank%d.json" % r))) for r in range(3)]
    assert [g["rank"] for g in got] == [0, 1, 2]
    assert all(g["world"] == 3 and g["n_gpus"] == 3 and g["tmax"] == 3.0 for g in got)


def test_world_size_must_match_gpus(monkeypatch):
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    args = argparse.Namespace(gpus=2, steps=1, warmup=3, impl="ours")
    with pytest.raises(SystemExit) as e:
        bench.run_ours(args)                                   # one process, but two GPUs asked for
    assert "--gpus 2" in str(e.value)
