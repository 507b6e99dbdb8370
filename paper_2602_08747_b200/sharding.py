"""Sharding of a planning job over several GPUs (one process per GPU).

Contexts are independent planning problems (one pipeline instance at one
decision epoch), so a job shards by ctx with no exchange on the data path:
every rank plans a contiguous block of contexts on its own GPU.  A job with a
single ctx shards by stage instead: the queues of one ctx are independent once
every rank holds the ctx's (small) state rows, so every rank plans a contiguous
block of stages.  The only communication is the combination of the per-ctx
goodput counters: gathered (by ctx) or summed (by stage).  Host logic only; the
planning itself is `binding.pard_plan`.
"""
from __future__ import annotations

import numpy as np

from . import inputs


def ctx_range(n_ctx: int, world: int, rank: int):
    """Contiguous, balanced block of contexts of `rank` (first ranks get the remainder)."""
    base, rem = divmod(n_ctx, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def shard_workload(wl: inputs.Workload, world: int, rank: int) -> inputs.Workload:
    """The requests and state rows of this rank's contexts, ctx ids renumbered from 0.
    The relative order of the requests is kept, so ties are broken as in the whole job."""
    lo, hi = ctx_range(wl.n_ctx, world, rank)
    st = wl.state
    sel = (wl.requests["ctx"] >= lo) & (wl.requests["ctx"] < hi)
    req = wl.requests[sel].copy()
    req["ctx"] -= lo

    def rows(a):
        return None if a is None else np.ascontiguousarray(a[lo:hi])

    state = inputs.QueueState(st.stage_stride, st.slot_stride, rows(st.now_us), rows(st.batch),
                              rows(st.free_at_us), rows(st.q_us), rows(st.w_us), rows(st.workers),
                              rows(st.pipeline_of_ctx), rows(st.priority))
    return inputs.Workload("%s[%d/%d]" % (wl.name, rank, world), wl.pipelines, req, state, hi - lo,
                           dict(wl.notes))


def stage_range(n_stages: int, world: int, rank: int):
    """Contiguous, balanced block of stages of `rank`."""
    return ctx_range(n_stages, world, rank)


def shard_by_stage(wl: inputs.Workload, world: int, rank: int) -> inputs.Workload:
    """The requests queued at this rank's block of stages; contexts, stage ids and the whole
    state are kept (L_sub of a stage reads the rows of the stages downstream of it), so segment
    ids mean the same on every rank and the queues of the other ranks' stages are simply empty
    here.  Service order is (ctx, stage)-major: with one ctx the ranks' outputs, in rank order,
    concatenate to the whole job's; per-ctx counters add up over the ranks."""
    lo, hi = stage_range(wl.state.stage_stride, world, rank)
    sel = (wl.requests["stage"] >= lo) & (wl.requests["stage"] < hi)
    req = np.ascontiguousarray(wl.requests[sel])
    return inputs.Workload("%s[stages %d/%d]" % (wl.name, rank, world), wl.pipelines, req, wl.state, wl.n_ctx,
                           dict(wl.notes))


def sum_counters(total, kept, group=None):
    """Per-ctx (total, kept) counters of a job sharded by stage: the sum over the ranks, on
    every rank (one all-reduce of 2 * n_ctx int64 values)."""
    import torch
    import torch.distributed as dist
    both = torch.stack([total, kept])
    dist.all_reduce(both, op=dist.ReduceOp.SUM, group=group)
    return both[0], both[1]


def gather_counters(total, kept, n_ctx: int, group=None):
    """All ranks' per-ctx (total, kept) counters in ctx order, on every rank.
    `total` and `kept` are this rank's int64 tensors; uses torch.distributed."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group)
    sizes = [ctx_range(n_ctx, world, r)[1] - ctx_range(n_ctx, world, r)[0] for r in range(world)]
    width = max(sizes) if sizes else 0
    mine = torch.zeros(2, width, dtype=torch.int64, device=total.device)
    mine[0, :total.numel()] = total
    mine[1, :kept.numel()] = kept
    parts = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(parts, mine, group=group)
    tot = torch.cat([p[0, :sizes[r]] for r, p in enumerate(parts)])
    kp = torch.cat([p[1, :sizes[r]] for r, p in enumerate(parts)])
    return tot, kp
