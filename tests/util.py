"""Small builders shared by the tests (inputs only, no planner arithmetic)."""
from __future__ import annotations

import os

import numpy as np

from paper_2602_08747_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_golden(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


def const_profile(n_stages, d_list, bmax=4):
    """d_k(b) = d_list[k] for every b."""
    return [np.full(bmax, d_list[k], dtype=np.int64) for k in range(n_stages)]


def pipeline(edges, n_stages, d_list, bmax=4):
    return inputs.make_pipeline(edges, n_stages, [bmax] * n_stages,
                                const_profile(n_stages, d_list, bmax))


def state(n_ctx, S, R, now, batch, free_at=None, q=None, w=None, workers=None, poc=None):
    now = np.broadcast_to(np.asarray(now, dtype=np.int64), (n_ctx,)).copy()
    b = np.broadcast_to(np.asarray(batch, dtype=np.int32), (n_ctx, S)).copy()
    fa = (np.zeros((n_ctx, S), np.int64) if free_at is None
          else np.broadcast_to(np.asarray(free_at, dtype=np.int64), (n_ctx, S)).copy())
    qq = (np.zeros((n_ctx, S), np.int64) if q is None
          else np.broadcast_to(np.asarray(q, dtype=np.int64), (n_ctx, S)).copy())
    ww = None if w is None else np.broadcast_to(np.asarray(w, dtype=np.int64), (n_ctx, R)).copy()
    mm = None if workers is None else np.broadcast_to(np.asarray(workers, dtype=np.int32),
                                                      (n_ctx, S)).copy()
    pc = None if poc is None else np.asarray(poc, dtype=np.int32)
    return inputs.QueueState(S, max(R, 1), now, b, fa, qq, ww, mm, pc)


def requests(deadline, stage=0, ctx=0):
    deadline = np.asarray(deadline, dtype=np.int64)
    r = np.zeros(len(deadline), dtype=inputs.REQUEST_DTYPE)
    r["deadline_us"] = deadline
    r["stage"] = stage
    r["ctx"] = ctx
    return r


def arrivals(arrive, slo):
    arrive = np.asarray(arrive, dtype=np.int64)
    a = np.zeros(len(arrive), dtype=inputs.ARRIVAL_DTYPE)
    a["arrive_us"] = arrive
    a["slo_us"] = slo
    return a


def explicit_paths(p, stage):
    """Every downstream path of `stage` as a tuple of stage ids, sorted
    lexicographically (written independently of the oracle and the library)."""
    out = []

    def rec(k, prefix):
        prefix = prefix + (int(k),)
        succ = sorted(int(j) for j in p.successors(k))
        if not succ:
            out.append(prefix)
        for j in succ:
            rec(j, prefix)

    for j in sorted(int(j) for j in p.successors(stage)):
        rec(j, ())
    return sorted(out)


def random_small_workload(rng, n, n_ctx=1, max_stages=5, keepish=True):
    """A small random DAG workload with a healthy mix of keeps and drops."""
    S = int(rng.integers(1, max_stages + 1))
    edges = inputs.random_dag_edges(rng, S) if S >= 2 else []
    bmax = int(rng.integers(1, 9))
    tables = [rng.integers(1, 60, size=bmax).astype(np.int64) for _ in range(S)]
    p = inputs.make_pipeline(edges, S, [bmax] * S, tables)
    R = max(1, inputs.n_slots(p))
    now = rng.integers(1000, 2000, size=n_ctx)
    st = state(n_ctx, S, R, now, rng.integers(1, bmax + 1, size=(n_ctx, S)),
               free_at=now[:, None] + rng.integers(-50, 50, size=(n_ctx, S)),
               q=rng.integers(0, 30, size=(n_ctx, S)),
               w=rng.integers(0, 40, size=(n_ctx, R)),
               workers=rng.integers(1, 3, size=(n_ctx, S)))
    span = 400 if keepish else 50
    r = requests(now[rng.integers(0, n_ctx, size=n)] * 0 + rng.integers(900, 2000 + span * S, size=n),
                 stage=rng.integers(0, S, size=n), ctx=rng.integers(0, n_ctx, size=n))
    return inputs.Workload("rand", [p], r, st, n_ctx)


# --------------------------------------------------------------------------
# closed-loop replay: a job (inputs only) and the loop composed of oracle calls
# --------------------------------------------------------------------------
def small_replay_job(rng, n_inst, n_epochs, per_epoch, n_samples=8, window_us=200_000):
    """n_inst independent pipeline instances (one ctx each) observed over
    n_epochs decision epochs; every epoch brings per_epoch new requests spread
    over the instances and stages.  Durations are sized so that some stages are
    overloaded and start dropping after a few epochs."""
    S = 3
    tables = [rng.integers(200, 900, size=4).astype(np.int64) for _ in range(S)]
    p = inputs.make_pipeline(inputs.chain_edges(S), S, [4] * S, tables)
    R = max(1, inputs.n_slots(p))
    epoch_len = 20_000
    now0 = 1_000_000
    batch = rng.integers(1, 5, size=(n_inst, S)).astype(np.int32)
    workers = rng.integers(1, 3, size=(n_inst, S)).astype(np.int32)
    epochs = []
    for e in range(n_epochs):
        now = np.full(n_inst, now0 + e * epoch_len, np.int64) + rng.integers(0, 50, size=n_inst)
        ctx = rng.integers(0, n_inst, size=per_epoch)
        r = requests(now[ctx] + rng.integers(-2000, 40_000, size=per_epoch),
                     stage=rng.integers(0, S, size=per_epoch), ctx=ctx)
        epochs.append((now, r))
    return {"pipelines": [p], "pipeline_of_ctx": None, "n_ctx": n_inst, "S": S, "R": R, "batch": batch,
            "workers": workers, "free_at0": np.full((n_inst, S), now0 - 5, np.int64),
            "w": rng.integers(0, 300, size=(n_inst, R)).astype(np.int64), "epochs": epochs,
            "n_samples": n_samples, "window_us": window_us, "priority": None}


def replay_with_oracle(job):
    """The closed loop, one epoch after the other, composed of oracle calls only:
    q from the recorded delays, the plan, then the state carried forward."""
    from oracle import oracle
    n_ctx, S, M = job["n_ctx"], job["S"], job["n_samples"]
    free_at = job["free_at0"].copy()
    t = np.full((n_ctx, S, M), -1, np.int64)
    d = np.zeros((n_ctx, S, M), np.int32)
    total, kept, fa_series, q_series = [], [], [], []
    for e, (now, req) in enumerate(job["epochs"]):
        q = oracle.queue_delay(now, t, d, job["window_us"])
        st = inputs.QueueState(S, job["R"], now, job["batch"], free_at.copy(), q, job["w"], job["workers"],
                               job["pipeline_of_ctx"], job["priority"])
        o = oracle.plan(job["pipelines"], req, st, n_ctx)
        oracle.advance_state(job["pipelines"], job["pipeline_of_ctx"], n_ctx, S, now, job["batch"],
                             job["workers"], o["seg_kept"], free_at, t, d, e % M)
        total.append(o["ctx_total"])
        kept.append(o["ctx_kept"])
        fa_series.append(free_at.copy())
        q_series.append(q)
    return {"total": np.array(total), "kept": np.array(kept), "free_at_series": np.array(fa_series),
            "q_series": np.array(q_series), "free_at": free_at, "sample_time": t, "sample_delay": d}
