"""Seeded synthetic inputs for the PARD drop planner.

This module only *draws inputs*: pipelines (stage graph + latency profile),
queued requests and the runtime state a State Planner would have synchronised.
It holds none of the planner's arithmetic (no ordering, no wait or path
estimate, no drop rule) and imports neither the CUDA binding nor the CPU
oracle; both sides of a parity test are fed the arrays produced here.

The five workloads stand in for the paper's evaluation inputs (Sec. 5.1,
Workload): 3-5 stage chains and one diamond-shaped DAG application, request
traces that are periodic or bursty, SLOs of a few hundred milliseconds, batch
wait uniform between 0 and the stage duration (Sec. 3.2, Fig. 3b).  Only the
shape of those workloads is reproduced; the traces themselves are not used.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

REQUEST_DTYPE = np.dtype(
    {"names": ["deadline_us", "ctx", "stage", "flags"],
     "formats": ["<i8", "<u4", "<u2", "<u2"],
     "offsets": [0, 8, 12, 14], "itemsize": 16})

# when a request reached its current module, and its end-to-end objective (only
# the Clipper++ comparison rule reads these)
ARRIVAL_DTYPE = np.dtype({"names": ["arrive_us", "slo_us"], "formats": ["<i8", "<i8"],
                          "offsets": [0, 8], "itemsize": 16})


@dataclass
class Pipeline:
    """Stage graph (successor lists in CSR form) and latency profile d_k(b)."""
    n_stages: int
    sub_offsets: np.ndarray   # int32 [n_stages+1]
    sub_ids: np.ndarray       # int32
    bmax: np.ndarray          # int32 [n_stages]
    lat_offsets: np.ndarray   # int64 [n_stages+1]
    lat_us: np.ndarray        # int64, d_k(b) at lat_offsets[k] + b - 1

    def successors(self, k: int) -> np.ndarray:
        return self.sub_ids[self.sub_offsets[k]:self.sub_offsets[k + 1]]

    def latency(self, k: int, b: int) -> int:
        return int(self.lat_us[self.lat_offsets[k] + b - 1])


@dataclass
class QueueState:
    stage_stride: int
    slot_stride: int
    now_us: np.ndarray                        # int64 [n_ctx]
    batch: np.ndarray                         # int32 [n_ctx, stage_stride]
    free_at_us: np.ndarray                    # int64 [n_ctx, stage_stride]
    q_us: np.ndarray                          # int64 [n_ctx, stage_stride]
    w_us: Optional[np.ndarray] = None         # int64 [n_ctx, slot_stride]
    workers: Optional[np.ndarray] = None      # int32 [n_ctx, stage_stride]
    pipeline_of_ctx: Optional[np.ndarray] = None   # int32 [n_ctx]
    priority: Optional[np.ndarray] = None     # uint8 [n_ctx, stage_stride]; 0 low / 1 high budget first


@dataclass
class Workload:
    name: str
    pipelines: List[Pipeline]
    requests: np.ndarray      # REQUEST_DTYPE [n]
    state: QueueState
    n_ctx: int
    notes: dict = field(default_factory=dict)

    @property
    def n(self) -> int:
        return int(self.requests.shape[0])


# --------------------------------------------------------------------------
# graph helpers (input structure only)
# --------------------------------------------------------------------------
def make_pipeline(edges, n_stages, bmax, tables) -> Pipeline:
    """edges: iterable of (from, to); tables: list of int64 arrays d_k(1..bmax_k)."""
    succ = [[] for _ in range(n_stages)]
    for a, b in edges:
        succ[a].append(b)
    offs = np.zeros(n_stages + 1, dtype=np.int32)
    ids = []
    for k in range(n_stages):
        ids.extend(succ[k])
        offs[k + 1] = len(ids)
    lat_offsets = np.zeros(n_stages + 1, dtype=np.int64)
    for k in range(n_stages):
        assert len(tables[k]) == bmax[k]
        lat_offsets[k + 1] = lat_offsets[k] + bmax[k]
    return Pipeline(n_stages, offs, np.asarray(ids, dtype=np.int32),
                    np.asarray(bmax, dtype=np.int32), lat_offsets,
                    np.concatenate([np.asarray(t, dtype=np.int64) for t in tables])
                    if n_stages else np.zeros(0, np.int64))


def paths_to_sink(p: Pipeline) -> np.ndarray:
    """Number of stage sequences from each stage to a sink (1 for a sink)."""
    cnt = np.zeros(p.n_stages, dtype=np.int64)
    order = _topological_order(p)
    for k in reversed(order):
        s = p.successors(k)
        cnt[k] = 1 if len(s) == 0 else int(sum(cnt[j] for j in s))
    return cnt


def n_slots(p: Pipeline) -> int:
    """Number of (stage, downstream path) pairs: the length of one w row."""
    cnt = paths_to_sink(p)
    return int(sum(sum(cnt[j] for j in p.successors(k)) for k in range(p.n_stages)))


def n_source_sink_paths(p: Pipeline) -> int:
    has_pred = np.zeros(p.n_stages, dtype=bool)
    has_pred[p.sub_ids] = True
    cnt = paths_to_sink(p)
    return int(sum(cnt[k] for k in range(p.n_stages) if not has_pred[k]))


def _topological_order(p: Pipeline):
    indeg = np.zeros(p.n_stages, dtype=np.int64)
    for j in p.sub_ids:
        indeg[j] += 1
    ready = [k for k in range(p.n_stages) if indeg[k] == 0]
    order = []
    while ready:
        k = ready.pop()
        order.append(k)
        for j in p.successors(k):
            indeg[j] -= 1
            if indeg[j] == 0:
                ready.append(int(j))
    assert len(order) == p.n_stages, "graph has a cycle"
    return order


def chain_edges(n):
    return [(i, i + 1) for i in range(n - 1)]


# 8 stages, branch after the first stage into {1->2, 3, 4}, rejoin at stage 5:
# three source-to-sink paths.
DAG8_EDGES = [(0, 1), (0, 3), (0, 4), (1, 2), (2, 5), (3, 5), (4, 5), (5, 6), (6, 7)]

# 16 stages, 12 source-to-sink paths, fan-out <= 3: the source splits into two
# branches, each holding a 3-wide diamond; they merge, a 2-wide diamond
# follows, then a tail stage.
DAG16_EDGES = [(0, 1), (0, 6),
               (1, 2), (1, 3), (1, 4), (2, 5), (3, 5), (4, 5),
               (6, 7), (6, 8), (6, 9), (7, 10), (8, 10), (9, 10),
               (5, 11), (10, 11),
               (11, 12), (11, 13), (12, 14), (13, 14), (14, 15)]


# --------------------------------------------------------------------------
# profiles
# --------------------------------------------------------------------------
def linear_profile(rng, n_stages, bmax):
    """d_s(b) = a_s + c_s*b, a_s in [2000, 8000], c_s in [200, 1500] us."""
    tables = []
    for _ in range(n_stages):
        a = int(rng.integers(2000, 8001))
        c = int(rng.integers(200, 1501))
        tables.append(a + c * np.arange(1, bmax + 1, dtype=np.int64))
    return tables


def piecewise_profile(rng, n_stages, bmax=128, n_seg=8):
    """Non-decreasing table built from n_seg linear pieces of bmax/n_seg batch sizes."""
    per = bmax // n_seg
    tables = []
    for _ in range(n_stages):
        a = int(rng.integers(2000, 8001))
        slopes = rng.integers(200, 1501, size=n_seg)
        steps = np.repeat(slopes, per).astype(np.int64)
        tables.append(a + np.cumsum(steps))
    return tables


# --------------------------------------------------------------------------
# runtime state
# --------------------------------------------------------------------------
def draw_state(rng, pipelines, pipeline_of_ctx, now_us, stage_stride=None,
               slot_stride=None) -> QueueState:
    """B_s uniform in [bmax/4, bmax]; the running batch ends uniformly inside one
    stage duration after now (batch wait is uniform on [0, d], Sec. 3.2); q_s
    uniform in [0, d_s(B_s)]; w uniform between 0 and 0.31 times the summed
    duration of all stages (0.31 is the largest fraction of the paper's worked
    example in Sec. 4.2)."""
    n_ctx = len(now_us)
    S = stage_stride or max(p.n_stages for p in pipelines)
    R = slot_stride or max(1, max(n_slots(p) for p in pipelines))
    batch = np.ones((n_ctx, S), dtype=np.int32)
    free_at = np.zeros((n_ctx, S), dtype=np.int64)
    q = np.zeros((n_ctx, S), dtype=np.int64)
    w = np.zeros((n_ctx, R), dtype=np.int64)
    for c in range(n_ctx):
        p = pipelines[int(pipeline_of_ctx[c]) if pipeline_of_ctx is not None else 0]
        dsum = 0
        for k in range(p.n_stages):
            bm = int(p.bmax[k])
            b = int(rng.integers(max(1, bm // 4), bm + 1))
            d = p.latency(k, b)
            batch[c, k] = b
            free_at[c, k] = int(now_us[c]) + int(rng.integers(0, d))
            q[c, k] = int(rng.integers(0, d + 1))
            dsum += d
        w[c, :] = rng.integers(0, int(0.31 * dsum) + 1, size=R)
    poc = None if pipeline_of_ctx is None else np.asarray(pipeline_of_ctx, dtype=np.int32)
    return QueueState(S, R, np.asarray(now_us, dtype=np.int64), batch, free_at, q, w,
                      None, poc)


def draw_wait_samples(rng, wl: "Workload", n_samples: int = 10_000) -> np.ndarray:
    """Recorded batch waits, int32 [n_ctx, stage_stride, n_samples] in microseconds.
    A request that reaches stage i while a batch of duration d_i(B_i) runs waits
    for the rest of it: a fraction of d_i(B_i) (Sec. 3.2).  The fraction is
    Beta(a, b) distributed with a, b drawn per (ctx, stage) from [0.6, 2.5], so
    that stages differ in how early or late in a batch their requests arrive;
    Beta(1, 1) is the uniform arrival of the paper's worked example."""
    st = wl.state
    S = st.stage_stride
    out = np.zeros((wl.n_ctx, S, n_samples), dtype=np.int32)
    for c in range(wl.n_ctx):
        p = wl.pipelines[int(st.pipeline_of_ctx[c]) if st.pipeline_of_ctx is not None else 0]
        for k in range(p.n_stages):
            d = min(p.latency(k, int(st.batch[c, k])), (1 << 24) - 1)
            a, b = rng.uniform(0.6, 2.5, size=2)
            out[c, k] = np.minimum((rng.beta(a, b, size=n_samples) * d).astype(np.int64), d - 1 if d > 1 else 0)
    return out


def balance_workers(wl: Workload, slo_us) -> None:
    """Balanced variant: m_s = ceil(n_s * d_s(B_s) / (B_s * SLO/2)) workers per
    queue, so that a queue drains in about half an SLO and a sizeable share of
    the requests is kept.  slo_us is a scalar or an [n_ctx] array."""
    st = wl.state
    S = st.stage_stride
    seg = wl.requests["ctx"].astype(np.int64) * S + wl.requests["stage"]
    counts = np.bincount(seg, minlength=wl.n_ctx * S).reshape(wl.n_ctx, S)
    slo = np.broadcast_to(np.asarray(slo_us, dtype=np.int64), (wl.n_ctx,))
    workers = np.ones((wl.n_ctx, S), dtype=np.int32)
    for c in range(wl.n_ctx):
        p = wl.pipelines[int(st.pipeline_of_ctx[c]) if st.pipeline_of_ctx is not None else 0]
        for k in range(p.n_stages):
            b = int(st.batch[c, k])
            d = p.latency(k, b)
            num = int(counts[c, k]) * d
            den = b * (int(slo[c]) // 2)
            workers[c, k] = max(1, -(-num // den))
    st.workers = workers
    wl.name += "b"


def _requests(deadline, ctx, stage) -> np.ndarray:
    r = np.zeros(len(deadline), dtype=REQUEST_DTYPE)
    r["deadline_us"] = deadline
    r["ctx"] = ctx
    r["stage"] = stage
    return r


def _zipf_stage(rng, n_stages, n, a=1.2):
    """Stage of each request: weights proportional to rank^-a over a seeded
    permutation of the stages (queue depths follow a Zipf law)."""
    ranks = rng.permutation(n_stages) + 1
    wts = ranks.astype(np.float64) ** (-a)
    wts /= wts.sum()
    return rng.choice(n_stages, size=n, p=wts).astype(np.uint16)


NOW0 = 1_000_000_000   # an arbitrary clock origin, 1000 s


# --------------------------------------------------------------------------
# the five workloads
# --------------------------------------------------------------------------
def c1(n=4096, seed=0, balanced=False) -> Workload:
    """Linear 3-stage pipeline, uniform stages, SLO 150 ms, arrivals uniform
    over the last 200 ms."""
    rng = np.random.default_rng(seed)
    p = make_pipeline(chain_edges(3), 3, [32] * 3, linear_profile(rng, 3, 32))
    now = NOW0
    arrival = now - rng.integers(0, 200_000, size=n)
    stage = rng.integers(0, 3, size=n).astype(np.uint16)
    st = draw_state(rng, [p], None, [now])
    wl = Workload("C1", [p], _requests(arrival + 150_000, 0, stage), st, 1,
                  {"slo_us": 150_000})
    if balanced:
        balance_workers(wl, 150_000)
    return wl


def c2(n=1 << 20, seed=1, balanced=False) -> Workload:
    """8-stage DAG with three paths, Zipf(1.2) queue depths, Poisson arrivals
    at 50k requests/s, SLO 300 ms."""
    rng = np.random.default_rng(seed)
    p = make_pipeline(DAG8_EDGES, 8, [64] * 8, linear_profile(rng, 8, 64))
    arrival = NOW0 + np.floor(np.cumsum(rng.exponential(20.0, size=n))).astype(np.int64)
    now = int(arrival[-1]) if n else NOW0
    stage = _zipf_stage(rng, 8, n)
    st = draw_state(rng, [p], None, [now])
    wl = Workload("C2", [p], _requests(arrival + 300_000, 0, stage), st, 1,
                  {"slo_us": 300_000})
    if balanced:
        balance_workers(wl, 300_000)
    return wl


def c3(n=1 << 24, seed=2, balanced=False) -> Workload:
    """16-stage DAG with 12 paths, piecewise-linear 128-entry profiles,
    per-request SLO drawn from {100, 200, 400} ms."""
    rng = np.random.default_rng(seed)
    p = make_pipeline(DAG16_EDGES, 16, [128] * 16, piecewise_profile(rng, 16))
    assert n_source_sink_paths(p) == 12
    assert max(len(p.successors(k)) for k in range(16)) == 3
    now = NOW0
    arrival = now - rng.integers(0, 400_000, size=n)
    slo = rng.choice(np.array([100_000, 200_000, 400_000], dtype=np.int64), size=n)
    stage = rng.integers(0, 16, size=n).astype(np.uint16)
    st = draw_state(rng, [p], None, [now])
    wl = Workload("C3", [p], _requests(arrival + slo, 0, stage), st, 1,
                  {"slo_us": [100_000, 200_000, 400_000]})
    if balanced:
        # The literal SLOs are shorter than the summed stage durations downstream
        # of most stages, so only the last stages can keep anything; the balanced
        # variant also grants every request 600 ms more.
        wl.requests["deadline_us"] += 600_000
        wl.notes["slo_us"] = [700_000, 800_000, 1_000_000]
        balance_workers(wl, 800_000)
    return wl


def _bursty_arrivals(rng, n, mean_rate=50_000.0, shape=0.3, burst_mult=10.0,
                     period_s=2.0, burst_s=0.05):
    """Gamma(shape) inter-arrivals in operational time, mapped through a
    periodic rate function that is burst_mult times higher during the first
    burst_s of every period; the long-run mean rate is mean_rate."""
    r = mean_rate * period_s / (burst_s * burst_mult + (period_s - burst_s))
    per_period = mean_rate * period_s
    burst_n = burst_s * burst_mult * r
    tau = np.cumsum(rng.gamma(shape, 1.0 / shape, size=n))      # unit-rate arrivals
    j = np.floor(tau / per_period)
    rem = tau - j * per_period
    t = np.where(rem < burst_n, rem / (burst_mult * r), burst_s + (rem - burst_n) / r)
    return NOW0 + np.floor((j * period_s + t) * 1e6).astype(np.int64)


def c4(n_epochs=4096, per_epoch=8192, seed=3, balanced=False) -> Workload:
    """Bursty load on the 8-stage DAG: one arrival stream cut into decision
    epochs (one ctx each); the queue state is carried from epoch to epoch on
    the host, open loop: free_at_s(e) = max(now_e, free_at_s(e-1)) +
    ceil(n_se / B_s) * d_s(B_s), and q_s(e) is the linearly weighted mean of
    the backlog (free_at_s - now) over the epochs of the last 5 s (the paper's
    default sliding window, Sec. 4.2)."""
    rng = np.random.default_rng(seed)
    p = make_pipeline(DAG8_EDGES, 8, [64] * 8, linear_profile(rng, 8, 64))
    n = n_epochs * per_epoch
    arrival = _bursty_arrivals(rng, n)
    stage = _zipf_stage(rng, 8, n)
    ctx = np.repeat(np.arange(n_epochs, dtype=np.uint32), per_epoch)
    now = arrival.reshape(n_epochs, per_epoch)[:, -1].copy() if n else np.zeros(0, np.int64)
    st = draw_state(rng, [p], None, now)
    # carry
    B = st.batch[0].copy() if n_epochs else np.ones(8, np.int32)
    d = np.array([p.latency(k, int(B[k])) for k in range(8)], dtype=np.int64)
    counts = np.zeros((n_epochs, 8), dtype=np.int64)
    if n:
        np.add.at(counts, (ctx, stage), 1)
    free_prev = np.full(8, int(now[0]) if n_epochs else 0, dtype=np.int64)
    hist_t, hist_backlog = [], []
    for e in range(n_epochs):
        st.batch[e] = B
        st.free_at_us[e] = np.maximum(now[e], free_prev)
        backlog = st.free_at_us[e] - now[e]
        hist_t.append(int(now[e]))
        hist_backlog.append(backlog)
        while hist_t and hist_t[0] < now[e] - 5_000_000:
            hist_t.pop(0)
            hist_backlog.pop(0)
        wts = np.arange(1, len(hist_t) + 1, dtype=np.int64)
        st.q_us[e] = (np.stack(hist_backlog) * wts[:, None]).sum(axis=0) // wts.sum()
        free_prev = st.free_at_us[e] + -(-counts[e] // B) * d
    wl = Workload("C4", [p], _requests(arrival + 300_000, ctx, stage), st, n_epochs,
                  {"slo_us": 300_000})
    if balanced:
        balance_workers(wl, 300_000)
    return wl


def random_dag_edges(rng, n_stages, max_paths=8, max_fanout=3):
    """Chain plus random forward edges, then random removal of chain edges whose
    ends stay connected; kept only while 1 <= source-to-sink paths <= max_paths."""
    edges = set(chain_edges(n_stages))

    def ok(es):
        fan = np.zeros(n_stages, dtype=np.int64)
        for a, _ in es:
            fan[a] += 1
        if fan.max(initial=0) > max_fanout:
            return False
        p = make_pipeline(sorted(es), n_stages, [1] * n_stages, [[1]] * n_stages)
        return 1 <= n_source_sink_paths(p) <= max_paths

    for _ in range(int(rng.integers(0, 7))):
        a = int(rng.integers(0, n_stages - 1))
        b = int(rng.integers(a + 1, n_stages))
        trial = edges | {(a, b)}
        if ok(trial):
            edges = trial
    for i in rng.permutation(n_stages - 1):
        i = int(i)
        if rng.random() < 0.5 and (i, i + 1) in edges:
            trial = edges - {(i, i + 1)}
            has_succ = any(a == i for a, _ in trial)
            has_pred = any(b == i + 1 for _, b in trial)
            if has_succ and has_pred and ok(trial):
                edges = trial
    return sorted(edges)


def c5(n_inst=256, per_inst=65536, seed=4, balanced=False) -> Workload:
    """What-if sweep: independent random pipelines (4-16 stages, 1-8 paths),
    each with its own Poisson request queue and SLO."""
    rng = np.random.default_rng(seed)
    pipelines = []
    for _ in range(n_inst):
        S = int(rng.integers(4, 17))
        bm = int(rng.choice([32, 64, 128]))
        pipelines.append(make_pipeline(random_dag_edges(rng, S), S, [bm] * S,
                                       linear_profile(rng, S, bm)))
    n = n_inst * per_inst
    deadline = np.zeros(n, dtype=np.int64)
    stage = np.zeros(n, dtype=np.uint16)
    now = np.zeros(n_inst, dtype=np.int64)
    slo = rng.integers(100_000, 400_001, size=n_inst)
    for c in range(n_inst):
        arr = NOW0 + np.floor(np.cumsum(rng.exponential(20.0, size=per_inst))).astype(np.int64)
        now[c] = arr[-1] if per_inst else NOW0
        sl = slice(c * per_inst, (c + 1) * per_inst)
        deadline[sl] = arr + slo[c]
        stage[sl] = _zipf_stage(rng, pipelines[c].n_stages, per_inst)
    ctx = np.repeat(np.arange(n_inst, dtype=np.uint32), per_inst)
    poc = np.arange(n_inst, dtype=np.int32)
    st = draw_state(rng, pipelines, poc, now, stage_stride=16)
    wl = Workload("C5", pipelines, _requests(deadline, ctx, stage), st, n_inst,
                  {"slo_us": slo})
    if balanced:
        balance_workers(wl, slo)
    return wl


CONFIGS = {"C1": c1, "C2": c2, "C3": c3, "C4": c4, "C5": c5}


def make(name: str, **kw) -> Workload:
    """make("C3") or make("C3b") for the balanced variant."""
    balanced = name.endswith("b")
    return CONFIGS[name[:2]](balanced=balanced, **kw)
