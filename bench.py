#!/usr/bin/env python
"""Benchmark of the PARD drop planner on B200.

One step = one pass of the whole hot path (pard_plan + pard_goodput) over one
snapshot of the 16-stage / 12-path / 2^24-request workload ("C3").  Prints ONE
JSON line.  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2602_08747_b200 import inputs  # noqa: E402

METRIC = "requests_planned_per_sec"
UNIT = "requests/s"
WORKLOAD = "C3"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def ncu_traffic(kernel):
    """DRAM bytes per launch of `kernel` from the committed ncu summary, or None
    when the kernel source has changed since the counters were taken."""
    import hashlib
    try:
        src = os.path.join(ROOT, "paper_2602_08747_b200", "csrc", "pard_plan.cu")
        sha = hashlib.sha256(open(src, "rb").read()).hexdigest()
        vals = {}
        for line in open(os.path.join(ROOT, "profiles", "dram_traffic_C3.txt")):
            if line.startswith("#") or not line.strip():
                continue
            k, v = line.split()
            vals[k] = v
        if vals.get("source_sha256") != sha:
            return None
        return int(vals[kernel]) if kernel in vals else None
    except Exception:
        return None


class ClockSampler(threading.Thread):
    """Polls SM clock and throttle reasons through NVML.  The thread is started ahead of time (NVML's
    start-up takes a while); only the samples taken between begin() and result() count."""

    def __init__(self, index, period_s=0.002):
        super().__init__(daemon=True)
        self.index, self.period, self.stop_flag = index, period_s, threading.Event()
        self.ready, self.active = threading.Event(), threading.Event()
        self.sm, self.reasons, self.max_mhz, self.err = [], set(), None, None

    def run(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
            names = {
                getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
                getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
                getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
                getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            }
            get = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                nv.nvmlDeviceGetCurrentClocksThrottleReasons
            self.ready.set()
            while not self.stop_flag.is_set():
                if self.active.is_set():
                    self.sm.append(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                    bits = get(h)
                    for bit, name in names.items():
                        if bits & bit:
                            self.reasons.add(name)
                time.sleep(self.period)
        except Exception as e:  # NVML missing: report it, do not fail the bench
            self.err = repr(e)
            self.ready.set()

    def begin(self):
        self.ready.wait(timeout=20)
        self.active.set()

    def result(self):
        self.active.clear()
        self.stop_flag.set()
        self.join(timeout=2)
        out = {"sm_mhz": statistics.median(self.sm) if self.sm else None,
               "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.sm)}
        if self.err:
            out["error"] = self.err
        return out


def physical_gpu_index(local):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


# --------------------------------------------------------------------------
def time_oracle(wl, repeats):
    from oracle import oracle
    best = None
    for _ in range(repeats):
        t = time.perf_counter()
        o = oracle.plan(wl.pipelines, wl.requests, wl.state, wl.n_ctx)
        dt = time.perf_counter() - t
        best = dt if best is None else min(best, dt)
    return best, o


def _oracle_shard(job):
    """Worker of the all-cores CPU baseline: draws the (reduced) workload, keeps
    this worker's share of its contexts and times the oracle on it."""
    name, kw, world, rank = job
    from oracle import oracle
    from paper_2602_08747_b200 import sharding
    wl = sharding.shard_workload(inputs.make(name, **kw), world, rank)
    t = time.perf_counter()
    oracle.plan(wl.pipelines, wl.requests, wl.state, wl.n_ctx)
    return wl.n, time.perf_counter() - t


def oracle_all_cores(name, kw):
    """The oracle, unchanged, over the contexts of a many-context workload on all
    host cores: one share of the contexts per process, no exchange (contexts are
    independent).  Processes are spawned, never forked: the parent holds a CUDA
    context.  Returns requests per second by the slowest worker's clock."""
    import multiprocessing as mp
    cores = max(1, min(os.cpu_count() or 1, 32))
    with mp.get_context("spawn").Pool(cores) as pool:
        res = pool.map(_oracle_shard, [(name, kw, cores, r) for r in range(cores)])
    n = sum(r[0] for r in res)
    return {"value": n / max(r[1] for r in res), "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "%s drawn with %s: %d requests, contexts split over %d processes" % (name, kw, n, cores)}


def run_reference(args):
    """The oracle, as it stands, on the host cores; each step plans a bounded
    sample (a smaller draw of the same workload)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    # the full 2^24-request snapshot costs about 3 s per step on one core: the whole snapshot while
    # steps + warm-up stay within about two and a half minutes, else the largest power-of-two
    # sample of it that does
    n = 1 << 24
    while n > (1 << 16) and (args.steps + args.warmup) * (n / 5.5e6) > 150.0:
        n >>= 1
    wl = inputs.make(WORKLOAD, n=n)
    from oracle import oracle
    for _ in range(args.warmup):
        oracle.plan(wl.pipelines, wl.requests, wl.state, wl.n_ctx)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.plan(wl.pipelines, wl.requests, wl.state, wl.n_ctx)
    dt = time.perf_counter() - t0
    value = wl.n * args.steps / dt
    sample = ("the full %s snapshot (%d requests) per step" % (WORKLOAD, n) if n == 1 << 24 else
              "%s workload drawn at n=%d requests per step" % (WORKLOAD, n))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "requests_per_step": n, "stages": 16, "paths": 12,
                   "contexts": wl.n_ctx,
                   "note": "CPU oracle (single thread)" + ("" if n == 1 << 24 else " on a bounded sample")},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample,
                         "host_cores": os.cpu_count()},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------
class DevicePlan:
    """Device-resident workload, outputs and workspace for repeated planning."""

    def __init__(self, wl, dev, mode=0, arrivals=None):
        import torch
        self.mode = mode
        self.d_arr = None
        from paper_2602_08747_b200 import binding as pb
        self.pb, self.torch, self.wl, self.dev = pb, torch, wl, dev
        self.S = wl.state.stage_stride
        self.n_seg = wl.n_ctx * self.S
        self.pipes = [pb.pard_load_pipeline(p) for p in wl.pipelines]
        self.d_req = pb.device_requests(wl.requests, dev)
        if arrivals is not None:
            self.d_arr = pb.device_requests(arrivals, dev)       # 16-byte records as well
        self.d_state = pb.device_state(wl.state, dev)
        self.out = pb.alloc_out(wl.n, self.n_seg, dev)
        self.ws = pb.alloc_workspace(pb.pard_plan_workspace_bytes(wl.n, wl.n_ctx, self.S), dev)
        self.total = torch.empty(wl.n_ctx, dtype=torch.int64, device=dev)
        self.kept = torch.empty(wl.n_ctx, dtype=torch.int64, device=dev)
        self.stream = torch.cuda.current_stream().cuda_stream
        self.launches = pb.pard_plan_kernel_launches(wl.n, wl.n_ctx, self.S) + 1   # + the goodput kernel

    def step(self, nowait=True):
        pb, wl = self.pb, self.wl
        rules = pb.PARD_MODE_PATH_MASK | pb.PARD_MODE_FCFS | pb.PARD_MODE_NEXUS | pb.PARD_MODE_CLIPPER
        if self.mode & rules:
            pb.pard_plan_policy(self.pipes, self.d_req, self.d_arr, wl.n, self.d_state, wl.n_ctx,
                                self.mode | (pb.PARD_MODE_NOWAIT if nowait else 0), self.out, self.ws, stream=self.stream)
        else:
            pb.pard_plan(self.pipes, self.d_req, wl.n, self.d_state, wl.n_ctx,
                         self.mode | (pb.PARD_MODE_NOWAIT if nowait else 0), self.out, self.ws, stream=self.stream)
        pb.pard_goodput(None, self.out.seg_offsets, self.out.seg_kept, wl.n, wl.n_ctx, self.S, self.total,
                        self.kept, stream=self.stream)

    def status(self):
        return self.pb.pard_plan_status(self.ws, self.stream)


def timed_steps(plan, steps, warmup, dist, profile_every=None):
    """K steps between two CUDA events on the launching stream; returns seconds
    (max over ranks) and the phase profile."""
    torch, pb = plan.torch, plan.pb
    for _ in range(warmup):
        plan.step()
    plan.status()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    if profile_every:
        pb.pard_profile_begin(profile_every, max(1, steps // (profile_every & 0xffff) + 1))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        plan.step()
    e1.record()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    plan.status()
    prof = pb.pard_profile_end() if profile_every else None
    sec = e0.elapsed_time(e1) / 1e3
    if dist is not None:
        t = torch.tensor([sec], dtype=torch.float64, device=plan.dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        sec = float(t.item())
    return sec, prof


def kernel_table(prof, n, keep_frac, peak, prof_coarse=None):
    """Per-kernel average duration and achieved algorithmic GB/s from the phase
    events the library records on its own stream.  "k_decide_win" is the decision
    kernel (threshold, estimate, keep, survivor lists; the phase also holds the
    three fallback launches that return at once); "decision_pass" is everything
    after the sort: k_seg_win, k_win_bounds, k_win_prefix, the decision, k_kept_scan
    and k_kept_move, timed as one phase (no events between its kernels) in a
    second, shorter run when prof_coarse is given."""
    k = prof["n_samples"]
    ms = prof["ms"]
    sort_names = [s for s in ms if s.startswith("sort")]
    sort_active = [s for s in sort_names if ms[s] / k > 0.03]       # passes that really ran
    rows = {}

    def add(name, total_ms, launches, bytes_per_req):
        if launches == 0:
            return
        per = total_ms / k / launches
        gbs = bytes_per_req * n / (per * 1e-3) / 1e9 if per > 0 else None
        rows[name] = {"launches_per_step": launches, "ms_per_launch": per,
                      "algorithmic_bytes_per_request": bytes_per_req, "achieved_gbs": gbs,
                      "frac": gbs / peak if gbs else None, "ms_per_step": total_ms / k}
    add("k_prepass", ms["prepass"], 1, 16.0)
    add("k_pack", ms["pack"], 1, 24.0)
    add("k_sort_pass", sum(ms[s] for s in sort_active), len(sort_active), 16.0)
    dec_bytes = 21.0 + 4.0 * keep_frac
    add("k_decide_win", ms["decide"], 1, dec_bytes)
    if prof_coarse:
        rows_k, k = k, prof_coarse["n_samples"]
        add("decision_pass", prof_coarse["ms"]["tables"], 1, dec_bytes)
        k = rows_k
    else:
        add("decision_pass", ms["tables"] + ms["decide"] + ms["compact"], 1, dec_bytes)
    other = ms["clear"] + ms["segments"] + sum(ms[s] for s in sort_names if s not in sort_active)
    rows["other"] = {"ms_per_step": other / k}
    return rows


def pass_scalars(rows, suffix=""):
    """The pass over the sorted queues (thresholds, positions, estimates, drop rule, compaction,
    goodput counters; window tables included) as three plain numbers."""
    r = rows["decision_pass"]
    return {"pass_ms" + suffix: r["ms_per_launch"], "pass_bytes_per_request" + suffix: r["algorithmic_bytes_per_request"],
            "pass_frac" + suffix: r["frac"]}


def run_e2e(wl, dev, steps, dist, lanes=1):
    """The same metric through pard_plan_host: pinned host inputs and outputs,
    copies inside the timed region.  lanes = 1: one blocking call after the
    other.  lanes = 2: two host threads, each with its own stream, host buffers
    and workspace, so that one call's copies to the host overlap the other's
    copies to the device (every call still moves all of its inputs and outputs);
    the span runs from the earlier start event to the later end event."""
    import torch
    from paper_2602_08747_b200 import binding as pb
    st = wl.state
    S, R = st.stage_stride, st.slot_stride
    n, n_seg = wl.n, wl.n_ctx * S
    pipes = [pb.pard_load_pipeline(p) for p in wl.pipelines]

    def pin(a, dt):
        if a is None:
            return None
        t = torch.from_numpy(np.ascontiguousarray(a, dtype=dt)).pin_memory()
        return t

    def pinned(shape, dt):
        return torch.empty(shape, dtype=dt).pin_memory()

    class Lane:
        def __init__(self):
            self.req = torch.from_numpy(np.ascontiguousarray(wl.requests).view(np.uint8).reshape(-1, 16)).pin_memory()
            self.hs = pb.QueueStateArrays(S, R, pin(st.now_us, np.int64), pin(st.batch, np.int32),
                                          pin(st.free_at_us, np.int64), pin(st.q_us, np.int64),
                                          pin(st.w_us, np.int64), pin(st.workers, np.int32),
                                          pin(st.pipeline_of_ctx, np.int32))
            self.out = pb.PlanOut(pinned(n, torch.uint8), pinned(n, torch.int64), pinned(n, torch.int32),
                                  pinned(n, torch.int32), pinned(1, torch.int64), pinned(n_seg + 1, torch.int32),
                                  pinned(n_seg, torch.int32))
            self.ws = pb.alloc_workspace(pb.pard_plan_host_workspace_bytes(n, wl.n_ctx, S, R), dev)
            self.stream = torch.cuda.Stream(device=dev) if lanes > 1 else torch.cuda.current_stream()
            self.e0 = torch.cuda.Event(enable_timing=True)
            self.e1 = torch.cuda.Event(enable_timing=True)

        def step(self):
            pb.pard_plan_host(pipes, self.req, n, self.hs, wl.n_ctx, 0, self.out, self.ws,
                              stream=self.stream.cuda_stream)

        def run(self, k):
            torch.cuda.set_device(dev)
            self.e0.record(self.stream)
            for _ in range(k):
                self.step()
            self.e1.record(self.stream)

    ls = [Lane() for _ in range(lanes)]
    for ln in ls:
        for _ in range(3):
            ln.step()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    per = [steps // lanes + (1 if i < steps % lanes else 0) for i in range(lanes)]
    if lanes == 1:
        ls[0].run(per[0])
    else:
        ts = [threading.Thread(target=ls[i].run, args=(per[i],)) for i in range(lanes)]
        for t in ts:
            t.start()
        for t in ts:
            t.join()
    torch.cuda.synchronize()
    sec = max(a.e0.elapsed_time(b.e1) for a in ls for b in ls) / 1e3
    if dist is not None:
        t = torch.tensor([sec], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        sec = float(t.item())
    nk = int(ls[0].out.n_kept[0])
    hs = ls[0].hs
    state_bytes = sum(t.numel() * t.element_size() for t in
                      (hs.now_us, hs.batch, hs.free_at_us, hs.q_us, hs.w_us, hs.workers,
                       hs.pipeline_of_ctx) if t is not None)
    h2d = 16 * n + state_bytes
    d2h = n + 8 * n + 4 * n + 4 * nk + 8 + 4 * (n_seg + 1) + 4 * n_seg
    for p in pipes:
        p.free()
    return sec, h2d, d2h



def run_aux(dev, peak, kernels_only=False):
    """Device time of the State Planner's input kernels and of the planner with
    mixed priorities, on seeded synthetic inputs larger than the L2 where a
    bandwidth figure is given.  CUDA events, 3 warm-ups, 10 timed calls."""
    import torch
    from paper_2602_08747_b200 import binding as pb
    from paper_2602_08747_b200 import replay as rp
    stream = torch.cuda.current_stream().cuda_stream
    out = {}

    def timed(fn, reps=10):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / 1e3 / reps

    g = torch.Generator(device=dev)
    g.manual_seed(7)
    # the 256 random DAG instances of the what-if sweep carry the per-queue state
    wl = inputs.make("C5b", n_inst=256, per_inst=256)
    st = wl.state
    S, R, n_ctx = st.stage_stride, st.slot_stride, wl.n_ctx
    pipes = [pb.pard_load_pipeline(p) for p in wl.pipelines]
    ds = pb.device_state(st, dev)
    n_slots = int(sum(inputs.n_slots(wl.pipelines[int(c)]) for c in st.pipeline_of_ctx))
    path_stages = int(sum(sum(len(pth) for pth in _paths(wl.pipelines[int(c)])) for c in st.pipeline_of_ctx))

    # batch-wait estimate: M = 10,000 samples per (stage, downstream path) slot (Sec. 4.2)
    M = 10_000
    samples = torch.randint(0, 8000, (n_ctx, S, M), dtype=torch.int32, device=dev, generator=g)
    d_w = torch.zeros((n_ctx, R), dtype=torch.int64, device=dev)
    ws = pb.alloc_workspace(pb.pard_estimate_w_workspace_bytes(len(pipes)), dev)
    sec = timed(lambda: pb.pard_estimate_w(pipes, ds.pipeline_of_ctx, n_ctx, S, R, samples, M, 1, 10, 5,
                                           pb.PARD_MODE_NOWAIT, d_w, ws, stream=stream))
    assert pb.pard_plan_status(ws, stream) == 0
    out["pard_estimate_w"] = {"workload": "256 random DAG instances, M=10000, lambda=0.1", "slots": n_slots,
                              "ms": 1e3 * sec, "slots_per_s": n_slots / sec, "draws_per_s": path_stages * M / sec,
                              "algorithmic_gbs": 4.0 * path_stages * M / sec / 1e9, "bound": "alu/shared memory"}
    del samples

    # priority update: 2,048 workload samples per queue
    H, W = 2048, 5
    x = torch.randint(0, 4000, (n_ctx * 16, S, H), dtype=torch.int32, device=dev, generator=g)
    big_ctx = n_ctx * 16
    poc = ds.pipeline_of_ctx.repeat(16)
    batch, workers = ds.batch.repeat(16, 1), ds.workers.repeat(16, 1)
    prio = torch.zeros((big_ctx, S), dtype=torch.uint8, device=dev)
    ws = pb.alloc_workspace(pb.pard_update_priority_workspace_bytes(len(pipes)), dev)
    sec = timed(lambda: pb.pard_update_priority(pipes, poc, big_ctx, S, batch, workers, x, H, W, 1_000_000,
                                                pb.PARD_MODE_NOWAIT, prio, ws, stream=stream))
    assert pb.pard_plan_status(ws, stream) == 0
    queues = int(sum(wl.pipelines[int(c)].n_stages for c in st.pipeline_of_ctx)) * 16
    gbs = 4.0 * H * queues / sec / 1e9
    out["pard_update_priority"] = {"workload": "%d queues x %d samples, window %d" % (queues, H, W), "ms": 1e3 * sec,
                                   "queues_per_s": queues / sec, "algorithmic_gbs": gbs, "frac": gbs / peak,
                                   "bound": "hbm"}
    del x

    # queueing-delay window: 2,048 samples per queue
    Mq = 2048
    now = torch.full((big_ctx,), 10**9, dtype=torch.int64, device=dev)
    t = now[:, None, None] - torch.randint(0, 8_000_000, (big_ctx, S, Mq), dtype=torch.int64, device=dev, generator=g)
    dly = torch.randint(0, 1 << 20, (big_ctx, S, Mq), dtype=torch.int32, device=dev, generator=g)
    q = torch.zeros((big_ctx, S), dtype=torch.int64, device=dev)
    ws = pb.alloc_workspace(pb.pard_update_queue_delay_workspace_bytes(), dev)
    sec = timed(lambda: pb.pard_update_queue_delay(big_ctx, S, now, t, dly, Mq, 5_000_000, pb.PARD_MODE_NOWAIT, q, ws,
                                                   stream=stream))
    assert pb.pard_plan_status(ws, stream) == 0
    rows = big_ctx * S
    gbs = 12.0 * Mq * rows / sec / 1e9
    out["pard_update_queue_delay"] = {"workload": "%d rows x %d samples, window 5 s" % (rows, Mq), "ms": 1e3 * sec,
                                      "rows_per_s": rows / sec, "algorithmic_gbs": gbs, "frac": gbs / peak,
                                      "bound": "hbm"}
    del t, dly
    for p in pipes:
        p.free()
    if kernels_only:
        return out

    # the planner with every second queue served high budget first
    wlh = inputs.make(WORKLOAD + "b", seed=2)
    rng = np.random.default_rng(3)
    wlh.state.priority = rng.integers(0, 2, size=(wlh.n_ctx, wlh.state.stage_stride)).astype(np.uint8)
    plan = DevicePlan(wlh, dev)
    sec, _ = timed_steps(plan, 40, 5, None)
    out["pard_plan_mixed_priority"] = {"workload": WORKLOAD + "b, priorities drawn per queue", "ms": 1e3 * sec / 40,
                                       "requests_per_s": wlh.n * 40 / sec}
    del plan

    # the comparison rules and order variants on the balanced 2^24-request workload
    rules = {}
    wlr = inputs.make(WORKLOAD + "b", seed=2)
    rr = np.random.default_rng(4)
    arr = np.zeros(wlr.n, dtype=inputs.ARRIVAL_DTYPE)
    arr["arrive_us"] = np.maximum(0, wlr.state.now_us[0] - rr.integers(0, 400_000, size=wlr.n))
    arr["slo_us"] = rr.integers(100_000, 400_000, size=wlr.n)
    masked = wlr.requests.copy()
    masked["flags"] = rr.choice(np.array([0, 1, 3], dtype=np.uint16), size=wlr.n)   # path unknown, the first, one of the first two
    for label, mode, a, req in (("known_paths", pb.PARD_MODE_PATH_MASK, None, masked), ("arrival_order", pb.PARD_MODE_FCFS, None, None),
                                ("nexus", pb.PARD_MODE_NEXUS, None, None), ("clipper_pp", pb.PARD_MODE_CLIPPER, arr, None)):
        w2 = wlr if req is None else inputs.Workload(wlr.name, wlr.pipelines, req, wlr.state, wlr.n_ctx)
        plan = DevicePlan(w2, dev, mode, a)
        plan.step(nowait=False)
        kf = float(plan.out.n_kept.cpu()[0]) / w2.n
        sec, _ = timed_steps(plan, 10, 3, None)
        rules[label] = {"ms": 1e3 * sec / 10, "requests_per_s": w2.n * 10 / sec, "keep_fraction": kf}
        del plan
    out["comparison_rules"] = {"workload": WORKLOAD + "b (16 queues of about 2^20 requests: one warp walks each queue)", **rules}

    # closed-loop replay: 16 instances, 64 epochs of 65,536 requests
    job_rng = np.random.default_rng(11)
    inst, n_ep, per = 16, 64, 65536
    wl5 = inputs.make("C5b", n_inst=inst, per_inst=per)
    st5 = wl5.state
    pipes = [pb.pard_load_pipeline(p) for p in wl5.pipelines]
    epochs = []
    for e in range(n_ep):
        r = wl5.requests.copy()
        r["deadline_us"] += e * 600_000 + job_rng.integers(0, 2000, size=r.shape[0])
        epochs.append((st5.now_us + e * 600_000, r))
    R5 = rp.Replay(pipes, st5.pipeline_of_ctx, inst, st5.stage_stride, st5.slot_stride, st5.batch, st5.workers,
                   st5.free_at_us, st5.w_us, None, 64, 5_000_000, wl5.n, dev)
    d_now = torch.from_numpy(np.stack([e[0] for e in epochs])).to(dev)
    d_req = [pb.device_requests(e[1], dev) for e in epochs]
    total = torch.zeros((n_ep, inst), dtype=torch.int64, device=dev)
    kept = torch.zeros((n_ep, inst), dtype=torch.int64, device=dev)

    fa0 = R5.state.free_at_us.clone()

    def one_replay():
        R5.state.free_at_us.copy_(fa0)                    # every run starts from the same state
        R5.sample_time.fill_(-1)
        R5.epoch = 0
        for i in range(n_ep):
            R5.step(d_now[i], d_req[i], wl5.n, total[i], kept[i])

    sec = timed(one_replay, reps=3)
    assert R5.statuses() == 0
    out["replay"] = {"workload": "%d instances, %d epochs x %d requests" % (inst, n_ep, wl5.n), "ms_per_epoch": 1e3 * sec / n_ep,
                     "epochs_per_s": n_ep / sec, "requests_per_s": wl5.n * n_ep / sec,
                     "epoch_spacing_us": 600_000,
                     "kept_fraction_last_run": float(kept.sum().item()) / float(max(1, total.sum().item()))}
    for p in pipes:
        p.free()
    return out


def _paths(p):
    """Downstream paths of every stage of a pipeline (input structure only), for counting."""
    out = []

    def rec(k, prefix):
        prefix = prefix + (int(k),)
        succ = [int(j) for j in p.successors(k)]
        if not succ:
            out.append(prefix)
        for j in succ:
            rec(j, prefix)

    for k in range(p.n_stages):
        for j in p.successors(k):
            rec(j, ())
    return out


def run_sharded(dev, dist, world, rank):
    """One job split over the ranks (fixed total work): the many-context workloads by ctx, the
    single-ctx workload by stage.  No exchange on the data path; the per-ctx goodput counters are
    gathered (by ctx) or summed (by stage) over NCCL after the timed region.  Time = max over ranks."""
    import torch
    from paper_2602_08747_b200 import sharding
    out = {}
    for name, how in (("C4", "ctx"), ("C5", "ctx"), (WORKLOAD, "stage")):
        wl = inputs.make(name)
        mine = sharding.shard_workload(wl, world, rank) if how == "ctx" else sharding.shard_by_stage(wl, world, rank)
        from paper_2602_08747_b200 import binding as pb
        plan = DevicePlan(mine, dev, pb.PARD_MODE_GROUPED if name in ("C4", "C5") else 0)
        plan.step(nowait=False)
        steps = 20
        sec, _ = timed_steps(plan, steps, 5, dist)
        if how == "ctx":
            tot, kept = sharding.gather_counters(plan.total, plan.kept, wl.n_ctx)
        else:
            tot, kept = sharding.sum_counters(plan.total, plan.kept)
        torch.cuda.synchronize()
        out[name] = {"split": "by " + how, "ranks": world, "requests": wl.n, "requests_this_rank": mine.n,
                     "us_per_step": 1e6 * sec / steps, "requests_per_s": wl.n * steps / sec, "scaling": "strong",
                     "counted_requests": int(tot.sum().item()), "kept_requests": int(kept.sum().item())}
        del plan, mine, wl
    return out


def _free_port():
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_entry(local_rank, world, port, target, args):
    os.environ.update({"MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port), "WORLD_SIZE": str(world),
                       "RANK": str(local_rank), "LOCAL_RANK": str(local_rank)})
    target(*args)


def spawn_ranks(world, target, args=()):
    """One process per GPU of this node, with the rendezvous environment a launcher would set
    (`python bench.py --gpus N` without torchrun)."""
    import torch.multiprocessing as mp
    mp.spawn(_rank_entry, args=(world, _free_port(), target, args), nprocs=world, join=True)


def run_ours(args):
    import torch
    from paper_2602_08747_b200 import build as pbuild
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world != args.gpus:
        raise SystemExit("bench.py: --gpus %d but WORLD_SIZE=%d: launch one rank per GPU" % (args.gpus, world))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the planner has no CPU path")
    if torch.cuda.device_count() <= local:
        raise SystemExit("bench.py: rank %d has no GPU (%d visible)" % (local, torch.cuda.device_count()))
    pbuild.build()
    torch.cuda.set_device(local)
    dev = "cuda:%d" % local
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=torch.device(dev))
        dist = dist_mod

    if args.only_aux:
        peak, _ = measured_peaks()
        print(json.dumps({"only_aux": True, "state_planner_kernels": run_aux(dev, peak, kernels_only=True)}))
        return
    if args.only_device:
        kw = {"n": args.n} if args.n else {}
        wl = inputs.make(args.workload or WORKLOAD, **kw)
        plan = DevicePlan(wl, dev)
        sec, _ = timed_steps(plan, args.steps, args.warmup, None)
        print(json.dumps({"only_device": True, "workload": wl.name, "n": wl.n,
                          "ms_per_step": 1e3 * sec / args.steps}))
        return

    # every rank plans its own, independently drawn snapshot (contexts are
    # independent planning problems: no data-path collective)
    wl = inputs.make(WORKLOAD, seed=2 + rank)
    plan = DevicePlan(wl, dev)
    plan.step(nowait=False)
    keep_frac = float(plan.out.n_kept.cpu()[0]) / wl.n

    sampler = ClockSampler(physical_gpu_index(local))
    sampler.start()
    # warm-up first so that the sampler only sees work under load
    for _ in range(args.warmup):
        plan.step()
    plan.status()
    sampler.begin()
    sec, _ = timed_steps(plan, args.steps, 0, dist)         # the timed region: K steps, nothing else on the stream
    # per-kernel durations from the library's own phase events, in a second run of the same steps
    # (an event between two kernels keeps the second from being scheduled while the first drains,
    # so a run with events is a little slower than the timed one)
    _, prof = timed_steps(plan, max(args.steps, 16), 0, dist, profile_every=4)
    # the decision pass as one phase, in a run of its own (same work, same load: the clock samples
    # run on through it, the timed region alone may last only a few milliseconds)
    from paper_2602_08747_b200 import binding as pb
    _, prof_coarse = timed_steps(plan, max(40, args.steps // 4), 0, dist,
                                 profile_every=4 | pb.PARD_PROFILE_COARSE)
    clocks = sampler.result()

    peak, peak_kind = measured_peaks()
    n_total = wl.n * world
    value = n_total * args.steps / sec
    e2e_steps = max(3, min(args.steps, 20))
    e2e_sec, h2d, d2h = run_e2e(wl, dev, e2e_steps, dist)
    e2e2_sec, _, _ = run_e2e(wl, dev, e2e_steps, dist, lanes=2)

    if rank == 0:
        kernels = kernel_table(prof, wl.n, keep_frac, peak, prof_coarse)
        timed = {k: v for k, v in kernels.items() if k not in ("other", "k_decide_win")}
        top = max(timed, key=lambda k: timed[k]["ms_per_step"])
        traffic = ncu_traffic(top)
        roofline = {"bound": "hbm", "kernel": top, "achieved": timed[top]["achieved_gbs"], "peak": peak,
                    "unit": "GB/s", "frac": timed[top]["frac"], "traffic": traffic,
                    "peak_kind": "of " + peak_kind,
                    "algorithmic_bytes_per_launch": timed[top]["algorithmic_bytes_per_request"] * wl.n,
                    "pass_note": "pass = everything after the sort, goodput counters included, timed as one "
                                 "phase; bytes = 21 + 4 * keep fraction per request",
                    "kernels": kernels}
        roofline.update(pass_scalars(kernels))
        # the balanced variant (about half of the requests kept) as a second data point
        variants = {}
        if not args.no_variants:
            wlb = inputs.make(WORKLOAD + "b", seed=2)
            pl2 = DevicePlan(wlb, dev)
            pl2.step(nowait=False)
            kf = float(pl2.out.n_kept.cpu()[0]) / wlb.n
            s2, prof2 = timed_steps(pl2, max(10, args.steps // 4), 5, None, profile_every=4)
            _, prof2c = timed_steps(pl2, 40, 0, None, profile_every=4 | pb.PARD_PROFILE_COARSE)
            kernels_b = kernel_table(prof2, wlb.n, kf, peak, prof2c)
            variants[WORKLOAD + "b"] = {"value": wlb.n * max(10, args.steps // 4) / s2, "unit": UNIT,
                                        "keep_fraction": kf, "kernels": kernels_b}
            roofline.update(pass_scalars(kernels_b, "_c3b"))
            roofline["keep_fraction_c3b"] = kf
            del pl2
        aux = {} if args.no_variants else run_aux(dev, peak)
        others = {}
        if not args.no_variants:
            # the other configurations of the workload list, device-resident, for the record
            for name in ("C1", "C2", "C4", "C5"):
                wlo = inputs.make(name)
                # C4's epochs and C5's instances arrive as one array grouped by epoch / instance (= ctx): the caller says so
                plo = DevicePlan(wlo, dev, pb.PARD_MODE_GROUPED if name in ("C4", "C5") else 0)
                plo.step(nowait=False)
                kfo = float(plo.out.n_kept.cpu()[0]) / wlo.n
                so, _ = timed_steps(plo, 50, 5, None)
                others[name] = {"requests": wlo.n, "contexts": wlo.n_ctx, "us_per_step": 1e6 * so / 50,
                                "requests_per_s": wlo.n * 50 / so, "keep_fraction": kfo,
                                "mode": "PARD_MODE_GROUPED" if name in ("C4", "C5") else "default"}
                del plo
                if name in ("C4", "C5"):                  # and without the caller's word, for comparison
                    plo = DevicePlan(wlo, dev, 0)
                    so, _ = timed_steps(plo, 50, 5, None)
                    others[name]["us_per_step_without_the_promise"] = 1e6 * so / 50
                    del plo
                del wlo
            # the many-context workloads also against the oracle on all host cores (bounded samples)
            others["C4"]["cpu_baseline_all_cores"] = oracle_all_cores("C4", {"n_epochs": 512, "per_epoch": 8192})
            others["C5"]["cpu_baseline_all_cores"] = oracle_all_cores("C5", {"n_inst": 64, "per_inst": 65536})
        t_cpu, _ = time_oracle(wl, 2)
    sharded = run_sharded(dev, dist, world, rank) if (world > 1 and not args.no_variants) else {}
    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * sec / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "requests_per_gpu": wl.n, "stages": 16, "paths": 12,
                       "contexts": wl.n_ctx, "keep_fraction": keep_frac,
                       "l2": "inputs (256 MiB) and sort buffers (2 x 128 MiB) exceed the 126 MB L2",
                       "parallelism": "independent snapshot per GPU, no collective"},
            "clocks": clocks,
            "e2e": {"value": n_total * e2e_steps / e2e_sec, "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                    "ms_per_step": 1e3 * e2e_sec / e2e_steps,
                    "host_link_gbs": (h2d + d2h) * e2e_steps / e2e_sec / 1e9,
                    "host_link_gbs_outside_device_time": (h2d + d2h) / max(1e-9, e2e_sec / e2e_steps - sec / args.steps) / 1e9,
                    "note": "one blocking pard_plan_host call after the other on one stream"},
            "e2e_two_streams": {"value": n_total * e2e_steps / e2e2_sec, "unit": UNIT, "steps": e2e_steps,
                                "ms_per_step": 1e3 * e2e2_sec / e2e_steps,
                                "note": "the same calls issued by two host threads on two streams, so that "
                                        "copies to the host and to the device overlap"},
            "gpu_launches": plan.launches * args.steps,
            "gpu_launches_per_step": plan.launches,
            "roofline": roofline,
            "cpu_baseline": {"value": wl.n / t_cpu, "unit": UNIT, "cores": 1, "kind": "oracle",
                             "sample": "the full %s snapshot (%d requests), best of 2 runs" % (WORKLOAD, wl.n),
                             "host_cores": os.cpu_count()},
            "variants": variants,
            "state_planner_kernels": aux,
            "other_workloads": others,
            "sharded_jobs": sharded,
        }
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-variants", action="store_true")
    ap.add_argument("--only-device", action="store_true",
                    help="run warm-up and timed steps of the device path only and print a short line "
                         "(for use under a profiler; not a bench value)")
    ap.add_argument("--only-aux", action="store_true",
                    help="run only the State Planner kernels' timings and print them "
                         "(for use under a profiler; not a bench value)")
    ap.add_argument("--workload", default=None, help="with --only-device: another workload name, e.g. C3b")
    ap.add_argument("--n", type=int, default=None, help="with --only-device: number of requests")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        spawn_ranks(args.gpus, run_ours, (args,))          # no launcher around us: start the ranks here
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
