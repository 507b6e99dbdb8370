"""ctypes loader for the CPU oracle (test infrastructure only).

Nothing in the product path imports this module; it is used by the tests, the
smoke check and the benchmark's CPU-baseline leg.  Inputs are duck-typed: any
object with the attributes used below (numpy arrays) is accepted, so that this
module imports nothing but numpy.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libpard_oracle.so")
_SRC = [os.path.join(_HERE, "pard_oracle.cpp"), os.path.join(_HERE, "pard_oracle.h")]
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ -O2 if the shared object is missing or stale."""
    stale = (not os.path.exists(_SO)
             or any(os.path.getmtime(s) > os.path.getmtime(_SO) for s in _SRC))
    if force or stale:
        tmp = _SO + ".tmp%d" % os.getpid()
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-shared", "-fPIC",
                               "-o", tmp, _SRC[0]])
        os.replace(tmp, _SO)
    return _SO


class _Pipeline(C.Structure):
    _fields_ = [("n_stages", C.c_int32), ("sub_offsets", C.c_void_p),
                ("sub_ids", C.c_void_p), ("bmax", C.c_void_p),
                ("lat_offsets", C.c_void_p), ("lat_us", C.c_void_p)]


class _State(C.Structure):
    _fields_ = [("stage_stride", C.c_int32), ("slot_stride", C.c_int32),
                ("pipeline_of_ctx", C.c_void_p), ("now_us", C.c_void_p),
                ("batch", C.c_void_p), ("free_at_us", C.c_void_p),
                ("q_us", C.c_void_p), ("w_us", C.c_void_p), ("workers", C.c_void_p),
                ("priority", C.c_void_p)]


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_count_paths.restype = C.c_int64
        _lib.oracle_count_paths.argtypes = [C.c_void_p, C.c_int32]
        _lib.oracle_slot_base.restype = C.c_int64
        _lib.oracle_slot_base.argtypes = [C.c_void_p, C.c_int32]
        _lib.oracle_lsub.restype = C.c_int64
        _lib.oracle_lsub.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
        _lib.oracle_lsub_masked.restype = C.c_int64
        _lib.oracle_lsub_masked.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint16]
        _lib.oracle_plan.restype = C.c_int
        _lib.oracle_plan.argtypes = ([C.c_void_p, C.c_int32, C.c_void_p, C.c_uint64,
                                      C.c_void_p, C.c_uint32, C.c_uint32] + [C.c_void_p] * 9)
        _lib.oracle_plan_policy.restype = C.c_int
        _lib.oracle_plan_policy.argtypes = ([C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_uint64,
                                             C.c_void_p, C.c_uint32, C.c_uint32] + [C.c_void_p] * 9)
        _lib.oracle_estimate_w.restype = C.c_int
        _lib.oracle_estimate_w.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_uint32, C.c_int32, C.c_int32,
                                           C.c_void_p, C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint64, C.c_void_p]
        _lib.oracle_update_priority.restype = C.c_int
        _lib.oracle_update_priority.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_uint32, C.c_int32,
                                                C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint32, C.c_uint32,
                                                C.c_uint32, C.c_void_p]
        _lib.oracle_queue_delay.restype = C.c_int
        _lib.oracle_queue_delay.argtypes = [C.c_uint32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                            C.c_uint32, C.c_uint32, C.c_void_p]
        _lib.oracle_advance_state.restype = C.c_int
        _lib.oracle_advance_state.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_uint32, C.c_int32] + \
            [C.c_void_p] * 7 + [C.c_uint32, C.c_uint32]
    return _lib


def _arr(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def _ptr(a):
    return None if a is None else a.ctypes.data


class _Keep:
    """Holds converted arrays alive next to the C struct that points at them."""

    def __init__(self):
        self.refs = []

    def add(self, a, dtype):
        if a is None:
            return None
        a = _arr(a, dtype)
        self.refs.append(a)
        return a.ctypes.data


def _c_pipeline(p, keep: _Keep) -> _Pipeline:
    return _Pipeline(int(p.n_stages), keep.add(p.sub_offsets, np.int32),
                     keep.add(p.sub_ids, np.int32), keep.add(p.bmax, np.int32),
                     keep.add(p.lat_offsets, np.int64), keep.add(p.lat_us, np.int64))


def count_paths(p, stage: int) -> int:
    k = _Keep()
    cp = _c_pipeline(p, k)
    return int(lib().oracle_count_paths(C.addressof(cp), stage))


def slot_base(p, stage: int) -> int:
    k = _Keep()
    cp = _c_pipeline(p, k)
    return int(lib().oracle_slot_base(C.addressof(cp), stage))


def lsub(p, stage: int, batch_row, q_row, w_row=None) -> int:
    k = _Keep()
    cp = _c_pipeline(p, k)
    return int(lib().oracle_lsub(C.addressof(cp), stage, k.add(batch_row, np.int32),
                                 k.add(q_row, np.int64), k.add(w_row, np.int64)))


def lsub_masked(p, stage: int, batch_row, q_row, w_row, mask: int) -> int:
    """L_sub over the downstream paths whose bit is set in `mask` (0 = all); -1 if none exists."""
    k = _Keep()
    cp = _c_pipeline(p, k)
    return int(lib().oracle_lsub_masked(C.addressof(cp), stage, k.add(batch_row, np.int32),
                                        k.add(q_row, np.int64), k.add(w_row, np.int64), mask))


def estimate_w(pipelines, pipeline_of_ctx, n_ctx: int, stage_stride: int, slot_stride: int, wait_samples,
               lambda_num: int = 1, lambda_den: int = 10, seed: int = 0) -> np.ndarray:
    """w[n_ctx, slot_stride] (int64): the batch-wait estimate of every (stage, downstream path) slot.
    wait_samples: int32 [n_ctx, stage_stride, M]."""
    k = _Keep()
    cps = (_Pipeline * len(pipelines))(*[_c_pipeline(p, k) for p in pipelines])
    ws = np.ascontiguousarray(wait_samples, dtype=np.int32)
    assert ws.shape[0] == n_ctx and ws.shape[1] == stage_stride
    M = int(ws.shape[2])
    w = np.zeros((n_ctx, slot_stride), dtype=np.int64)
    rc = lib().oracle_estimate_w(C.addressof(cps), len(pipelines), k.add(pipeline_of_ctx, np.int32), n_ctx,
                                 stage_stride, slot_stride, ws.ctypes.data, M, lambda_num, lambda_den,
                                 seed & (2**64 - 1), w.ctypes.data)
    if rc != 0:
        raise ValueError("oracle_estimate_w: bad input")
    return w


def update_priority(pipelines, pipeline_of_ctx, n_ctx: int, stage_stride: int, batch, workers, arrivals,
                    window: int, interval_us: int, priority) -> np.ndarray:
    """New decision order of every (ctx, stage) queue (uint8 [n_ctx, stage_stride]; 0 = low budget
    first, 1 = high budget first) from the previous one and the arrival history
    (uint32 [n_ctx, stage_stride, n_hist])."""
    k = _Keep()
    cps = (_Pipeline * len(pipelines))(*[_c_pipeline(p, k) for p in pipelines])
    x = np.ascontiguousarray(arrivals, dtype=np.uint32)
    assert x.shape[0] == n_ctx and x.shape[1] == stage_stride
    out = np.array(priority, dtype=np.uint8).reshape(n_ctx, stage_stride).copy()
    rc = lib().oracle_update_priority(C.addressof(cps), len(pipelines), k.add(pipeline_of_ctx, np.int32), n_ctx,
                                      stage_stride, k.add(batch, np.int32), k.add(workers, np.int32),
                                      x.ctypes.data, int(x.shape[2]), window, interval_us, out.ctypes.data)
    if rc != 0:
        raise ValueError("oracle_update_priority: bad input")
    return out


def queue_delay(now_us, sample_time_us, sample_delay_us, window_us: int) -> np.ndarray:
    """q[n_ctx, stage_stride] (int64): the linear weighted sliding-window average of the recorded
    queueing delays.  sample_time_us int64 and sample_delay_us int32 are [n_ctx, stage_stride, M]."""
    t = np.ascontiguousarray(sample_time_us, dtype=np.int64)
    d = np.ascontiguousarray(sample_delay_us, dtype=np.int32)
    now = np.ascontiguousarray(now_us, dtype=np.int64)
    assert t.shape == d.shape and t.ndim == 3 and now.shape == (t.shape[0],)
    q = np.zeros(t.shape[:2], dtype=np.int64)
    rc = lib().oracle_queue_delay(t.shape[0], t.shape[1], now.ctypes.data, t.ctypes.data, d.ctypes.data,
                                  t.shape[2], window_us, q.ctypes.data)
    if rc != 0:
        raise ValueError("oracle_queue_delay: bad input")
    return q


def advance_state(pipelines, pipeline_of_ctx, n_ctx: int, stage_stride: int, now_us, batch, workers, seg_kept,
                  free_at_us, sample_time_us, sample_delay_us, slot: int) -> None:
    """In place: free_at_us (int64 [n_ctx, S]) and slot `slot` of the sample rings (int64 / int32
    [n_ctx, S, M]; pass None, None to keep no samples)."""
    k = _Keep()
    cps = (_Pipeline * len(pipelines))(*[_c_pipeline(p, k) for p in pipelines])
    assert free_at_us.dtype == np.int64 and free_at_us.flags.c_contiguous
    M = 0
    if sample_time_us is not None:
        assert sample_time_us.dtype == np.int64 and sample_delay_us.dtype == np.int32
        assert sample_time_us.flags.c_contiguous and sample_delay_us.flags.c_contiguous
        M = int(sample_time_us.shape[2])
    rc = lib().oracle_advance_state(C.addressof(cps), len(pipelines), k.add(pipeline_of_ctx, np.int32), n_ctx,
                                    stage_stride, k.add(now_us, np.int64), k.add(batch, np.int32),
                                    k.add(workers, np.int32), k.add(seg_kept, np.uint32), free_at_us.ctypes.data,
                                    None if M == 0 else sample_time_us.ctypes.data,
                                    None if M == 0 else sample_delay_us.ctypes.data, M, slot)
    if rc != 0:
        raise ValueError("oracle_advance_state: bad input")


MODE_RAW, MODE_PATH_MASK, MODE_FCFS, MODE_NEXUS, MODE_CLIPPER = 1, 16, 32, 64, 128


def plan(pipelines, requests, state, n_ctx: int, mode: int = 0, arrivals=None) -> dict:
    """Runs the oracle planner; returns a dict of numpy outputs.  `arrivals` (records of
    two int64: arrive_us, slo_us) is needed by MODE_CLIPPER only."""
    k = _Keep()
    cps = (_Pipeline * len(pipelines))(*[_c_pipeline(p, k) for p in pipelines])
    req = np.ascontiguousarray(requests)
    assert req.dtype.itemsize == 16
    n = int(req.shape[0])
    S = int(state.stage_stride)
    cst = _State(S, int(state.slot_stride),
                 k.add(state.pipeline_of_ctx, np.int32), k.add(state.now_us, np.int64),
                 k.add(state.batch, np.int32), k.add(state.free_at_us, np.int64),
                 k.add(state.q_us, np.int64), k.add(state.w_us, np.int64),
                 k.add(state.workers, np.int32),
                 k.add(getattr(state, "priority", None), np.uint8))
    out = {
        "keep": np.zeros(n, np.uint8), "est_us": np.zeros(n, np.int64),
        "perm": np.zeros(n, np.uint32), "kept_idx": np.zeros(n, np.uint32),
        "n_kept": np.zeros(1, np.uint64),
        "seg_offsets": np.zeros(n_ctx * S + 1, np.uint32),
        "seg_kept": np.zeros(n_ctx * S, np.uint32),
        "ctx_total": np.zeros(n_ctx, np.int64), "ctx_kept": np.zeros(n_ctx, np.int64),
    }
    arr = None
    if arrivals is not None:
        arr = np.ascontiguousarray(arrivals)
        assert arr.dtype.itemsize == 16 and arr.shape[0] == n
    rc = lib().oracle_plan_policy(C.addressof(cps), len(pipelines), req.ctypes.data, _ptr(arr), n,
                           C.addressof(cst), n_ctx, mode,
                           *[out[key].ctypes.data for key in
                             ("keep", "est_us", "perm", "kept_idx", "n_kept",
                              "seg_offsets", "seg_kept", "ctx_total", "ctx_kept")])
    if rc != 0:
        raise ValueError("oracle_plan: input out of range")
    out["n_kept"] = int(out["n_kept"][0])
    out["kept_idx"] = out["kept_idx"][:out["n_kept"]]
    return out
