"""Thin Python binding of libpard (the C-ABI CUDA library).

Argument marshalling only: every step of the planner runs in the library's
kernels.  PyTorch is used for device memory and streams.  The functions carry
the names of the C entry points declared in include/pard.h.  There is no CPU
fallback: a missing library raises at the first call.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpard.so")

PARD_OK = 0
PARD_EINVAL, PARD_ECYCLE, PARD_ERANGE, PARD_ENOMEM = -1, -2, -3, -4
PARD_EWORKSPACE, PARD_ETIMEOUT, PARD_ECUDA, PARD_EDATA, PARD_ESTATIC = -5, -6, -7, -8, -9
PARD_STATIC_SCRATCH_BYTES = 8 << 20
PARD_LOAD_HOST_ONLY = 1
PARD_MODE_ADMITTED, PARD_MODE_RAW, PARD_MODE_NOWAIT, PARD_MODE_SCAN, PARD_MODE_TEST_STALL = 0, 1, 2, 4, 8
PARD_MODE_PATH_MASK, PARD_MODE_FCFS, PARD_MODE_NEXUS, PARD_MODE_CLIPPER = 16, 32, 64, 128
PARD_MODE_GROUPED = 256
PARD_N_PHASES = 15
PARD_PROFILE_COARSE = 0x80000000
PARD_MAX_WAIT_SAMPLES = 1 << 15
PARD_WAIT_LIMIT_US = 1 << 24
PARD_MAX_HISTORY = 4096
PARD_RATE_LIMIT = 1 << 24
PARD_MAX_DELAY_SAMPLES = 1 << 15
PARD_MAX_DELAY_WINDOW_US = 1 << 24

EXPORTS = ["pard_strerror", "pard_load_pipeline", "pard_free_pipeline", "pard_pipeline_n_stages",
           "pard_pipeline_n_slots", "pard_pipeline_paths", "pard_plan_workspace_bytes", "pard_plan",
           "pard_plan_host_workspace_bytes", "pard_plan_host", "pard_goodput", "pard_plan_status", "pard_plan_policy",
           "pard_plan_kernel_launches", "pard_profile_begin", "pard_profile_end",
           "pard_profile_phase_name", "pard_plan_static", "pard_estimate_w_workspace_bytes",
           "pard_estimate_w", "pard_update_priority_workspace_bytes", "pard_update_priority",
           "pard_update_queue_delay_workspace_bytes", "pard_update_queue_delay",
           "pard_advance_state_workspace_bytes", "pard_advance_state"]


class PardError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (%d)" % (where, pard_strerror(status), status))


class _Dag(C.Structure):
    _fields_ = [("n_stages", C.c_int32), ("sub_offsets", C.c_void_p), ("sub_ids", C.c_void_p)]


class _Profile(C.Structure):
    _fields_ = [("bmax", C.c_void_p), ("lat_offsets", C.c_void_p), ("lat_us", C.c_void_p)]


class _State(C.Structure):
    _fields_ = [("stage_stride", C.c_int32), ("slot_stride", C.c_int32),
                ("d_pipeline_of_ctx", C.c_void_p), ("d_now_us", C.c_void_p),
                ("d_batch", C.c_void_p), ("d_free_at_us", C.c_void_p), ("d_q_us", C.c_void_p),
                ("d_w_us", C.c_void_p), ("d_workers", C.c_void_p), ("d_priority", C.c_void_p)]


class _Out(C.Structure):
    _fields_ = [("d_keep", C.c_void_p), ("d_est_us", C.c_void_p), ("d_perm", C.c_void_p),
                ("d_kept_idx", C.c_void_p), ("d_n_kept", C.c_void_p),
                ("d_seg_offsets", C.c_void_p), ("d_seg_kept", C.c_void_p)]


_lib = None


def library() -> C.CDLL:
    """Loads libpard.so; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libpard.so is missing: run `python -m paper_2602_08747_b200.build`")
        lib = C.CDLL(LIB_PATH)
        lib.pard_strerror.restype = C.c_char_p
        lib.pard_strerror.argtypes = [C.c_int]
        lib.pard_load_pipeline.argtypes = [C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p]
        lib.pard_free_pipeline.argtypes = [C.c_void_p]
        lib.pard_pipeline_n_stages.argtypes = [C.c_void_p, C.c_void_p]
        lib.pard_pipeline_n_slots.argtypes = [C.c_void_p, C.c_void_p]
        lib.pard_pipeline_paths.argtypes = [C.c_void_p, C.c_int32] + [C.c_void_p] * 4
        lib.pard_plan_workspace_bytes.argtypes = [C.c_uint64, C.c_uint32, C.c_int32, C.c_void_p]
        lib.pard_plan_host_workspace_bytes.argtypes = [C.c_uint64, C.c_uint32, C.c_int32, C.c_int32,
                                                       C.c_void_p]
        plan_args = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_uint64, C.c_void_p, C.c_uint32,
                     C.c_uint32, C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p]
        lib.pard_plan.argtypes = plan_args
        lib.pard_plan_policy.argtypes = plan_args[:3] + [C.c_void_p] + plan_args[3:]
        lib.pard_plan_host.argtypes = plan_args
        lib.pard_goodput.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint32, C.c_int32,
                                     C.c_void_p, C.c_void_p, C.c_void_p]
        lib.pard_plan_static.argtypes = plan_args[:8] + [C.c_void_p]
        lib.pard_plan_status.argtypes = [C.c_void_p, C.c_void_p]
        lib.pard_plan_kernel_launches.argtypes = [C.c_uint64, C.c_uint32, C.c_int32, C.c_void_p]
        lib.pard_estimate_w_workspace_bytes.argtypes = [C.c_uint32, C.c_void_p]
        lib.pard_estimate_w.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_uint32, C.c_int32, C.c_int32,
                                        C.c_void_p, C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint64, C.c_uint32,
                                        C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p]
        lib.pard_update_priority_workspace_bytes.argtypes = [C.c_uint32, C.c_void_p]
        lib.pard_update_priority.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_uint32, C.c_int32,
                                             C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint32, C.c_uint32,
                                             C.c_uint32, C.c_uint32, C.c_void_p, C.c_void_p, C.c_uint64,
                                             C.c_void_p]
        lib.pard_update_queue_delay_workspace_bytes.argtypes = [C.c_void_p]
        lib.pard_update_queue_delay.argtypes = [C.c_uint32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                                C.c_uint32, C.c_uint32, C.c_uint32, C.c_void_p, C.c_void_p,
                                                C.c_uint64, C.c_void_p]
        lib.pard_advance_state_workspace_bytes.argtypes = [C.c_uint32, C.c_void_p]
        lib.pard_advance_state.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_uint32, C.c_int32] + \
            [C.c_void_p] * 7 + [C.c_uint32, C.c_uint32, C.c_uint32, C.c_void_p, C.c_uint64, C.c_void_p]
        lib.pard_profile_begin.argtypes = [C.c_uint32, C.c_uint32]
        lib.pard_profile_end.argtypes = [C.c_void_p, C.c_void_p]
        lib.pard_profile_phase_name.restype = C.c_char_p
        lib.pard_profile_phase_name.argtypes = [C.c_uint32]
        for name in EXPORTS:
            if name not in ("pard_strerror", "pard_profile_phase_name"):
                getattr(lib, name).restype = C.c_int
        _lib = lib
    return _lib


def pard_strerror(status: int) -> str:
    return library().pard_strerror(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != PARD_OK:
        raise PardError(status, where)


def _ptr(t) -> Optional[int]:
    """Address of a torch tensor / numpy array (None stays NULL)."""
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


class Pipeline:
    """Owns one pard_pipeline_t handle."""

    def __init__(self, handle: int):
        self._h = C.c_void_p(handle)

    def __del__(self):
        try:
            self.free()
        except Exception:          # interpreter shutdown: the module globals are already gone
            pass

    def free(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            library().pard_free_pipeline(self._h)
            self._h = C.c_void_p(None)

    @property
    def handle(self) -> int:
        return self._h.value

    @property
    def n_stages(self) -> int:
        v = C.c_int32()
        _check(library().pard_pipeline_n_stages(self._h, C.byref(v)), "pard_pipeline_n_stages")
        return v.value

    @property
    def n_slots(self) -> int:
        v = C.c_int32()
        _check(library().pard_pipeline_n_slots(self._h, C.byref(v)), "pard_pipeline_n_slots")
        return v.value

    def paths(self, stage: int):
        """(slot_base, [tuple of stage ids per downstream path])."""
        n, base = C.c_int32(), C.c_int32()
        offs, ids = C.POINTER(C.c_int32)(), C.POINTER(C.c_int32)()
        _check(library().pard_pipeline_paths(self._h, stage, C.byref(n), C.byref(base),
                                             C.byref(offs), C.byref(ids)), "pard_pipeline_paths")
        out = [tuple(ids[offs[j]:offs[j + 1]]) for j in range(n.value)]
        return base.value, out


def pard_load_pipeline(p, host_only: bool = False) -> Pipeline:
    """p: object with n_stages, sub_offsets, sub_ids, bmax, lat_offsets, lat_us."""
    so = np.ascontiguousarray(p.sub_offsets, dtype=np.int32)
    si = np.ascontiguousarray(p.sub_ids, dtype=np.int32)
    bm = np.ascontiguousarray(p.bmax, dtype=np.int32)
    lo = np.ascontiguousarray(p.lat_offsets, dtype=np.int64)
    lu = np.ascontiguousarray(p.lat_us, dtype=np.int64)
    dag = _Dag(int(p.n_stages), so.ctypes.data, si.ctypes.data if si.size else None)
    prof = _Profile(bm.ctypes.data, lo.ctypes.data, lu.ctypes.data)
    h = C.c_void_p()
    _check(library().pard_load_pipeline(C.byref(dag), C.byref(prof),
                                        PARD_LOAD_HOST_ONLY if host_only else 0, C.byref(h)),
           "pard_load_pipeline")
    return Pipeline(h.value)


@dataclass
class QueueStateArrays:
    """The pard_queue_state_t members as tensors (device) or arrays (host)."""
    stage_stride: int
    slot_stride: int
    now_us: object
    batch: object
    free_at_us: object
    q_us: object
    w_us: object = None
    workers: object = None
    pipeline_of_ctx: object = None
    priority: object = None

    def c_struct(self) -> _State:
        return _State(self.stage_stride, self.slot_stride, _ptr(self.pipeline_of_ctx),
                      _ptr(self.now_us), _ptr(self.batch), _ptr(self.free_at_us), _ptr(self.q_us),
                      _ptr(self.w_us), _ptr(self.workers), _ptr(self.priority))


@dataclass
class PlanOut:
    """The pard_plan_out_t members as tensors (device) or arrays (host)."""
    keep: object = None
    est_us: object = None
    perm: object = None
    kept_idx: object = None
    n_kept: object = None
    seg_offsets: object = None
    seg_kept: object = None

    def c_struct(self) -> _Out:
        return _Out(_ptr(self.keep), _ptr(self.est_us), _ptr(self.perm), _ptr(self.kept_idx),
                    _ptr(self.n_kept), _ptr(self.seg_offsets), _ptr(self.seg_kept))


def pard_plan_workspace_bytes(n: int, n_ctx: int, stage_stride: int) -> int:
    v = C.c_uint64()
    _check(library().pard_plan_workspace_bytes(n, n_ctx, stage_stride, C.byref(v)),
           "pard_plan_workspace_bytes")
    return v.value


def pard_plan_host_workspace_bytes(n: int, n_ctx: int, stage_stride: int, slot_stride: int) -> int:
    v = C.c_uint64()
    _check(library().pard_plan_host_workspace_bytes(n, n_ctx, stage_stride, slot_stride, C.byref(v)),
           "pard_plan_host_workspace_bytes")
    return v.value


def _handles(pipelines: Sequence[Pipeline]):
    return (C.c_void_p * len(pipelines))(*[p.handle for p in pipelines])


def pard_plan(pipelines: Sequence[Pipeline], d_requests, n: int, state: QueueStateArrays,
              n_ctx: int, mode: int, out: PlanOut, d_workspace, workspace_bytes: Optional[int] = None,
              stream: int = 0, check: bool = True) -> int:
    hs = _handles(pipelines)
    st, o = state.c_struct(), out.c_struct()
    wb = workspace_bytes if workspace_bytes is not None else d_workspace.numel() * d_workspace.element_size()
    rc = library().pard_plan(hs, len(pipelines), _ptr(d_requests), n, C.byref(st), n_ctx, mode,
                             C.byref(o), _ptr(d_workspace), wb, stream or None)
    if check:
        _check(rc, "pard_plan")
    return rc


def pard_plan_policy(pipelines: Sequence[Pipeline], d_requests, d_arrivals, n: int, state: QueueStateArrays,
                     n_ctx: int, mode: int, out: PlanOut, d_workspace, workspace_bytes: Optional[int] = None,
                     stream: int = 0, check: bool = True) -> int:
    hs = _handles(pipelines)
    st, o = state.c_struct(), out.c_struct()
    wb = workspace_bytes if workspace_bytes is not None else d_workspace.numel() * d_workspace.element_size()
    rc = library().pard_plan_policy(hs, len(pipelines), _ptr(d_requests), _ptr(d_arrivals), n, C.byref(st), n_ctx,
                                    mode, C.byref(o), _ptr(d_workspace), wb, stream or None)
    if check:
        _check(rc, "pard_plan_policy")
    return rc


def pard_plan_host(pipelines: Sequence[Pipeline], requests, n: int, state: QueueStateArrays,
                   n_ctx: int, mode: int, out: PlanOut, d_workspace,
                   workspace_bytes: Optional[int] = None, stream: int = 0, check: bool = True) -> int:
    hs = _handles(pipelines)
    st, o = state.c_struct(), out.c_struct()
    wb = workspace_bytes if workspace_bytes is not None else d_workspace.numel() * d_workspace.element_size()
    rc = library().pard_plan_host(hs, len(pipelines), _ptr(requests), n, C.byref(st), n_ctx, mode,
                                  C.byref(o), _ptr(d_workspace), wb, stream or None)
    if check:
        _check(rc, "pard_plan_host")
    return rc


def pard_plan_static(pipelines: Sequence[Pipeline], d_requests, n: int, state: QueueStateArrays,
                     n_ctx: int, mode: int, out: PlanOut, stream: int = 0, check: bool = True) -> int:
    """pard_plan without a workspace argument: the scratch is the library's own
    fixed device array, for callers that must not allocate device memory
    (problems up to PARD_STATIC_SCRATCH_BYTES of scratch; larger ones return
    PARD_ESTATIC).  Calls on one device share that array and must not overlap."""
    hs = _handles(pipelines)
    st, o = state.c_struct(), out.c_struct()
    rc = library().pard_plan_static(hs, len(pipelines), _ptr(d_requests), n, C.byref(st), n_ctx, mode,
                                    C.byref(o), stream or None)
    if check:
        _check(rc, "pard_plan_static")
    return rc


def pard_plan_status(d_workspace, stream: int = 0, check: bool = True) -> int:
    rc = library().pard_plan_status(_ptr(d_workspace), stream or None)
    if check:
        _check(rc, "pard_plan_status")
    return rc


def pard_plan_kernel_launches(n: int, n_ctx: int, stage_stride: int) -> int:
    v = C.c_uint32()
    _check(library().pard_plan_kernel_launches(n, n_ctx, stage_stride, C.byref(v)),
           "pard_plan_kernel_launches")
    return v.value


def pard_profile_begin(every: int, max_samples: int) -> None:
    _check(library().pard_profile_begin(every, max_samples), "pard_profile_begin")


def pard_profile_end() -> dict:
    """{"n_samples": k, "ms": {phase name: milliseconds summed over the k sampled calls}}"""
    ms = (C.c_float * PARD_N_PHASES)()
    k = C.c_uint32()
    _check(library().pard_profile_end(ms, C.byref(k)), "pard_profile_end")
    names = [library().pard_profile_phase_name(i).decode() for i in range(PARD_N_PHASES)]
    return {"n_samples": k.value, "ms": {names[i]: float(ms[i]) for i in range(PARD_N_PHASES)}}


def pard_goodput(d_keep, d_seg_offsets, d_seg_kept, n: int, n_ctx: int, stage_stride: int, d_out_total,
                 d_out_kept, stream: int = 0, check: bool = True) -> int:
    rc = library().pard_goodput(_ptr(d_keep), _ptr(d_seg_offsets), _ptr(d_seg_kept), n, n_ctx, stage_stride,
                                _ptr(d_out_total), _ptr(d_out_kept), stream or None)
    if check:
        _check(rc, "pard_goodput")
    return rc


def pard_estimate_w_workspace_bytes(n_pipelines: int) -> int:
    b = C.c_uint64()
    _check(library().pard_estimate_w_workspace_bytes(n_pipelines, C.byref(b)), "pard_estimate_w_workspace_bytes")
    return b.value


def pard_estimate_w(pipelines: Sequence[Pipeline], d_pipeline_of_ctx, n_ctx: int, stage_stride: int,
                    slot_stride: int, d_wait_samples, n_samples: int, lambda_num: int, lambda_den: int,
                    seed: int, mode: int, d_w_us, d_workspace, workspace_bytes: Optional[int] = None,
                    stream: int = 0, check: bool = True) -> int:
    hs = _handles(pipelines)
    wb = workspace_bytes if workspace_bytes is not None else d_workspace.numel() * d_workspace.element_size()
    rc = library().pard_estimate_w(hs, len(pipelines), _ptr(d_pipeline_of_ctx), n_ctx, stage_stride,
                                   slot_stride, _ptr(d_wait_samples), n_samples, lambda_num, lambda_den,
                                   seed & (2**64 - 1), mode, _ptr(d_w_us), _ptr(d_workspace),
                                   wb, stream or None)
    if check:
        _check(rc, "pard_estimate_w")
    return rc


def pard_update_priority_workspace_bytes(n_pipelines: int) -> int:
    b = C.c_uint64()
    _check(library().pard_update_priority_workspace_bytes(n_pipelines, C.byref(b)),
           "pard_update_priority_workspace_bytes")
    return b.value


def pard_update_priority(pipelines: Sequence[Pipeline], d_pipeline_of_ctx, n_ctx: int, stage_stride: int,
                         d_batch, d_workers, d_arrivals, n_hist: int, window: int, interval_us: int,
                         mode: int, d_priority, d_workspace, workspace_bytes: Optional[int] = None,
                         stream: int = 0, check: bool = True) -> int:
    hs = _handles(pipelines)
    wb = workspace_bytes if workspace_bytes is not None else d_workspace.numel() * d_workspace.element_size()
    rc = library().pard_update_priority(hs, len(pipelines), _ptr(d_pipeline_of_ctx), n_ctx, stage_stride,
                                        _ptr(d_batch), _ptr(d_workers), _ptr(d_arrivals), n_hist, window,
                                        interval_us, mode, _ptr(d_priority), _ptr(d_workspace), wb,
                                        stream or None)
    if check:
        _check(rc, "pard_update_priority")
    return rc


def pard_update_queue_delay_workspace_bytes() -> int:
    b = C.c_uint64()
    _check(library().pard_update_queue_delay_workspace_bytes(C.byref(b)), "pard_update_queue_delay_workspace_bytes")
    return b.value


def pard_update_queue_delay(n_ctx: int, stage_stride: int, d_now_us, d_sample_time_us, d_sample_delay_us,
                            n_samples: int, window_us: int, mode: int, d_q_us, d_workspace,
                            workspace_bytes: Optional[int] = None, stream: int = 0, check: bool = True) -> int:
    wb = workspace_bytes if workspace_bytes is not None else d_workspace.numel() * d_workspace.element_size()
    rc = library().pard_update_queue_delay(n_ctx, stage_stride, _ptr(d_now_us), _ptr(d_sample_time_us),
                                           _ptr(d_sample_delay_us), n_samples, window_us, mode, _ptr(d_q_us),
                                           _ptr(d_workspace), wb, stream or None)
    if check:
        _check(rc, "pard_update_queue_delay")
    return rc


def pard_advance_state_workspace_bytes(n_pipelines: int) -> int:
    b = C.c_uint64()
    _check(library().pard_advance_state_workspace_bytes(n_pipelines, C.byref(b)), "pard_advance_state_workspace_bytes")
    return b.value


def pard_advance_state(pipelines: Sequence[Pipeline], d_pipeline_of_ctx, n_ctx: int, stage_stride: int, d_now_us,
                       d_batch, d_workers, d_seg_kept, d_free_at_us, d_sample_time_us, d_sample_delay_us,
                       n_samples: int, slot: int, mode: int, d_workspace, workspace_bytes: Optional[int] = None,
                       stream: int = 0, check: bool = True) -> int:
    hs = _handles(pipelines)
    wb = workspace_bytes if workspace_bytes is not None else d_workspace.numel() * d_workspace.element_size()
    rc = library().pard_advance_state(hs, len(pipelines), _ptr(d_pipeline_of_ctx), n_ctx, stage_stride,
                                      _ptr(d_now_us), _ptr(d_batch), _ptr(d_workers), _ptr(d_seg_kept),
                                      _ptr(d_free_at_us), _ptr(d_sample_time_us), _ptr(d_sample_delay_us),
                                      n_samples, slot, mode, _ptr(d_workspace), wb, stream or None)
    if check:
        _check(rc, "pard_advance_state")
    return rc


# --------------------------------------------------------------------------
# conveniences: move a workload to the device and allocate outputs (memory only)
# --------------------------------------------------------------------------
def device_requests(requests: np.ndarray, device="cuda"):
    import torch
    raw = np.ascontiguousarray(requests).view(np.uint8).reshape(-1, 16)
    return torch.from_numpy(raw).to(device)


def device_state(state, device="cuda") -> QueueStateArrays:
    import torch

    def mv(a, dt):
        return None if a is None else torch.from_numpy(np.ascontiguousarray(a, dtype=dt)).to(device)

    return QueueStateArrays(int(state.stage_stride), int(state.slot_stride),
                            mv(state.now_us, np.int64), mv(state.batch, np.int32),
                            mv(state.free_at_us, np.int64), mv(state.q_us, np.int64),
                            mv(state.w_us, np.int64), mv(state.workers, np.int32),
                            mv(state.pipeline_of_ctx, np.int32),
                            mv(getattr(state, "priority", None), np.uint8))


def alloc_out(n: int, n_seg: int, device="cuda") -> PlanOut:
    import torch
    m = max(n, 1)
    return PlanOut(keep=torch.empty(m, dtype=torch.uint8, device=device),
                   est_us=torch.empty(m, dtype=torch.int64, device=device),
                   perm=torch.empty(m, dtype=torch.int32, device=device),
                   kept_idx=torch.empty(m, dtype=torch.int32, device=device),
                   n_kept=torch.zeros(1, dtype=torch.int64, device=device),
                   seg_offsets=torch.empty(n_seg + 1, dtype=torch.int32, device=device),
                   seg_kept=torch.empty(n_seg, dtype=torch.int32, device=device))


def alloc_workspace(nbytes: int, device="cuda"):
    import torch
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)


def out_to_numpy(out: PlanOut, n: int) -> dict:
    """Copies outputs to the host as the unsigned types of the C interface."""
    nk = int(out.n_kept.cpu()[0])
    return {
        "keep": out.keep[:n].cpu().numpy(),
        "est_us": out.est_us[:n].cpu().numpy(),
        "perm": out.perm[:n].cpu().numpy().view(np.uint32),
        "n_kept": nk,
        "kept_idx": out.kept_idx[:nk].cpu().numpy().view(np.uint32),
        "seg_offsets": out.seg_offsets.cpu().numpy().view(np.uint32),
        "seg_kept": out.seg_kept.cpu().numpy().view(np.uint32),
    }
