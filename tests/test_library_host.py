"""Host-side checks of libpard that need no GPU: the library loads, exports
every entry point the header declares, enumerates downstream paths like an
independent enumeration, and rejects malformed pipelines."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import oracle
from paper_2602_08747_b200 import binding as pb
from paper_2602_08747_b200 import build as pbuild
from paper_2602_08747_b200 import inputs
from tests import util

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _lib():
    pbuild.build()
    return pb.library()


def test_every_declared_symbol_is_exported():
    text = open(os.path.join(ROOT, "include", "pard.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(pard_[a-z_0-9]+)\s*\(", text))
    assert declared, "no declarations found"
    lib = pb.library()
    for name in sorted(declared):
        assert hasattr(lib, name), name
    assert declared == set(pb.EXPORTS)


def test_strerror_covers_all_codes():
    seen = set()
    for code in range(0, -10, -1):
        s = pb.pard_strerror(code)
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 10
    assert pb.pard_strerror(-99) == "unknown status"


@pytest.mark.parametrize("seed", range(10))
def test_path_enumeration_matches_independent_enumeration(seed):
    rng = np.random.default_rng(700 + seed)
    S = int(rng.integers(1, 17))
    edges = inputs.random_dag_edges(rng, S) if S > 1 else []
    # shuffle successor order: the library must order paths itself
    edges = [edges[i] for i in rng.permutation(len(edges))]
    p = inputs.make_pipeline(edges, S, [2] * S, [[5, 6]] * S)
    h = pb.pard_load_pipeline(p, host_only=True)
    assert h.n_stages == S
    assert h.n_slots == inputs.n_slots(p)
    base = 0
    for k in range(S):
        want = util.explicit_paths(p, k)
        slot_base, got = h.paths(k)
        assert slot_base == base == oracle.slot_base(p, k)
        assert got == want
        assert len(got) == oracle.count_paths(p, k)
        base += len(want)
    h.free()


def test_named_dags_have_the_stated_shape():
    p8 = inputs.make_pipeline(inputs.DAG8_EDGES, 8, [1] * 8, [[1]] * 8)
    p16 = inputs.make_pipeline(inputs.DAG16_EDGES, 16, [1] * 16, [[1]] * 16)
    assert inputs.n_source_sink_paths(p8) == 3
    assert inputs.n_source_sink_paths(p16) == 12
    h = pb.pard_load_pipeline(p16, host_only=True)
    assert h.paths(0)[1][0] == (1, 2, 5, 11, 12, 14, 15)
    assert len(h.paths(0)[1]) == 12 and h.n_slots == 45


def _load_raw(n_stages, sub_offsets, sub_ids, bmax, lat_offsets, lat_us, flags=1):
    so = np.asarray(sub_offsets, np.int32)
    si = np.asarray(sub_ids, np.int32)
    bm = np.asarray(bmax, np.int32)
    lo = np.asarray(lat_offsets, np.int64)
    lu = np.asarray(lat_us, np.int64)
    dag = pb._Dag(n_stages, so.ctypes.data, si.ctypes.data if si.size else None)
    prof = pb._Profile(bm.ctypes.data, lo.ctypes.data, lu.ctypes.data)
    h = C.c_void_p()
    rc = pb.library().pard_load_pipeline(C.byref(dag), C.byref(prof), flags, C.byref(h))
    if rc == 0:
        pb.library().pard_free_pipeline(h)
    else:
        assert h.value is None
    return rc


def test_malformed_pipelines_are_rejected():
    ok = dict(n_stages=2, sub_offsets=[0, 1, 1], sub_ids=[1], bmax=[1, 1], lat_offsets=[0, 1, 2],
              lat_us=[5, 5])
    assert _load_raw(**ok) == pb.PARD_OK
    assert _load_raw(**{**ok, "sub_ids": [0]}) == pb.PARD_EINVAL                 # self loop
    assert _load_raw(**{**ok, "sub_ids": [2]}) == pb.PARD_EINVAL                 # id out of range
    assert _load_raw(**{**ok, "sub_offsets": [0, 2, 2], "sub_ids": [1, 1]}) == pb.PARD_EINVAL  # duplicate edge
    assert _load_raw(**{**ok, "sub_offsets": [1, 1, 1]}) == pb.PARD_EINVAL
    assert _load_raw(**{**ok, "sub_offsets": [0, 1, 0]}) == pb.PARD_EINVAL
    assert _load_raw(**{**ok, "sub_offsets": [0, 1, 2], "sub_ids": [1, 0]}) == pb.PARD_ECYCLE
    assert _load_raw(**{**ok, "bmax": [0, 1]}) == pb.PARD_EINVAL
    assert _load_raw(**{**ok, "bmax": [1, 5000], "lat_offsets": [0, 1, 5001],
                        "lat_us": [5] * 5001}) == pb.PARD_ERANGE
    assert _load_raw(**{**ok, "lat_offsets": [0, 1, 3], "lat_us": [5, 5, 5]}) == pb.PARD_EINVAL
    assert _load_raw(**{**ok, "lat_us": [5, 0]}) == pb.PARD_ERANGE
    assert _load_raw(**{**ok, "lat_us": [5, 1 << 40]}) == pb.PARD_ERANGE
    assert _load_raw(**{**ok, "n_stages": 0}) == pb.PARD_EINVAL
    assert _load_raw(**{**ok, "n_stages": 65}) == pb.PARD_ERANGE
    assert _load_raw(**ok, flags=2) == pb.PARD_EINVAL
    lib = pb.library()
    assert lib.pard_load_pipeline(None, None, 1, None) == pb.PARD_EINVAL
    # 3-cycle behind a valid prefix
    assert _load_raw(4, [0, 1, 2, 3, 4], [1, 2, 3, 1], [1] * 4, [0, 1, 2, 3, 4], [5] * 4) == pb.PARD_ECYCLE


def test_path_explosion_is_rejected_before_enumeration():
    # 40 stages in 20 layers of 2, fully connected between layers: 2^19 paths per source
    S = 40
    edges = []
    for layer in range(19):
        for a in (2 * layer, 2 * layer + 1):
            for b in (2 * layer + 2, 2 * layer + 3):
                edges.append((a, b))
    p = inputs.make_pipeline(edges, S, [1] * S, [[1]] * S)
    with pytest.raises(pb.PardError) as e:
        pb.pard_load_pipeline(p, host_only=True)
    assert e.value.status == pb.PARD_ERANGE


def test_plan_argument_checks_happen_before_any_launch():
    p = inputs.make_pipeline(inputs.chain_edges(2), 2, [1, 1], [[5], [5]])
    h = pb.pard_load_pipeline(p, host_only=True)
    lib = pb.library()
    v = C.c_uint64()
    assert lib.pard_plan_workspace_bytes(10, 0, 2, C.byref(v)) == pb.PARD_EINVAL
    assert lib.pard_plan_workspace_bytes(10, 1, 0, C.byref(v)) == pb.PARD_EINVAL
    assert lib.pard_plan_workspace_bytes(1 << 30, 1, 2, C.byref(v)) == pb.PARD_ERANGE
    assert lib.pard_plan_workspace_bytes(10, 1 << 20, 64, C.byref(v)) == pb.PARD_ERANGE
    assert lib.pard_plan_workspace_bytes(10, 1, 2, None) == pb.PARD_EINVAL
    assert lib.pard_plan_workspace_bytes(1 << 24, 1, 16, C.byref(v)) == pb.PARD_OK
    assert v.value >= 2 * 8 * (1 << 24)
    dummy = np.zeros(64, np.int64)
    st = pb.QueueStateArrays(2, 1, dummy, dummy, dummy, dummy)
    out = pb.PlanOut()
    hs = (C.c_void_p * 1)(h.handle)
    cst, cout = st.c_struct(), out.c_struct()
    # null pipelines / bad mode / n_ctx = 0 / missing state arrays
    assert lib.pard_plan(None, 1, None, 0, C.byref(cst), 1, 0, C.byref(cout), None, 0, None) == pb.PARD_EINVAL
    assert lib.pard_plan(hs, 1, None, 0, C.byref(cst), 1, 1 << 20, C.byref(cout), None, 0, None) == pb.PARD_EINVAL
    # rules that exclude each other, and the split-budget rule without its arrival records
    assert lib.pard_plan(hs, 1, None, 0, C.byref(cst), 1, 64 | 128, C.byref(cout), None, 0, None) == pb.PARD_EINVAL
    assert lib.pard_plan(hs, 1, None, 5, C.byref(cst), 1, 128, C.byref(cout), None, 0, None) == pb.PARD_EINVAL
    assert lib.pard_plan(hs, 1, None, 0, C.byref(cst), 1, 32 | 1, C.byref(cout), None, 0, None) == pb.PARD_EINVAL
    assert lib.pard_plan(hs, 1, None, 0, C.byref(cst), 0, 0, C.byref(cout), None, 0, None) == pb.PARD_EINVAL
    bad = pb.QueueStateArrays(2, 1, None, dummy, dummy, dummy).c_struct()
    assert lib.pard_plan(hs, 1, None, 0, C.byref(bad), 1, 0, C.byref(cout), None, 0, None) == pb.PARD_EINVAL
    assert lib.pard_plan(hs, 1, None, 5, C.byref(cst), 1, 0, C.byref(cout), None, 0, None) == pb.PARD_EINVAL
    assert lib.pard_goodput(None, None, None, 0, 1, 2, None, None, None) == pb.PARD_EINVAL


def test_estimate_w_argument_checks_happen_before_any_launch():
    p = inputs.make_pipeline(inputs.chain_edges(2), 2, [1, 1], [[5], [5]])
    h = pb.pard_load_pipeline(p, host_only=True)
    lib = pb.library()
    v = C.c_uint64()
    assert lib.pard_estimate_w_workspace_bytes(0, C.byref(v)) == pb.PARD_EINVAL
    assert lib.pard_estimate_w_workspace_bytes(1, None) == pb.PARD_EINVAL
    assert lib.pard_estimate_w_workspace_bytes(3, C.byref(v)) == pb.PARD_OK and v.value >= 256 + 24
    hs = (C.c_void_p * 1)(h.handle)
    buf = np.zeros(64, np.int64)
    a = buf.ctypes.data

    def call(pipes=hs, n_pipes=1, poc=None, n_ctx=1, S=2, R=1, samples=a, M=8, num=1, den=10, mode=0, w=a):
        return lib.pard_estimate_w(pipes, n_pipes, poc, n_ctx, S, R, samples, M, num, den, 0, mode, w, None, 0, None)

    assert call(pipes=None) == pb.PARD_EINVAL
    assert call(samples=None) == pb.PARD_EINVAL
    assert call(w=None) == pb.PARD_EINVAL
    assert call(n_ctx=0) == pb.PARD_EINVAL
    assert call(num=11) == pb.PARD_EINVAL                  # lambda > 1
    assert call(den=0) == pb.PARD_EINVAL
    assert call(mode=pb.PARD_MODE_RAW) == pb.PARD_EINVAL
    assert call(n_pipes=2) == pb.PARD_EINVAL               # several pipelines need the ctx map
    assert call(S=0) == pb.PARD_EINVAL
    assert call(M=0) == pb.PARD_ERANGE
    assert call(M=pb.PARD_MAX_WAIT_SAMPLES + 1) == pb.PARD_ERANGE
    assert call(S=65) == pb.PARD_ERANGE
    assert call(n_ctx=1 << 20, R=1 << 12) == pb.PARD_ERANGE


def test_update_priority_argument_checks_happen_before_any_launch():
    p = inputs.make_pipeline(inputs.chain_edges(2), 2, [1, 1], [[5], [5]])
    h = pb.pard_load_pipeline(p, host_only=True)
    lib = pb.library()
    v = C.c_uint64()
    assert lib.pard_update_priority_workspace_bytes(0, C.byref(v)) == pb.PARD_EINVAL
    assert lib.pard_update_priority_workspace_bytes(1, None) == pb.PARD_EINVAL
    assert lib.pard_update_priority_workspace_bytes(3, C.byref(v)) == pb.PARD_OK and v.value >= 256 + 24
    hs = (C.c_void_p * 1)(h.handle)
    buf = np.zeros(64, np.int64)
    a = buf.ctypes.data

    def call(pipes=hs, n_pipes=1, poc=None, n_ctx=1, S=2, batch=a, workers=None, x=a, H=8, W=4, tau=1000,
             mode=0, prio=a):
        return lib.pard_update_priority(pipes, n_pipes, poc, n_ctx, S, batch, workers, x, H, W, tau, mode, prio,
                                        None, 0, None)

    assert call(pipes=None) == pb.PARD_EINVAL
    assert call(batch=None) == pb.PARD_EINVAL
    assert call(x=None) == pb.PARD_EINVAL
    assert call(prio=None) == pb.PARD_EINVAL
    assert call(n_ctx=0) == pb.PARD_EINVAL
    assert call(S=0) == pb.PARD_EINVAL
    assert call(W=0) == pb.PARD_EINVAL
    assert call(W=9) == pb.PARD_EINVAL                     # window longer than the history
    assert call(tau=0) == pb.PARD_EINVAL
    assert call(mode=pb.PARD_MODE_RAW) == pb.PARD_EINVAL
    assert call(n_pipes=2) == pb.PARD_EINVAL               # several pipelines need the ctx map
    assert call(S=65) == pb.PARD_ERANGE
    assert call(H=pb.PARD_MAX_HISTORY + 1, W=4) == pb.PARD_ERANGE
    assert call(tau=1 << 31) == pb.PARD_ERANGE
    # a host-only handle cannot be used on a device (without a device the CUDA call fails first)
    assert call() in (pb.PARD_EINVAL, pb.PARD_ECUDA)
    h.free()


def test_update_queue_delay_argument_checks_happen_before_any_launch():
    lib = pb.library()
    v = C.c_uint64()
    assert lib.pard_update_queue_delay_workspace_bytes(None) == pb.PARD_EINVAL
    assert lib.pard_update_queue_delay_workspace_bytes(C.byref(v)) == pb.PARD_OK and v.value >= 256
    buf = np.zeros(64, np.int64)
    a = buf.ctypes.data

    def call(n_ctx=1, S=2, now=a, t=a, d=a, M=8, window=1000, mode=0, q=a, ws=None, wsb=0):
        return lib.pard_update_queue_delay(n_ctx, S, now, t, d, M, window, mode, q, ws, wsb, None)

    assert call(n_ctx=0) == pb.PARD_EINVAL
    assert call(S=0) == pb.PARD_EINVAL
    assert call(now=None) == pb.PARD_EINVAL
    assert call(q=None) == pb.PARD_EINVAL
    assert call(t=None) == pb.PARD_EINVAL
    assert call(d=None) == pb.PARD_EINVAL
    assert call(window=0) == pb.PARD_EINVAL
    assert call(mode=pb.PARD_MODE_RAW) == pb.PARD_EINVAL
    assert call(S=65) == pb.PARD_ERANGE
    assert call(M=pb.PARD_MAX_DELAY_SAMPLES + 1) == pb.PARD_ERANGE
    assert call(window=pb.PARD_MAX_DELAY_WINDOW_US + 1) == pb.PARD_ERANGE
    assert call(t=a + 4) == pb.PARD_EINVAL                 # misaligned timestamps
    assert call() == pb.PARD_EINVAL                        # no workspace
    assert call(ws=a + 256 - a % 256, wsb=8) == pb.PARD_EWORKSPACE


def test_advance_state_argument_checks_happen_before_any_launch():
    p = inputs.make_pipeline(inputs.chain_edges(2), 2, [1, 1], [[5], [5]])
    h = pb.pard_load_pipeline(p, host_only=True)
    lib = pb.library()
    v = C.c_uint64()
    assert lib.pard_advance_state_workspace_bytes(0, C.byref(v)) == pb.PARD_EINVAL
    assert lib.pard_advance_state_workspace_bytes(2, C.byref(v)) == pb.PARD_OK and v.value >= 256 + 16
    hs = (C.c_void_p * 1)(h.handle)
    a = np.zeros(64, np.int64).ctypes.data

    def call(pipes=hs, n_pipes=1, poc=None, n_ctx=1, S=2, now=a, batch=a, workers=None, kept=a, fa=a, t=a, d=a,
             M=4, slot=0, mode=0):
        return lib.pard_advance_state(pipes, n_pipes, poc, n_ctx, S, now, batch, workers, kept, fa, t, d, M, slot,
                                      mode, None, 0, None)

    assert call(pipes=None) == pb.PARD_EINVAL
    assert call(now=None) == pb.PARD_EINVAL
    assert call(batch=None) == pb.PARD_EINVAL
    assert call(kept=None) == pb.PARD_EINVAL
    assert call(fa=None) == pb.PARD_EINVAL
    assert call(t=None) == pb.PARD_EINVAL                  # a ring is announced but missing
    assert call(slot=4) == pb.PARD_EINVAL
    assert call(n_ctx=0) == pb.PARD_EINVAL
    assert call(mode=pb.PARD_MODE_SCAN) == pb.PARD_EINVAL
    assert call(n_pipes=2) == pb.PARD_EINVAL
    assert call(S=65) == pb.PARD_ERANGE
    assert call(M=pb.PARD_MAX_DELAY_SAMPLES + 1, slot=0) == pb.PARD_ERANGE
    h.free()
