"""ctypes front end of the CPU oracle (g10_oracle.c) -- TEST INFRASTRUCTURE, NOT THE PRODUCT.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this module.
It compiles g10_oracle.c with gcc on first use and exposes the oracle's functions on numpy
arrays.  It imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from types import SimpleNamespace

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "g10_oracle.c")
_LIB = os.path.join(_HERE, "libg10_oracle.so")

MIGRATION_DTYPE = np.dtype([
    ("period", "<i4"), ("tensor", "<i4"), ("dest", "<i4"),
    ("absent_first", "<i4"), ("absent_last", "<i4"), ("iteration", "<i4"),
    ("evict_issue_ns", "<i8"), ("prefetch_issue_ns", "<i8"), ("transfer_ns", "<i8"),
])
assert MIGRATION_DTYPE.itemsize == 48

INSTRUCTION_DTYPE = np.dtype([("opcode", "<i4"), ("tensor", "<i4"), ("target", "<i4"), ("record", "<i4"),
                              ("bytes", "<i8"), ("time_ns", "<i8")])
assert INSTRUCTION_DTYPE.itemsize == 32
OPCODES = {0: "g10_free", 1: "g10_pre_evict", 2: "g10_alloc", 3: "g10_prefetch"}

STATUS = {0: "ALREADY_FITS", 1: "FIT", 2: "EXHAUSTED", 3: "ITERATION_LIMIT"}


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-Wall", "-Wextra", "-shared", "-fPIC", "-o", _LIB, _SRC])
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


def _c(a, dt):
    return np.ascontiguousarray(a, dtype=dt)


def slot_clock(kernel_ns):
    dur = _c(kernel_ns, np.int64)
    start = np.zeros(dur.shape[0] + 1, dtype=np.int64)
    lib().g10o_slot_clock(C.c_int64(dur.shape[0]), _p(dur), _p(start))
    return start


def vitality(kernel_ptr, kernel_tensors, N):
    ptr = _c(kernel_ptr, np.int64)
    kt = _c(kernel_tensors, np.int32)
    K, E = ptr.shape[0] - 1, kt.shape[0]
    first = np.zeros(N, np.int32); last = np.zeros(N, np.int32); nuse = np.zeros(N, np.int32)
    use_ptr = np.zeros(N + 1, np.int64); uses = np.zeros(max(E, 1), np.int32)
    per_ptr = np.zeros(N + 1, np.int64)
    pt = np.zeros(max(E, 1), np.int32); pu = np.zeros(max(E, 1), np.int32); pv = np.zeros(max(E, 1), np.int32)
    counts = np.zeros(2, np.int64)
    rc = lib().g10o_vitality(C.c_int64(K), C.c_int64(N), _p(ptr), _p(kt), _p(first), _p(last), _p(nuse),
                             _p(use_ptr), _p(uses), C.c_int64(E), _p(per_ptr), _p(pt), _p(pu), _p(pv),
                             C.c_int64(E), _p(counts))
    assert rc == 0
    e2, pn = int(counts[0]), int(counts[1])
    return SimpleNamespace(first_use=first, last_use=last, num_uses=nuse, use_ptr=use_ptr, uses=uses[:e2].copy(),
                           period_ptr=per_ptr, period_tensor=pt[:pn].copy(), period_prev_use=pu[:pn].copy(),
                           period_next_use=pv[:pn].copy(), counts=counts)


def pressure(K, tensor_bytes, tensor_global, first_use, last_use):
    tb = _c(tensor_bytes, np.int64)
    tg = _c(tensor_global, np.uint8) if tensor_global is not None else None
    f = _c(first_use, np.int32); l = _c(last_use, np.int32)
    P = np.zeros(K, np.int64)
    peak = C.c_int64(0); slot = C.c_int32(0)
    lib().g10o_pressure(C.c_int64(K), C.c_int64(tb.shape[0]), _p(tb), _p(tg), _p(f), _p(l), _p(P),
                        C.byref(peak), C.byref(slot))
    return P, int(peak.value), int(slot.value)


def geometry(start, tensor_bytes, period_tensor, period_prev_use, period_next_use, host_bw, ssd_bw):
    st = _c(start, np.int64); tb = _c(tensor_bytes, np.int64)
    pt = _c(period_tensor, np.int32); pu = _c(period_prev_use, np.int32); pv = _c(period_next_use, np.int32)
    Pn = pt.shape[0]
    t = np.zeros((2, Pn), np.int64); a = np.zeros((2, Pn), np.int32); b = np.zeros((2, Pn), np.int32)
    lib().g10o_geometry(C.c_int64(st.shape[0] - 1), C.c_int64(Pn), _p(st), _p(tb), _p(pt), _p(pu), _p(pv),
                        C.c_uint64(host_bw), C.c_uint64(ssd_bw), _p(t), _p(a), _p(b))
    return SimpleNamespace(transfer_ns=t, absent_first=a, absent_last=b)


def timeline(trace):
    """start, unplanned pressure, peak, peak slot of a Trace-like object."""
    v = vitality(trace.kernel_ptr, trace.kernel_tensors, trace.N)
    P, peak, slot = pressure(trace.K, trace.tensor_bytes, trace.tensor_global, v.first_use, v.last_use)
    return slot_clock(trace.kernel_ns), P, peak, slot


def plan(trace, gpu_capacity_bytes, host_bw=None, ssd_bw=None, host_capacity_bytes=None, max_iterations=0,
         lazy=False):
    host_bw = trace.host_bw if host_bw is None else host_bw
    ssd_bw = trace.ssd_bw if ssd_bw is None else ssd_bw
    hc = trace.host_capacity_bytes if host_capacity_bytes is None else host_capacity_bytes
    ptr = _c(trace.kernel_ptr, np.int64); kt = _c(trace.kernel_tensors, np.int32)
    tb = _c(trace.tensor_bytes, np.int64); dur = _c(trace.kernel_ns, np.int64)
    tg = _c(trace.tensor_global, np.uint8) if trace.tensor_global is not None else None
    K, N, E = trace.K, trace.N, trace.E
    cap = max(E, 1)
    out = np.zeros(cap, MIGRATION_DTYPE)
    finalP = np.zeros(K, np.int64)
    summary = np.zeros(8, np.int64)
    wb = np.zeros(2 * cap, np.uint64); wc = np.zeros(cap, np.int64)
    rc = lib().g10o_plan(C.c_int64(K), C.c_int64(N), _p(ptr), _p(kt), _p(tb), _p(dur), _p(tg),
                         C.c_uint64(gpu_capacity_bytes), C.c_uint64(host_bw), C.c_uint64(ssd_bw), C.c_uint64(hc),
                         C.c_int64(max_iterations), C.c_int32(1 if lazy else 0),
                         _p(out), C.c_int64(cap), _p(finalP), _p(summary), _p(wb), _p(wc))
    assert rc == 0
    n = int(summary[0])
    ben = [int(wb[2 * j]) | (int(wb[2 * j + 1]) << 64) for j in range(n)]
    return SimpleNamespace(migrations=out[:n].copy(), final_pressure=finalP, summary=summary,
                           status=STATUS[int(summary[2])], win_benefit=ben, win_cost=wc[:n].copy())


def schedule_prefetch(K, migrations, start, tensor_bytes, gpu_capacity_bytes, pressure):
    """Section 4.4 eager prefetch pass over a finished eviction plan.  Returns new pressure and per-record results."""
    mig = np.ascontiguousarray(migrations)
    assert mig.dtype == MIGRATION_DTYPE
    n = mig.shape[0]
    st = _c(start, np.int64); tb = _c(tensor_bytes, np.int64)
    P = _c(pressure, np.int64).copy()
    order = np.zeros(max(n, 1), np.int32); nal = np.zeros(max(n, 1), np.int32); nis = np.zeros(max(n, 1), np.int64)
    summary = np.zeros(4, np.int64)
    lib().g10o_schedule_prefetch(C.c_int64(K), C.c_int64(n), _p(mig), _p(st), _p(tb), C.c_uint64(gpu_capacity_bytes),
                                 _p(P), _p(order), _p(nal), _p(nis), _p(summary))
    return SimpleNamespace(pressure=P, order=order[:n].copy(), new_absent_last=nal[:n].copy(),
                           new_prefetch_issue_ns=nis[:n].copy(), summary=summary)


def emit_instructions(K, first_use, last_use, tensor_bytes, tensor_global, start, migrations, new_issue_ns=None):
    """Section 4.4 code instrumentation: the alloc / free / pre-evict / prefetch stream by kernel boundary."""
    f = _c(first_use, np.int32); l = _c(last_use, np.int32); tb = _c(tensor_bytes, np.int64)
    tg = _c(tensor_global, np.uint8) if tensor_global is not None else None
    st = _c(start, np.int64); mig = np.ascontiguousarray(migrations)
    ni = _c(new_issue_ns, np.int64) if new_issue_ns is not None else None
    N, n = f.shape[0], mig.shape[0]
    cap = 2 * N + 2 * n + 1
    out = np.zeros(cap, INSTRUCTION_DTYPE)
    ptr = np.zeros(K + 2, np.int64)
    lib().g10o_emit_instructions.restype = C.c_int64
    m = lib().g10o_emit_instructions(C.c_int64(K), C.c_int64(N), _p(f), _p(l), _p(tb), _p(tg), _p(st), C.c_int64(n), _p(mig),
                                     _p(ni), _p(ptr), _p(out), C.c_int64(cap))
    return SimpleNamespace(inst_ptr=ptr, instructions=out[:int(m)].copy())


def characterize(K, vit, tensor_bytes, start, host_bw, ssd_bw):
    """Section 3 statistics (Figures 2-4) of a trace from its vitality results."""
    up = _c(vit.use_ptr, np.int64); us = _c(vit.uses, np.int32); tb = _c(tensor_bytes, np.int64); st = _c(start, np.int64)
    pt = _c(vit.period_tensor, np.int32); pu = _c(vit.period_prev_use, np.int32); pv = _c(vit.period_next_use, np.int32)
    active = np.zeros(K, np.int64); lh = np.zeros(64, np.int64); slh = np.zeros(41 * 45, np.int64)
    hide = np.zeros(2, np.int64); summary = np.zeros(2, np.int64)
    lib().g10o_characterize(C.c_int64(K), C.c_int64(tb.shape[0]), _p(up), _p(us), _p(tb), _p(st), C.c_int64(pt.shape[0]),
                            _p(pt), _p(pu), _p(pv), C.c_uint64(host_bw), C.c_uint64(ssd_bw), _p(active), _p(lh), _p(slh),
                            _p(hide), _p(summary))
    return SimpleNamespace(active_bytes=active, len_hist=lh, size_len_hist=slh.reshape(41, 45), hide=hide, summary=summary)


def plan_batch(trace, variants, max_iterations=0, lazy=True):
    """Re-planning under changed conditions (Section 5's sensitivity studies seen from the planner): every variant is a
    whole plan of the same trace with its own kernel durations (profiling error), bandwidths, capacities.  A variant is
    a dict with any of kernel_ns, gpu_capacity_bytes, host_bw, ssd_bw, host_capacity_bytes; gpu_capacity_bytes is
    required.  Plan stability of variant v against variant 0 is reported as the pair (|M_v & M_0|, |M_v | M_0|) over
    the sets of migrated periods (their quotient is the Jaccard index)."""
    import copy
    plans, stability = [], []
    base = None
    for v in variants:
        tr = copy.copy(trace)
        if v.get("kernel_ns") is not None:
            tr.kernel_ns = _c(v["kernel_ns"], np.int64)
        r = plan(tr, int(v["gpu_capacity_bytes"]), host_bw=v.get("host_bw"), ssd_bw=v.get("ssd_bw"),
                 host_capacity_bytes=v.get("host_capacity_bytes", 0), max_iterations=max_iterations, lazy=lazy)
        mine = set(int(p) for p in r.migrations["period"])
        if base is None:
            base = mine
        stability.append((len(mine & base), len(mine | base)))
        plans.append(r)
    return SimpleNamespace(plans=plans, stability=np.asarray(stability, dtype=np.int64).reshape(-1, 2))


def plan_cyclic(trace, gpu_capacity_bytes, host_bw=None, ssd_bw=None, host_capacity_bytes=None, max_iterations=0):
    """Steady-state planning on the cyclic timeline (wrap-around periods of global tensors; plain tier)."""
    host_bw = trace.host_bw if host_bw is None else host_bw
    ssd_bw = trace.ssd_bw if ssd_bw is None else ssd_bw
    hc = trace.host_capacity_bytes if host_capacity_bytes is None else host_capacity_bytes
    ptr = _c(trace.kernel_ptr, np.int64); kt = _c(trace.kernel_tensors, np.int32)
    tb = _c(trace.tensor_bytes, np.int64); dur = _c(trace.kernel_ns, np.int64)
    tg = _c(trace.tensor_global, np.uint8) if trace.tensor_global is not None else None
    K, N, E = trace.K, trace.N, trace.E
    cap = max(E + N, 1)
    out = np.zeros(cap, MIGRATION_DTYPE)
    finalP = np.zeros(K, np.int64)
    summary = np.zeros(8, np.int64)
    periods = np.zeros(3 * cap, np.int32)
    npd = C.c_int64(0)
    rc = lib().g10o_plan_cyclic(C.c_int64(K), C.c_int64(N), _p(ptr), _p(kt), _p(tb), _p(dur), _p(tg),
                                C.c_uint64(gpu_capacity_bytes), C.c_uint64(host_bw), C.c_uint64(ssd_bw), C.c_uint64(hc),
                                C.c_int64(max_iterations), _p(out), C.c_int64(cap), _p(finalP), _p(summary), _p(periods),
                                C.byref(npd))
    assert rc == 0
    n = int(summary[0])
    return SimpleNamespace(migrations=out[:n].copy(), final_pressure=finalP, summary=summary, status=STATUS[int(summary[2])],
                           periods=periods[:3 * npd.value].reshape(-1, 3).copy())
