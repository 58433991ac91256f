"""Thin ctypes binding of the C ABI in include/g10.h: argument marshalling only.

Every step of the path runs in the CUDA library; PyTorch is used for device / pinned memory and
streams.  There is no CPU fallback: if libg10.so is missing or no CUDA device is present the calls
raise.
"""
from __future__ import annotations

import ctypes as C
import os
from types import SimpleNamespace

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libg10.so")

MEM_DEVICE, MEM_HOST = 0, 1
WS_VITALITY, WS_TIMELINE, WS_PLAN, WS_GEOMETRY, WS_EMIT, WS_BATCH, WS_PREFETCH, WS_ANALYSIS = 0, 1, 2, 3, 4, 5, 6, 7
DEST_SSD, DEST_HOST = 0, 1
FLAG_RESCORE_ALL = 1
FLAG_GLOBAL_STATE = 2
FLAG_MULTI_BLOCK = 4
STATUS = {0: "ALREADY_FITS", 1: "FIT", 2: "EXHAUSTED", 3: "ITERATION_LIMIT"}
EXPORTS = ("g10_vitality", "g10_pressure_timeline", "g10_candidate_geometry", "g10_plan_migrations",
           "g10_workspace_bytes", "g10_strerror", "g10_version", "g10_pressure_timeline_static", "g10_schedule_prefetch", "g10_emit_instructions", "g10_characterize", "g10_plan_batch", "g10_plan_cyclic", "g10_launch_count")
STATIC_MAX_KERNELS, STATIC_MAX_TENSORS = 32768, 131072

INSTRUCTION_DTYPE = np.dtype([("opcode", "<i4"), ("tensor", "<i4"), ("target", "<i4"), ("record", "<i4"),
                              ("bytes", "<i8"), ("time_ns", "<i8")])
OPCODES = {0: "g10_free", 1: "g10_pre_evict", 2: "g10_alloc", 3: "g10_prefetch"}

MIGRATION_DTYPE = np.dtype([
    ("period", "<i4"), ("tensor", "<i4"), ("dest", "<i4"),
    ("absent_first", "<i4"), ("absent_last", "<i4"), ("iteration", "<i4"),
    ("evict_issue_ns", "<i8"), ("prefetch_issue_ns", "<i8"), ("transfer_ns", "<i8"),
])


class _Trace(C.Structure):
    _fields_ = [("num_kernels", C.c_int64), ("num_tensors", C.c_int64), ("num_events", C.c_int64),
                ("kernel_ptr", C.c_void_p), ("kernel_tensors", C.c_void_p), ("tensor_bytes", C.c_void_p),
                ("kernel_ns", C.c_void_p), ("tensor_global", C.c_void_p), ("mem", C.c_int32)]


class _TimelineOut(C.Structure):
    _fields_ = [("kernel_start_ns", C.c_void_p), ("pressure", C.c_void_p), ("peak_bytes", C.c_void_p),
                ("peak_slot", C.c_void_p), ("status", C.c_void_p), ("first_use", C.c_void_p), ("last_use", C.c_void_p)]


class _VitalityOut(C.Structure):
    _fields_ = [("first_use", C.c_void_p), ("last_use", C.c_void_p), ("num_uses", C.c_void_p),
                ("use_ptr", C.c_void_p), ("uses", C.c_void_p), ("uses_cap", C.c_int64),
                ("period_ptr", C.c_void_p), ("period_tensor", C.c_void_p), ("period_prev_use", C.c_void_p),
                ("period_next_use", C.c_void_p), ("periods_cap", C.c_int64), ("counts", C.c_void_p),
                ("timeline", C.POINTER(_TimelineOut))]


class _GeometryOut(C.Structure):
    _fields_ = [("transfer_ns", C.c_void_p), ("absent_first", C.c_void_p), ("absent_last", C.c_void_p)]


class _PlanOut(C.Structure):
    _fields_ = [("migrations", C.c_void_p), ("migrations_cap", C.c_int64), ("final_pressure", C.c_void_p),
                ("summary", C.c_void_p)]


class _Variant(C.Structure):
    _fields_ = [("kernel_ns", C.c_void_p), ("gpu_capacity_bytes", C.c_uint64), ("host_bw", C.c_uint64), ("ssd_bw", C.c_uint64),
                ("host_capacity_bytes", C.c_uint64)]


class _BatchOut(C.Structure):
    _fields_ = [("migrations", C.c_void_p), ("migrations_cap", C.c_int64), ("final_pressure", C.c_void_p),
                ("summary", C.c_void_p), ("stability", C.c_void_p)]


class _PrefetchOut(C.Structure):
    _fields_ = [("pressure", C.c_void_p), ("order", C.c_void_p), ("new_absent_last", C.c_void_p),
                ("new_prefetch_issue_ns", C.c_void_p), ("summary", C.c_void_p)]


class _StatsOut(C.Structure):
    _fields_ = [("active_bytes", C.c_void_p), ("len_hist", C.c_void_p), ("size_len_hist", C.c_void_p), ("hide", C.c_void_p),
                ("summary", C.c_void_p)]


class _EmitOut(C.Structure):
    _fields_ = [("inst_ptr", C.c_void_p), ("instructions", C.c_void_p), ("instructions_cap", C.c_int64), ("counts", C.c_void_p)]


class _Options(C.Structure):
    _fields_ = [("host_capacity_bytes", C.c_uint64), ("max_iterations", C.c_int64), ("flags", C.c_uint32),
                ("stage_events", C.POINTER(C.c_void_p)), ("num_stage_events", C.c_int32)]


_lib = None


def load_library():
    """Loads libg10.so.  Raises if it has not been built: there is no other implementation to fall back to."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libg10.so not found at %s: run `python -m paper_2310_09443_b200.build`" % LIB_PATH)
        lib = C.CDLL(LIB_PATH)
        lib.g10_strerror.restype = C.c_char_p
        lib.g10_strerror.argtypes = [C.c_int32]
        lib.g10_version.restype = C.c_int32
        lib.g10_launch_count.restype = C.c_uint64
        lib.g10_launch_count.argtypes = []
        lib.g10_workspace_bytes.restype = C.c_int32
        lib.g10_workspace_bytes.argtypes = [C.c_int32, C.c_int64, C.c_int64, C.c_int64, C.c_int32, C.POINTER(C.c_size_t)]
        lib.g10_vitality.restype = C.c_int32
        lib.g10_vitality.argtypes = [C.POINTER(_Trace), C.POINTER(_VitalityOut), C.c_void_p, C.c_size_t, C.c_void_p]
        lib.g10_pressure_timeline.restype = C.c_int32
        lib.g10_pressure_timeline.argtypes = [C.POINTER(_Trace), C.POINTER(_TimelineOut), C.c_void_p, C.c_size_t, C.c_void_p]
        lib.g10_pressure_timeline_static.restype = C.c_int32
        lib.g10_pressure_timeline_static.argtypes = [C.POINTER(_Trace), C.POINTER(_TimelineOut), C.c_void_p]
        lib.g10_candidate_geometry.restype = C.c_int32
        lib.g10_candidate_geometry.argtypes = [C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                               C.c_uint64, C.c_uint64, C.POINTER(_GeometryOut), C.c_void_p]
        lib.g10_schedule_prefetch.restype = C.c_int32
        lib.g10_schedule_prefetch.argtypes = [C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64,
                                              C.POINTER(_PrefetchOut), C.c_void_p, C.c_size_t, C.c_void_p]
        lib.g10_emit_instructions.restype = C.c_int32
        lib.g10_emit_instructions.argtypes = [C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                              C.c_int64, C.c_void_p, C.c_void_p, C.POINTER(_EmitOut), C.c_void_p, C.c_size_t,
                                              C.c_void_p]
        lib.g10_characterize.restype = C.c_int32
        lib.g10_characterize.argtypes = [C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p,
                                         C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint64, C.POINTER(_StatsOut), C.c_void_p]
        lib.g10_plan_cyclic.restype = C.c_int32
        lib.g10_plan_cyclic.argtypes = [C.POINTER(_Trace), C.c_uint64, C.c_uint64, C.c_uint64, C.POINTER(_Options),
                                        C.POINTER(_PlanOut), C.c_void_p, C.c_size_t, C.c_void_p]
        lib.g10_plan_batch.restype = C.c_int32
        lib.g10_plan_batch.argtypes = [C.POINTER(_Trace), C.c_int32, C.POINTER(_Variant), C.c_int64, C.POINTER(_BatchOut),
                                       C.c_void_p, C.c_size_t, C.c_void_p]
        lib.g10_plan_migrations.restype = C.c_int32
        lib.g10_plan_migrations.argtypes = [C.POINTER(_Trace), C.c_uint64, C.c_uint64, C.c_uint64, C.POINTER(_Options),
                                            C.POINTER(_PlanOut), C.c_void_p, C.c_size_t, C.c_void_p]
        _lib = lib
    return _lib


class G10Error(RuntimeError):
    pass


def _check(rc):
    if rc != 0:
        raise G10Error("g10 error %d: %s" % (rc, load_library().g10_strerror(rc).decode()))


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


class TraceBuffers:
    """The five trace arrays as torch tensors, either all on one CUDA device or all in pinned host memory."""

    def __init__(self, kernel_ptr, kernel_tensors, tensor_bytes, kernel_ns, tensor_global, K=None, N=None, E=None):
        self.kernel_ptr, self.kernel_tensors, self.tensor_bytes = kernel_ptr, kernel_tensors, tensor_bytes
        self.kernel_ns, self.tensor_global = kernel_ns, tensor_global
        # explicit sizes let an empty array be backed by a one-element buffer (torch gives empty tensors no address)
        self.K = int(kernel_ns.shape[0]) if K is None else K
        self.N = int(tensor_bytes.shape[0]) if N is None else N
        self.E = int(kernel_tensors.shape[0]) if E is None else E
        self.mem = MEM_DEVICE if kernel_ptr.is_cuda else MEM_HOST
        assert kernel_ptr.dtype == torch.int64 and kernel_tensors.dtype == torch.int32
        assert tensor_bytes.dtype == torch.int64 and kernel_ns.dtype == torch.int64
        assert tensor_global is None or tensor_global.dtype == torch.uint8

    def c_struct(self):
        return _Trace(self.K, self.N, self.E, _ptr(self.kernel_ptr), _ptr(self.kernel_tensors), _ptr(self.tensor_bytes),
                      _ptr(self.kernel_ns), _ptr(self.tensor_global), self.mem)

    def nbytes(self):
        return sum(t.numel() * t.element_size() for t in (self.kernel_ptr, self.kernel_tensors, self.tensor_bytes,
                                                          self.kernel_ns, self.tensor_global) if t is not None)


def _nonempty(a):
    a = np.ascontiguousarray(a)
    return a if a.size else np.zeros(1, dtype=a.dtype)


def upload(trace, device="cuda:0") -> TraceBuffers:
    """Trace (numpy) -> device-resident TraceBuffers."""
    f = lambda a: torch.from_numpy(_nonempty(a)).to(device)
    return TraceBuffers(f(trace.kernel_ptr), f(trace.kernel_tensors), f(trace.tensor_bytes), f(trace.kernel_ns),
                        f(trace.tensor_global) if trace.tensor_global is not None else None, trace.K, trace.N, trace.E)


def pin(trace) -> TraceBuffers:
    """Trace (numpy) -> TraceBuffers in pinned host memory (for the host-pointer form of the calls)."""
    f = lambda a: torch.from_numpy(_nonempty(a)).pin_memory()
    return TraceBuffers(f(trace.kernel_ptr), f(trace.kernel_tensors), f(trace.tensor_bytes), f(trace.kernel_ns),
                        f(trace.tensor_global) if trace.tensor_global is not None else None, trace.K, trace.N, trace.E)


def g10_launch_count() -> int:
    """Kernels the library has launched in this process so far."""
    return int(load_library().g10_launch_count())


def g10_workspace_bytes(which, K, N, E, mem=MEM_DEVICE) -> int:
    out = C.c_size_t(0)
    _check(load_library().g10_workspace_bytes(which, K, N, E, mem, C.byref(out)))
    return int(out.value)


def _device_of(tb, device):
    if tb.mem == MEM_DEVICE:
        return tb.kernel_ptr.device
    return torch.device(device if device is not None else "cuda:0")


def _workspace(tb, which, ws, device):
    need = g10_workspace_bytes(which, tb.K, tb.N, tb.E, tb.mem)
    if ws is None:
        ws = torch.empty(max(need, 256), dtype=torch.uint8, device=_device_of(tb, device))
    return ws, ws.numel()


def _alloc(tb, shape, dtype, device):
    shape = max(int(shape), 1)
    if tb.mem == MEM_DEVICE:
        return torch.empty(shape, dtype=dtype, device=tb.kernel_ptr.device)
    return torch.empty(shape, dtype=dtype).pin_memory()


def g10_vitality(tb: TraceBuffers, ws=None, stream=None, device=None, uses_cap=None, periods_cap=None, out=None, timeline=False):
    """Section 4.2 tensor vitality analysis.  Returns tensors in the memory space of `tb`; in device mode the
    call is asynchronous on `stream` (trim `uses` / the period arrays with counts after synchronising).
    `out`: the result of an earlier call on a trace of the same sizes, to write into instead of allocating.
    timeline=True (device traces): the same call also produces the Section 4.3 pressure timeline, returned as
    `.timeline` (the fields of g10_pressure_timeline); pass an earlier such result as `timeline` to write into it."""
    lib = load_library()
    ucap = tb.E if uses_cap is None else uses_cap
    pcap = tb.E if periods_cap is None else periods_cap
    r = out if out is not None else SimpleNamespace(
        first_use=_alloc(tb, tb.N, torch.int32, device), last_use=_alloc(tb, tb.N, torch.int32, device),
        num_uses=_alloc(tb, tb.N, torch.int32, device), use_ptr=_alloc(tb, tb.N + 1, torch.int64, device),
        uses=_alloc(tb, max(ucap, 1), torch.int32, device), period_ptr=_alloc(tb, tb.N + 1, torch.int64, device),
        period_tensor=_alloc(tb, max(pcap, 1), torch.int32, device), period_prev_use=_alloc(tb, max(pcap, 1), torch.int32, device),
        period_next_use=_alloc(tb, max(pcap, 1), torch.int32, device), counts=_alloc(tb, 3, torch.int64, device))
    to = None
    if timeline:
        t = timeline if not isinstance(timeline, bool) else SimpleNamespace(
            kernel_start_ns=_alloc(tb, tb.K + 1, torch.int64, device), pressure=_alloc(tb, max(tb.K, 1), torch.int64, device),
            peak_bytes=_alloc(tb, 1, torch.int64, device), peak_slot=_alloc(tb, 1, torch.int32, device),
            status=_alloc(tb, 1, torch.int64, device))
        to = _TimelineOut(_ptr(t.kernel_start_ns), _ptr(t.pressure), _ptr(t.peak_bytes), _ptr(t.peak_slot), _ptr(t.status), None, None)
        r.timeline = t
    ws, ws_bytes = _workspace(tb, WS_ANALYSIS if timeline else WS_VITALITY, ws, device)
    vo = _VitalityOut(_ptr(r.first_use), _ptr(r.last_use), _ptr(r.num_uses), _ptr(r.use_ptr), _ptr(r.uses), ucap,
                       _ptr(r.period_ptr), _ptr(r.period_tensor), _ptr(r.period_prev_use), _ptr(r.period_next_use), pcap,
                       _ptr(r.counts), C.pointer(to) if to is not None else None)
    tr = tb.c_struct()
    _check(lib.g10_vitality(C.byref(tr), C.byref(vo), _ptr(ws), ws_bytes, _stream(stream)))
    r.workspace = ws
    return r


def g10_pressure_timeline(tb: TraceBuffers, ws=None, stream=None, device=None, out=None, first_last=None):
    """Section 4.3 memory-pressure timeline before any migration.  `out`: an earlier result to write into.
    first_last: (first_use, last_use) device tensors of an earlier g10_vitality call on the same trace; with them the
    call does not derive first / last use from the trace again."""
    lib = load_library()
    r = out if out is not None else SimpleNamespace(
        kernel_start_ns=_alloc(tb, tb.K + 1, torch.int64, device), pressure=_alloc(tb, max(tb.K, 1), torch.int64, device),
        peak_bytes=_alloc(tb, 1, torch.int64, device), peak_slot=_alloc(tb, 1, torch.int32, device),
        status=_alloc(tb, 1, torch.int64, device))
    ws, ws_bytes = _workspace(tb, WS_TIMELINE, ws, device)
    to = _TimelineOut(_ptr(r.kernel_start_ns), _ptr(r.pressure), _ptr(r.peak_bytes), _ptr(r.peak_slot), _ptr(r.status),
                      _ptr(first_last[0]) if first_last is not None else None, _ptr(first_last[1]) if first_last is not None else None)
    tr = tb.c_struct()
    _check(lib.g10_pressure_timeline(C.byref(tr), C.byref(to), _ptr(ws), ws_bytes, _stream(stream)))
    r.workspace = ws
    return r


def g10_pressure_timeline_static(tb: TraceBuffers, stream=None):
    """g10_pressure_timeline for callers that cannot allocate: no workspace argument, the scratch is a fixed
    array inside the library (traces up to STATIC_MAX_KERNELS kernels / STATIC_MAX_TENSORS tensors, device
    memory only).  Calls on one device share that array, so do not let two of them overlap on the GPU.  The
    output tensors are still the caller's; this wrapper creates them with torch for convenience."""
    lib = load_library()
    dev = tb.kernel_ptr.device
    r = SimpleNamespace(
        kernel_start_ns=torch.empty(tb.K + 1, dtype=torch.int64, device=dev),
        pressure=torch.empty(max(tb.K, 1), dtype=torch.int64, device=dev),
        peak_bytes=torch.empty(1, dtype=torch.int64, device=dev), peak_slot=torch.empty(1, dtype=torch.int32, device=dev),
        status=torch.empty(1, dtype=torch.int64, device=dev))
    out = _TimelineOut(_ptr(r.kernel_start_ns), _ptr(r.pressure), _ptr(r.peak_bytes), _ptr(r.peak_slot), _ptr(r.status))
    tr = tb.c_struct()
    _check(lib.g10_pressure_timeline_static(C.byref(tr), C.byref(out), _stream(stream)))
    return r


def g10_candidate_geometry(K, kernel_start_ns, tensor_bytes, period_tensor, period_prev_use, period_next_use,
                           host_bw, ssd_bw, stream=None):
    """Transfer time and absent-slot range of every period for SSD (row 0) and host (row 1).  Device tensors only."""
    lib = load_library()
    Pn = int(period_tensor.shape[0])
    dev = kernel_start_ns.device
    r = SimpleNamespace(transfer_ns=torch.empty((2, Pn), dtype=torch.int64, device=dev),
                        absent_first=torch.empty((2, Pn), dtype=torch.int32, device=dev),
                        absent_last=torch.empty((2, Pn), dtype=torch.int32, device=dev))
    out = _GeometryOut(_ptr(r.transfer_ns), _ptr(r.absent_first), _ptr(r.absent_last))
    _check(lib.g10_candidate_geometry(K, Pn, _ptr(kernel_start_ns), _ptr(tensor_bytes), _ptr(period_tensor),
                                      _ptr(period_prev_use), _ptr(period_next_use), host_bw, ssd_bw, C.byref(out),
                                      _stream(stream)))
    return r


def g10_plan_migrations(tb: TraceBuffers, gpu_capacity_bytes, host_bw, ssd_bw, host_capacity_bytes=0, max_iterations=0,
                        flags=0, ws=None, stream=None, device=None, migrations_cap=None, out=None, stage_events=None):
    """Algorithm 1: the eviction plan.  `migrations` is a uint8 tensor of 48-byte records (see MIGRATION_DTYPE);
    use `migrations_numpy` after synchronising.  stage_events: up to five torch.cuda.Event objects (already
    recorded once, so that they own a handle) that the library records at its stage boundaries."""
    lib = load_library()
    mcap = tb.E if migrations_cap is None else migrations_cap
    if out is None:
        out = SimpleNamespace(migrations=_alloc(tb, max(mcap, 1) * 48, torch.uint8, device),
                              final_pressure=_alloc(tb, max(tb.K, 1), torch.int64, device),
                              summary=_alloc(tb, 8, torch.int64, device))
    ws, ws_bytes = _workspace(tb, WS_PLAN, ws, device)
    po = _PlanOut(_ptr(out.migrations), mcap, _ptr(out.final_pressure), _ptr(out.summary))
    opt = _Options(host_capacity_bytes, max_iterations, flags, None, 0)
    if stage_events:
        handles = (C.c_void_p * len(stage_events))(*[C.c_void_p(e.cuda_event) for e in stage_events])
        opt.stage_events = C.cast(handles, C.POINTER(C.c_void_p))
        opt.num_stage_events = len(stage_events)
    tr = tb.c_struct()
    _check(lib.g10_plan_migrations(C.byref(tr), gpu_capacity_bytes, host_bw, ssd_bw, C.byref(opt), C.byref(po), _ptr(ws),
                                   ws_bytes, _stream(stream)))
    out.workspace = ws
    return out


def g10_plan_cyclic(tb: TraceBuffers, gpu_capacity_bytes, host_bw, ssd_bw, host_capacity_bytes=0, max_iterations=0, ws=None,
                    stream=None, migrations_cap=None, device=None):
    """Steady-state plan on the cyclic timeline (wrap-around periods of global tensors).  Records as in
    g10_plan_migrations with unrolled slots and times; results in the memory space of `tb`."""
    lib = load_library()
    mcap = tb.E if migrations_cap is None else migrations_cap
    out = SimpleNamespace(migrations=_alloc(tb, max(mcap, 1) * 48, torch.uint8, device),
                          final_pressure=_alloc(tb, max(tb.K, 1), torch.int64, device),
                          summary=_alloc(tb, 8, torch.int64, device))
    ws, ws_bytes = _workspace(tb, WS_PLAN, ws, device)
    po = _PlanOut(_ptr(out.migrations), mcap, _ptr(out.final_pressure), _ptr(out.summary))
    opt = _Options(host_capacity_bytes, max_iterations, 0, None, 0)
    tr = tb.c_struct()
    _check(lib.g10_plan_cyclic(C.byref(tr), gpu_capacity_bytes, host_bw, ssd_bw, C.byref(opt), C.byref(po), _ptr(ws), ws_bytes,
                               _stream(stream)))
    out.workspace = ws
    return out


def g10_plan_batch(tb: TraceBuffers, variants, max_iterations=0, migrations_cap=None, ws=None, stream=None):
    """Plans the device-resident trace under every variant at once (one thread block each).  A variant is a dict with
    gpu_capacity_bytes, host_bw, ssd_bw and optionally kernel_ns (int64 device tensor [K]) and host_capacity_bytes.
    Returns migrations [V, migrations_cap * 48] (uint8), final_pressure [V, K], summary [V, 8], stability [V, 2]."""
    lib = load_library()
    V = len(variants)
    dev = tb.kernel_ptr.device
    mcap = tb.E if migrations_cap is None else migrations_cap
    out = SimpleNamespace(migrations=torch.empty((max(V, 1), max(mcap, 1) * 48), dtype=torch.uint8, device=dev),
                          final_pressure=torch.empty((max(V, 1), max(tb.K, 1)), dtype=torch.int64, device=dev),
                          summary=torch.empty((max(V, 1), 8), dtype=torch.int64, device=dev),
                          stability=torch.empty((max(V, 1), 2), dtype=torch.int64, device=dev), migrations_cap=mcap)
    arr = (_Variant * max(V, 1))()
    keep = []
    for j, v in enumerate(variants):
        kn = v.get("kernel_ns")
        if kn is not None:
            assert kn.dtype == torch.int64 and kn.is_contiguous() and kn.numel() >= tb.K
            keep.append(kn)
        arr[j] = _Variant(_ptr(kn) if kn is not None else None, int(v["gpu_capacity_bytes"]), int(v["host_bw"]), int(v["ssd_bw"]),
                          int(v.get("host_capacity_bytes", 0)))
    ws, ws_bytes = _workspace(tb, WS_BATCH, ws, None)
    bo = _BatchOut(_ptr(out.migrations), mcap, _ptr(out.final_pressure), _ptr(out.summary), _ptr(out.stability))
    tr = tb.c_struct()
    _check(lib.g10_plan_batch(C.byref(tr), V, arr, max_iterations, C.byref(bo), _ptr(ws), ws_bytes, _stream(stream)))
    out.workspace = ws
    out.keep = keep
    return out


def batch_migrations_numpy(batch, v) -> np.ndarray:
    """Committed migration records of variant v of a finished batch (synchronises)."""
    n = min(int(batch.summary[v, 0].item()), batch.migrations_cap)
    return batch.migrations[v, : n * 48].cpu().numpy().view(MIGRATION_DTYPE).copy()


def g10_schedule_prefetch(K, num_migrations, migrations, kernel_start_ns, tensor_bytes, gpu_capacity_bytes, pressure,
                          ws=None, one_block=False, stream=None):
    """Section 4.4 eager prefetch pass.  `migrations` is the uint8 record tensor of a finished plan, `pressure` its
    final pressure (updated in place).  Device tensors only.  `ws`: a uint8 device tensor of at least
    g10_workspace_bytes(WS_PREFETCH, K, 0, n) bytes (allocated here when None); one_block=True calls without a
    workspace, which makes one thread block do the whole pass.  summary[4] is the device status word."""
    lib = load_library()
    dev = kernel_start_ns.device
    n = int(num_migrations)
    r = SimpleNamespace(pressure=pressure, order=torch.empty(max(n, 1), dtype=torch.int32, device=dev),
                        new_absent_last=torch.empty(max(n, 1), dtype=torch.int32, device=dev),
                        new_prefetch_issue_ns=torch.empty(max(n, 1), dtype=torch.int64, device=dev),
                        summary=torch.empty(5, dtype=torch.int64, device=dev))
    out = _PrefetchOut(_ptr(r.pressure), _ptr(r.order), _ptr(r.new_absent_last), _ptr(r.new_prefetch_issue_ns), _ptr(r.summary))
    ws_ptr, ws_bytes = None, 0
    if not one_block:
        need = g10_workspace_bytes(WS_PREFETCH, K, 0, n)
        if ws is None:
            ws = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
        ws_ptr, ws_bytes = _ptr(ws), ws.numel()
        r.ws = ws
    _check(lib.g10_schedule_prefetch(K, n, _ptr(migrations), _ptr(kernel_start_ns), _ptr(tensor_bytes), gpu_capacity_bytes,
                                     C.byref(out), ws_ptr, ws_bytes, _stream(stream)))
    return r


def g10_emit_instructions(K, N, first_use, last_use, tensor_bytes, tensor_global, kernel_start_ns, num_migrations, migrations,
                          new_prefetch_issue_ns=None, ws=None, stream=None):
    """Section 4.4 code instrumentation: the alloc / free / pre-evict / prefetch stream by kernel boundary (device tensors).
    `instructions` is a uint8 tensor of 32-byte records (INSTRUCTION_DTYPE); counts = [number of instructions, status]."""
    lib = load_library()
    dev = kernel_start_ns.device
    n = int(num_migrations)
    cap = 2 * N + 2 * n
    r = SimpleNamespace(inst_ptr=torch.empty(K + 2, dtype=torch.int64, device=dev),
                        instructions=torch.empty(max(cap, 1) * 32, dtype=torch.uint8, device=dev),
                        counts=torch.empty(2, dtype=torch.int64, device=dev))
    need = g10_workspace_bytes(WS_EMIT, K, N, n)
    if ws is None:
        ws = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
    out = _EmitOut(_ptr(r.inst_ptr), _ptr(r.instructions), cap, _ptr(r.counts))
    _check(lib.g10_emit_instructions(K, N, _ptr(first_use), _ptr(last_use), _ptr(tensor_bytes), _ptr(tensor_global),
                                     _ptr(kernel_start_ns), n, _ptr(migrations), _ptr(new_prefetch_issue_ns), C.byref(out),
                                     _ptr(ws), ws.numel(), _stream(stream)))
    r.workspace = ws
    return r


def g10_characterize(K, N, use_ptr, uses, tensor_bytes, kernel_start_ns, num_periods, period_tensor, period_prev_use,
                     period_next_use, host_bw, ssd_bw, stream=None):
    """Section 3 statistics (Figures 2-4) from the vitality results and the slot clock (device tensors)."""
    lib = load_library()
    dev = kernel_start_ns.device
    r = SimpleNamespace(active_bytes=torch.empty(max(K, 1), dtype=torch.int64, device=dev),
                        len_hist=torch.empty(64, dtype=torch.int64, device=dev),
                        size_len_hist=torch.empty(41 * 45, dtype=torch.int64, device=dev),
                        hide=torch.empty(2, dtype=torch.int64, device=dev), summary=torch.empty(2, dtype=torch.int64, device=dev))
    out = _StatsOut(_ptr(r.active_bytes), _ptr(r.len_hist), _ptr(r.size_len_hist), _ptr(r.hide), _ptr(r.summary))
    _check(lib.g10_characterize(K, N, _ptr(use_ptr), _ptr(uses), _ptr(tensor_bytes), _ptr(kernel_start_ns), int(num_periods),
                                _ptr(period_tensor), _ptr(period_prev_use), _ptr(period_next_use), host_bw, ssd_bw, C.byref(out),
                                _stream(stream)))
    return r


def instructions_numpy(em) -> np.ndarray:
    n = int(em.counts[0].item())
    return em.instructions[: n * 32].cpu().numpy().view(INSTRUCTION_DTYPE).copy()


def migrations_numpy(plan) -> np.ndarray:
    """Committed migration records of a finished plan as a numpy structured array (synchronises)."""
    summary = plan.summary.cpu().numpy()
    n = int(summary[0])
    raw = plan.migrations[: n * 48].cpu().numpy()
    return raw.view(MIGRATION_DTYPE).copy()
