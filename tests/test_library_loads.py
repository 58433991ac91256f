"""CPU-side checks of the CUDA library: it loads, exports every symbol the header declares, and its
host-side argument validation answers before anything is launched (no compute calls here)."""
import ctypes as C
import os
import re

import pytest

from paper_2310_09443_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def test_exports_match_header(lib):
    header = open(os.path.join(ROOT, "include", "g10.h")).read()
    declared = set(re.findall(r"\b(g10_[a-z_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name
    assert lib.g10_version() == 1
    assert lib.g10_strerror(-3).decode().startswith("workspace")


def test_workspace_bytes_and_limits(lib):
    a = binding.g10_workspace_bytes(binding.WS_PLAN, 96, 130, 320)
    b = binding.g10_workspace_bytes(binding.WS_PLAN, 1000, 2000, 5000)
    h = binding.g10_workspace_bytes(binding.WS_PLAN, 1000, 2000, 5000, binding.MEM_HOST)
    assert 0 < a < b < h and a % 256 == 0
    assert binding.g10_workspace_bytes(binding.WS_GEOMETRY, 10, 10, 10) == 0
    out = C.c_size_t(0)
    assert lib.g10_workspace_bytes(2, -1, 0, 0, 0, C.byref(out)) == -1
    assert lib.g10_workspace_bytes(2, 1 << 31, 0, 0, 0, C.byref(out)) == -2
    assert lib.g10_workspace_bytes(9, 1, 1, 1, 0, C.byref(out)) == -1


def test_argument_errors_before_any_launch(lib):
    tr = binding._Trace(4, 4, 4, None, None, None, None, None, 0)
    vo = binding._VitalityOut()
    assert lib.g10_vitality(C.byref(tr), C.byref(vo), None, 0, None) == -1        # NULL kernel_ptr
    assert lib.g10_vitality(None, C.byref(vo), None, 0, None) == -1
    tr2 = binding._Trace(-1, 4, 4, None, None, None, None, None, 0)
    assert lib.g10_pressure_timeline(C.byref(tr2), None, None, 0, None) == -1
    tr3 = binding._Trace(1 << 31, 4, 4, None, None, None, None, None, 0)
    assert lib.g10_vitality(C.byref(tr3), C.byref(vo), None, 0, None) == -2
    po = binding._PlanOut()
    buf = (C.c_int64 * 8)()
    tr4 = binding._Trace(0, 0, 0, C.cast(buf, C.c_void_p), None, None, None, None, 0)
    assert lib.g10_plan_migrations(C.byref(tr4), 1, 0, 1, None, C.byref(po), None, 0, None) == -1      # zero bandwidth
    po.summary = C.cast(buf, C.c_void_p)
    assert lib.g10_plan_migrations(C.byref(tr4), 1, 1, 1, None, C.byref(po), None, 0, None) == -3      # no workspace
    go = binding._GeometryOut()
    assert lib.g10_candidate_geometry(1, 1, None, None, None, None, None, 1, 1, C.byref(go), None) == -1


def test_argument_errors_of_the_later_entry_points(lib):
    buf = (C.c_int64 * 8)()
    ptr = C.cast(buf, C.c_void_p)
    # statistics: zero bandwidth, missing outputs, oversize
    so = binding._StatsOut()
    assert lib.g10_characterize(1, 1, None, None, None, None, 0, None, None, None, 0, 1, C.byref(so), None) == -1
    assert lib.g10_characterize(1, 1, ptr, ptr, ptr, ptr, 0, None, None, None, 1, 1, C.byref(so), None) == -1
    assert lib.g10_characterize(1 << 31, 1, ptr, ptr, ptr, ptr, 0, None, None, None, 1, 1, C.byref(so), None) == -2
    # batch: host traces refused, variant count, zero bandwidth, workspace
    bo = binding._BatchOut()
    bo.summary = ptr; bo.stability = ptr
    var = (binding._Variant * 1)(binding._Variant(None, 1, 1, 1, 0))
    tr_host = binding._Trace(0, 0, 0, ptr, None, None, None, None, binding.MEM_HOST)
    assert lib.g10_plan_batch(C.byref(tr_host), 1, var, 0, C.byref(bo), None, 0, None) == -1
    tr_dev = binding._Trace(0, 0, 0, ptr, None, None, None, None, binding.MEM_DEVICE)
    assert lib.g10_plan_batch(C.byref(tr_dev), 0, var, 0, C.byref(bo), None, 0, None) == -2
    assert lib.g10_plan_batch(C.byref(tr_dev), 2000, var, 0, C.byref(bo), None, 0, None) == -2
    bad = (binding._Variant * 1)(binding._Variant(None, 1, 0, 1, 0))
    assert lib.g10_plan_batch(C.byref(tr_dev), 1, bad, 0, C.byref(bo), None, 0, None) == -1
    assert lib.g10_plan_batch(C.byref(tr_dev), 1, var, -1, C.byref(bo), None, 0, None) == -1
    assert lib.g10_plan_batch(C.byref(tr_dev), 1, var, 0, C.byref(bo), None, 0, None) == -3
    # prefetch pass and instruction stream
    pf = binding._PrefetchOut()
    assert lib.g10_schedule_prefetch(1, 1, None, None, None, 1, C.byref(pf), None, 0, None) == -1
    assert binding.g10_workspace_bytes(binding.WS_PREFETCH, 1000000, 0, 13505) < (1 << 20)        # a few words per record
    eo = binding._EmitOut()
    assert lib.g10_emit_instructions(1, 1, None, None, None, None, None, 0, None, None, C.byref(eo), None, 0, None) == -1
    # the workspace of the batch call is the planner's
    plan_ws = binding.g10_workspace_bytes(binding.WS_PLAN, 96, 130, 320)
    assert binding.g10_workspace_bytes(binding.WS_BATCH, 96, 130, 320) >= plan_ws       # the planner's, plus the variant table
    # the analysis calls ask only for what they use
    big = (1_000_000, 4_000_000, 5_000_000)
    assert binding.g10_workspace_bytes(binding.WS_TIMELINE, *big) < 64 << 20
    assert binding.g10_workspace_bytes(binding.WS_VITALITY, *big) < 128 << 20
    assert binding.g10_workspace_bytes(binding.WS_PLAN, *big) > binding.g10_workspace_bytes(binding.WS_VITALITY, *big)
