"""g10_pressure_timeline_static -- the timeline call for hosts that cannot allocate device memory -- must give
exactly what g10_pressure_timeline gives.  Its scratch is one array shared by every call on the device and never
cleared between calls except by the call itself, so the check runs on consecutive calls with different traces:
a stale flag or count left behind by the previous call would show up as a wrong prefix sum or a hang-free
timeout bit in the status word.  (Named to be collected last: a failure here cannot hide another test.)"""
import ctypes as C

import numpy as np
import pytest

from paper_2310_09443_b200 import traces

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    import torch
    assert torch.cuda.is_available(), "this test needs a CUDA device"
    from paper_2310_09443_b200 import binding, build
    build.build()
    binding.load_library()
    return binding


def _same(a, b, K):
    for name in ("kernel_start_ns", "pressure", "peak_bytes", "peak_slot", "status"):
        x, y = getattr(a, name).cpu().numpy(), getattr(b, name).cpu().numpy()
        if name == "pressure":
            x, y = x[:K], y[:K]
        assert np.array_equal(x, y), name      # integer outputs: the tolerance is bit-exact


def _same_as_oracle(got, tr):
    from oracle import g10_oracle as O
    O.build()
    start, P0, peak, slot = O.timeline(tr)
    assert np.array_equal(got.kernel_start_ns.cpu().numpy(), start)
    assert np.array_equal(got.pressure.cpu().numpy()[:tr.K], P0)
    assert int(got.peak_bytes.item()) == peak and int(got.peak_slot.item()) == slot


def test_static_scratch_matches_workspace_variant_on_consecutive_calls(gpu):
    import torch
    seq = [traces.config1_resnet152(), traces.config0_mlp_chain(), traces.config3_vit_huge(), traces.config1_resnet152()]
    for tr in seq:                                  # back-to-back calls, sizes going down and up again
        tb = gpu.upload(tr)
        got = gpu.g10_pressure_timeline_static(tb)
        ref = gpu.g10_pressure_timeline(tb)
        torch.cuda.synchronize()
        assert int(got.status.item()) == 0
        _same(got, ref, tr.K)
        _same_as_oracle(got, tr)                    # and both agree with the CPU oracle, not only with each other
    # twice in a row on the very same inputs, without anything in between
    tb = gpu.upload(seq[0])
    a = gpu.g10_pressure_timeline_static(tb)
    b = gpu.g10_pressure_timeline_static(tb)
    ref = gpu.g10_pressure_timeline(tb)
    torch.cuda.synchronize()
    _same(a, ref, seq[0].K)
    _same(b, ref, seq[0].K)


def test_static_variant_at_its_largest_trace(gpu):
    """Exactly the documented maxima (32 768 kernels, 131 072 tensors): the scratch layout still fits the static
    array and the result is the oracle's."""
    import torch
    tr = traces.config4_stress_dag(K=gpu.STATIC_MAX_KERNELS, N=gpu.STATIC_MAX_TENSORS)
    assert tr.K == gpu.STATIC_MAX_KERNELS and tr.N == gpu.STATIC_MAX_TENSORS
    tb = gpu.upload(tr)
    for _ in range(2):
        got = gpu.g10_pressure_timeline_static(tb)
        torch.cuda.synchronize()
        assert int(got.status.item()) == 0
        _same_as_oracle(got, tr)


def test_static_variant_refuses_what_does_not_fit(gpu):
    lib = gpu.load_library()
    buf = (C.c_int64 * 8)()
    p = C.cast(buf, C.c_void_p)
    out = gpu._TimelineOut(p, p, p, p, p)
    too_many_kernels = gpu._Trace(gpu.STATIC_MAX_KERNELS + 1, 4, 4, p, p, p, p, None, gpu.MEM_DEVICE)
    assert lib.g10_pressure_timeline_static(C.byref(too_many_kernels), C.byref(out), None) == -2
    too_many_tensors = gpu._Trace(4, gpu.STATIC_MAX_TENSORS + 1, 4, p, p, p, p, None, gpu.MEM_DEVICE)
    assert lib.g10_pressure_timeline_static(C.byref(too_many_tensors), C.byref(out), None) == -2
    host_memory = gpu._Trace(4, 4, 4, p, p, p, p, None, gpu.MEM_HOST)
    assert lib.g10_pressure_timeline_static(C.byref(host_memory), C.byref(out), None) == -1
    assert b"limits" in lib.g10_strerror(-2)
