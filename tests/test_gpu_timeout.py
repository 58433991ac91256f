"""The give-up path of the bounded device waits.  Every wait in the kernels has a limit (polls or nanoseconds) after which
the kernel sets G10_DEV_TIMEOUT and returns; in normal runs no wait ever gets there.  This test makes one run out, in
the allowed form: a test build of the library (-DG10_TEST_HOOKS, libg10_hooks.so, never loaded by the binding) in which
one block of the planner's cooperative grid does not arrive at the grid barrier and waits last a millisecond.  The other
blocks give up, the call returns with the timeout bit, the outputs stay in bounds, the context stays usable and the
next (ordinary) call gives the right plan.  Nothing traps, faults or spins on."""
import ctypes as C
import time

import numpy as np
import pytest

from paper_2310_09443_b200 import traces

pytestmark = pytest.mark.gpu

FLAG_RESCORE_ALL = 0x1                 # the cooperative multi-block planner (two grid barriers per iteration)
FLAG_TEST_SKIP_ARRIVAL = 0x40000000    # honoured by the test build only
DEV_TIMEOUT = 0x80


def test_a_wait_that_runs_out_returns_with_the_timeout_bit(oracle):
    import torch
    assert torch.cuda.is_available(), "this test needs a CUDA device"
    from paper_2310_09443_b200 import binding, build
    build.build()
    binding.load_library()
    hooks = C.CDLL(build.build(hooks=True))
    hooks.g10_plan_migrations.restype = C.c_int32
    hooks.g10_plan_migrations.argtypes = [C.POINTER(binding._Trace), C.c_uint64, C.c_uint64, C.c_uint64, C.POINTER(binding._Options),
                                          C.POINTER(binding._PlanOut), C.c_void_p, C.c_size_t, C.c_void_p]
    tr = traces.config0_mlp_chain()
    tb = binding.upload(tr)
    start, P0, peak, slot = oracle.timeline(tr)
    cap = tr.capacity_from_peak(peak)
    ref = oracle.plan(tr, cap)
    ws = torch.zeros(binding.g10_workspace_bytes(binding.WS_PLAN, tb.K, tb.N, tb.E), dtype=torch.uint8, device="cuda")
    mig = torch.zeros(max(tb.E, 1) * 48, dtype=torch.uint8, device="cuda")
    finalp = torch.zeros(tb.K, dtype=torch.int64, device="cuda")
    summary = torch.zeros(8, dtype=torch.int64, device="cuda")
    po = binding._PlanOut(mig.data_ptr(), tb.E, finalp.data_ptr(), summary.data_ptr())
    ctr = tb.c_struct()
    stream = torch.cuda.current_stream().cuda_stream

    def call(flags):
        opt = binding._Options(0, 0, flags, None, 0)
        t0 = time.perf_counter()
        rc = hooks.g10_plan_migrations(C.byref(ctr), cap, tr.host_bw, tr.ssd_bw, C.byref(opt), C.byref(po), ws.data_ptr(), ws.numel(), stream)
        torch.cuda.synchronize()
        return rc, time.perf_counter() - t0

    # 1. the test build plans correctly when nothing is injected
    rc, _ = call(FLAG_RESCORE_ALL)
    assert rc == 0
    s = summary.cpu().numpy()
    assert s[7] == 0 and np.array_equal(s[:7], ref.summary[:7])
    # 2. one block never arrives: the others' waits run out after a millisecond each
    rc, dt = call(FLAG_RESCORE_ALL | FLAG_TEST_SKIP_ARRIVAL)
    assert rc == 0
    s = summary.cpu().numpy()
    assert s[7] & DEV_TIMEOUT, "the status word must carry G10_DEV_TIMEOUT"
    assert dt < 1.0, "the call must come back within milliseconds, not after the seconds of the production limit (%.3f s)" % dt
    n = int(s[0])
    assert 0 <= n <= tb.E                                   # whatever was written is in bounds
    # 3. the context is intact: the same call without the injection gives the oracle's plan again, and so does the product library
    rc, _ = call(FLAG_RESCORE_ALL)
    assert rc == 0
    s = summary.cpu().numpy()
    assert s[7] == 0 and np.array_equal(s[:7], ref.summary[:7])
    got = mig[:int(s[0]) * 48].cpu().numpy().view(binding.MIGRATION_DTYPE)
    assert np.array_equal(got, ref.migrations) and np.array_equal(finalp.cpu().numpy(), ref.final_pressure)
    plan = binding.g10_plan_migrations(tb, cap, tr.host_bw, tr.ssd_bw, flags=FLAG_RESCORE_ALL)
    torch.cuda.synchronize()
    assert int(plan.summary[7].item()) == 0 and np.array_equal(binding.migrations_numpy(plan), ref.migrations)
