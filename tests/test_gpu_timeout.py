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


def test_a_prefetch_hand_over_that_never_comes(oracle):
    """The many-block form of the eager prefetch pass: blocks wait for records handed over by the block on their right.  In
    the test build one block (named by an environment variable that only that build reads) keeps its records to itself
    and waits last a millisecond: the blocks that wait for it give up, the others stop as soon as they see the status
    word, summary[4] carries G10_DEV_TIMEOUT, and the same call without the injection matches the oracle."""
    import os
    import torch
    from paper_2310_09443_b200 import binding, build
    from test_gpu_parity import synthetic_prefetch_records
    build.build()
    binding.load_library()
    hooks = C.CDLL(build.build(hooks=True))
    hooks.g10_schedule_prefetch.restype = C.c_int32
    hooks.g10_schedule_prefetch.argtypes = [C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64,
                                            C.POINTER(binding._PrefetchOut), C.c_void_p, C.c_size_t, C.c_void_p]
    rng = np.random.default_rng(77)
    K, n, cap = 40000, 6000, 1 << 22
    mig, start, nbytes, P = synthetic_prefetch_records(binding, rng, K, n, wrap=False)
    ref = oracle.schedule_prefetch(K, mig, start, nbytes, cap, P)
    dm = torch.from_numpy(mig.view(np.uint8).copy()).cuda()
    dstart, dbytes = torch.from_numpy(start).cuda(), torch.from_numpy(nbytes).cuda()
    ws = torch.zeros(binding.g10_workspace_bytes(binding.WS_PREFETCH, K, 0, n), dtype=torch.uint8, device="cuda")
    order = torch.zeros(n, dtype=torch.int32, device="cuda")
    new_last = torch.zeros(n, dtype=torch.int32, device="cuda")
    new_issue = torch.zeros(n, dtype=torch.int64, device="cuda")
    summary = torch.zeros(5, dtype=torch.int64, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream

    def call():
        dP = torch.from_numpy(P.copy()).cuda()
        out = binding._PrefetchOut(dP.data_ptr(), order.data_ptr(), new_last.data_ptr(), new_issue.data_ptr(), summary.data_ptr())
        t0 = time.perf_counter()
        rc = hooks.g10_schedule_prefetch(K, n, dm.data_ptr(), dstart.data_ptr(), dbytes.data_ptr(), cap, C.byref(out), ws.data_ptr(),
                                         ws.numel(), stream)
        torch.cuda.synchronize()
        return rc, time.perf_counter() - t0, dP

    def check_against_oracle(dP):
        s = summary.cpu().numpy()
        assert s[4] == 0 and np.array_equal(s[:4], ref.summary)
        assert np.array_equal(order.cpu().numpy(), ref.order) and np.array_equal(new_last.cpu().numpy(), ref.new_absent_last)
        assert np.array_equal(new_issue.cpu().numpy(), ref.new_prefetch_issue_ns) and np.array_equal(dP.cpu().numpy(), ref.pressure)

    os.environ.pop("G10_TEST_PREFETCH_MUTE_BLOCK", None)
    rc, _, dP = call()
    assert rc == 0
    check_against_oracle(dP)
    os.environ["G10_TEST_PREFETCH_MUTE_BLOCK"] = "100"
    try:
        rc, dt, dP = call()
    finally:
        os.environ.pop("G10_TEST_PREFETCH_MUTE_BLOCK", None)
    assert rc == 0
    assert int(summary[4].item()) & DEV_TIMEOUT, "summary[4] must carry G10_DEV_TIMEOUT"
    assert dt < 1.0, "the call must come back within milliseconds (%.3f s)" % dt
    rc, _, dP = call()
    assert rc == 0
    check_against_oracle(dP)
