"""Parity of the CUDA path with the CPU oracle, element by element, through the C ABI."""
import numpy as np
import pytest

import helpers
from paper_2310_09443_b200 import traces

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    import torch
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from paper_2310_09443_b200 import binding, build
    build.build()
    binding.load_library()
    return binding


def _np(t):
    return t.cpu().numpy()


def check_vitality(gpu, oracle, tr, tb):
    import torch
    v = gpu.g10_vitality(tb)
    torch.cuda.synchronize()
    ov = oracle.vitality(tr.kernel_ptr, tr.kernel_tensors, tr.N)
    counts = _np(v.counts)
    assert counts[2] == 0, "device status %x" % counts[2]
    assert counts[0] == len(ov.uses) and counts[1] == len(ov.period_tensor)
    N = tr.N
    assert np.array_equal(_np(v.first_use)[:N], ov.first_use) and np.array_equal(_np(v.last_use)[:N], ov.last_use)
    assert np.array_equal(_np(v.num_uses)[:N], ov.num_uses)
    assert np.array_equal(_np(v.use_ptr)[:N + 1], ov.use_ptr) and np.array_equal(_np(v.period_ptr)[:N + 1], ov.period_ptr)
    e2, pn = int(counts[0]), int(counts[1])
    assert np.array_equal(_np(v.uses)[:e2], ov.uses)
    assert np.array_equal(_np(v.period_tensor)[:pn], ov.period_tensor)
    assert np.array_equal(_np(v.period_prev_use)[:pn], ov.period_prev_use)
    assert np.array_equal(_np(v.period_next_use)[:pn], ov.period_next_use)
    return v, ov


def check_timeline(gpu, oracle, tr, tb):
    import torch
    tl = gpu.g10_pressure_timeline(tb)
    torch.cuda.synchronize()
    start, P0, peak, slot = oracle.timeline(tr)
    assert int(tl.status.item()) == 0
    assert np.array_equal(_np(tl.kernel_start_ns)[:tr.K + 1], start)
    assert np.array_equal(_np(tl.pressure)[:tr.K], P0)
    assert int(tl.peak_bytes.item()) == peak and int(tl.peak_slot.item()) == slot
    # the same call with first / last use handed over from the vitality call
    v = gpu.g10_vitality(tb)
    tg = gpu.g10_pressure_timeline(tb, first_last=(v.first_use, v.last_use))
    torch.cuda.synchronize()
    assert int(tg.status.item()) == 0
    assert np.array_equal(_np(tg.kernel_start_ns)[:tr.K + 1], start) and np.array_equal(_np(tg.pressure)[:tr.K], P0)
    assert int(tg.peak_bytes.item()) == peak and int(tg.peak_slot.item()) == slot
    # ... and both analyses from one call (the vitality kernels book the sizes on their way)
    vf = gpu.g10_vitality(tb, timeline=True)
    torch.cuda.synchronize()
    tf = vf.timeline
    assert int(tf.status.item()) == 0 and _np(vf.counts).tolist() == _np(v.counts).tolist()
    for name, cnt in (("first_use", tr.N), ("last_use", tr.N), ("num_uses", tr.N), ("use_ptr", tr.N + 1), ("period_ptr", tr.N + 1)):
        assert np.array_equal(_np(getattr(vf, name))[:cnt], _np(getattr(v, name))[:cnt]), name
    nu, npd = int(_np(v.counts)[0]), int(_np(v.counts)[1])
    assert np.array_equal(_np(vf.uses)[:nu], _np(v.uses)[:nu])
    for name in ("period_tensor", "period_prev_use", "period_next_use"):
        assert np.array_equal(_np(getattr(vf, name))[:npd], _np(getattr(v, name))[:npd]), name
    assert np.array_equal(_np(tf.kernel_start_ns)[:tr.K + 1], start) and np.array_equal(_np(tf.pressure)[:tr.K], P0)
    assert int(tf.peak_bytes.item()) == peak and int(tf.peak_slot.item()) == slot
    return tl, (start, P0, peak, slot)


def check_geometry(gpu, oracle, tr, tb, v, ov, tl):
    import torch
    pn = len(ov.period_tensor)
    g = gpu.g10_candidate_geometry(tr.K, tl.kernel_start_ns, tb.tensor_bytes, v.period_tensor[:pn].contiguous(),
                                   v.period_prev_use[:pn].contiguous(), v.period_next_use[:pn].contiguous(),
                                   tr.host_bw, tr.ssd_bw)
    torch.cuda.synchronize()
    if pn == 0:
        return
    og = oracle.geometry(_np(tl.kernel_start_ns)[:tr.K + 1], tr.tensor_bytes, ov.period_tensor, ov.period_prev_use,
                         ov.period_next_use, tr.host_bw, tr.ssd_bw)
    assert np.array_equal(_np(g.transfer_ns), og.transfer_ns)
    assert np.array_equal(_np(g.absent_first), og.absent_first) and np.array_equal(_np(g.absent_last), og.absent_last)


def check_plan(gpu, tr, tb, cap, ref, host_capacity=0, max_iterations=0, flags=0):
    import torch
    plan = gpu.g10_plan_migrations(tb, cap, tr.host_bw, tr.ssd_bw, host_capacity_bytes=host_capacity,
                                   max_iterations=max_iterations, flags=flags)
    torch.cuda.synchronize()
    summary = _np(plan.summary)
    assert summary[7] == 0, "device status %x" % summary[7]
    assert np.array_equal(summary[:7], ref.summary[:7]), (summary, ref.summary)
    assert np.array_equal(gpu.migrations_numpy(plan), ref.migrations)
    assert np.array_equal(_np(plan.final_pressure)[:tr.K], ref.final_pressure)
    return plan


def full_parity(gpu, oracle, tr, lazy_oracle=False, repeats=1, **plan_kw):
    tb = gpu.upload(tr)
    v, ov = check_vitality(gpu, oracle, tr, tb)
    tl, (start, P0, peak, slot) = check_timeline(gpu, oracle, tr, tb)
    check_geometry(gpu, oracle, tr, tb, v, ov, tl)
    cap = tr.capacity_from_peak(int(tl.peak_bytes.item()))
    also = plan_kw.pop("also_rescore_all", True)
    ref = oracle.plan(tr, tr.capacity_from_peak(peak), lazy=lazy_oracle,
                      host_capacity_bytes=plan_kw.get("host_capacity", 0), max_iterations=plan_kw.get("max_iterations", 0))
    for _ in range(repeats):
        check_plan(gpu, tr, tb, cap, ref, **plan_kw)
    if also:
        check_plan(gpu, tr, tb, cap, ref, flags=gpu.FLAG_RESCORE_ALL, **plan_kw)      # Algorithm 1 as printed
        check_plan(gpu, tr, tb, cap, ref, flags=gpu.FLAG_GLOBAL_STATE, **plan_kw)     # the large-trace planner
        check_plan(gpu, tr, tb, cap, ref, flags=gpu.FLAG_MULTI_BLOCK, **plan_kw)      # never the single-block planner
    return ref


def test_hand_worked_examples(gpu, oracle):
    import json, os
    ex_all = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "hand_worked_examples.json")))["examples"]
    for name, ex in ex_all.items():
        tr = traces.from_lists(name, ex["kernel_lists"], ex["tensor_bytes"], ex["kernel_ns"], host_bw=ex["host_bw"],
                               ssd_bw=ex["ssd_bw"], capacity_bytes=ex["capacity"])
        ref = full_parity(gpu, oracle, tr)
        assert ref.status == ex["status"] and ref.final_pressure.tolist() == ex["final_pressure"]


def test_random_toy_traces(gpu, oracle):
    """Empty kernels, repeats inside a kernel, unused tensors, globals; several capacities and a finite host memory."""
    rng = np.random.default_rng(777)
    for trial in range(60):
        K = int(rng.integers(1, 40)); N = int(rng.integers(1, 30))
        tr = traces.random_toy(rng, K, N, max_deg=5)
        tr.capacity_frac = [(1, 2), (1, 5), (0, 1), (9, 10)][trial % 4]
        hc = int(rng.integers(0, 3)) * int(rng.integers(1, 80))
        full_parity(gpu, oracle, tr, host_capacity=hc)


@pytest.mark.parametrize("cfg", [0, 1, 2, 3])
def test_configs_bit_exact(gpu, oracle, cfg):
    """Configs 0-3 at full size: every output of the three calls equals the oracle's; plan repeated 3 times."""
    tr = traces.make_config(cfg)
    ref = full_parity(gpu, oracle, tr, lazy_oracle=(cfg == 3), repeats=3)
    assert len(ref.migrations) > 10


def test_bandwidth_and_capacity_sweep(gpu, oracle):
    """The planner-side half of the paper's sensitivity studies (SSD bandwidth, host memory): configs 1 and 2 with
    SSD bandwidths from one SSD to sixteen times the default, a sixteen times faster host link, two GPU capacities
    and a finite host memory.  Faster links make more periods usable and the greedy loop longer."""
    import dataclasses
    GiB = 1 << 30
    n = 0
    for cfg, caps in ((1, (12, 16)), (2, (20,))):
        base = traces.make_config(cfg)
        for ssd in (3_200_000_000, 12_800_000_000, 102_400_000_000):
            for host in (32_000_000_000, 512_000_000_000):
                for capg in caps:
                    for hc in (0, 8 * GiB):
                        tr = dataclasses.replace(base, ssd_bw=ssd, host_bw=host, capacity_bytes=capg * GiB)
                        ref = full_parity(gpu, oracle, tr, lazy_oracle=True, host_capacity=hc, also_rescore_all=(n % 9 == 0))
                        assert len(ref.migrations) > 300
                        n += 1


def test_wide_kernels(gpu, oracle):
    """Kernels that list hundreds or thousands of tensors (an optimizer step over everything): more events in one
    kernel than a warp row, and more in one partition tile than its staging area holds."""
    rng = np.random.default_rng(99)
    N = 15000
    lists = []
    for k in range(48):
        if k in (3, 40):
            lists.append(list(range(N)) if k == 3 else list(range(0, N, 2)))      # 15 000 and 7 500 tensors
        elif k in (7, 8):
            lists.append(rng.integers(0, N, size=300 if k == 7 else 65).tolist()) # repeats inside the list allowed
        else:
            lists.append(rng.integers(0, N, size=int(rng.integers(0, 6))).tolist())
    tr = traces.from_lists("wide", lists, rng.integers(1, 1 << 20, size=N).tolist(), rng.integers(1000, 50000, size=48).tolist(),
                           capacity_frac=(1, 2))
    ref = full_parity(gpu, oracle, tr)
    assert len(ref.migrations) > 0


def _csr_trace(name, rng, K, N, degrees):
    """A trace from per-kernel degrees (tensor ids uniform, repeats allowed), sizes and durations random."""
    ptr = np.zeros(K + 1, dtype=np.int64)
    ptr[1:] = np.cumsum(degrees)
    E = int(ptr[-1])
    return traces.Trace(name=name, kernel_ptr=ptr, kernel_tensors=rng.integers(0, N, size=E).astype(np.int32),
                        tensor_bytes=rng.integers(1, 1 << 24, size=N).astype(np.int64),
                        kernel_ns=rng.integers(1, 100000, size=K).astype(np.int64),
                        tensor_global=(rng.random(N) < 0.01).astype(np.uint8), capacity_frac=(1, 2))


@pytest.mark.parametrize("shape", ["one_event_per_kernel", "mostly_empty_kernels", "few_tensors_many_uses", "every_kernel_wide", "many_tensors",
                                   "odd_narrow_buckets", "odd_wide_buckets"])
def test_pass_shapes(gpu, oracle, shape):
    """Vitality and timeline on traces whose shape drives the partition differently: the widest and the narrowest tiles,
    empty kernels, buckets that overflow shared memory, kernels all wider than a warp row, thousands of buckets, and bucket
    widths that are no powers of two (more buckets than the last kernel has blocks: 113 and 2534 tensors per bucket on a
    148-SM part), with many and with few events per tensor."""
    rng = np.random.default_rng(1000 + len(shape))
    if shape == "one_event_per_kernel":
        K, N = 200_000, 50_000
        tr = _csr_trace(shape, rng, K, N, np.ones(K, dtype=np.int64))
    elif shape == "mostly_empty_kernels":
        K, N = 100_000, 30_000
        tr = _csr_trace(shape, rng, K, N, (rng.random(K) < 0.1) * rng.integers(1, 12, size=K))
    elif shape == "few_tensors_many_uses":
        K, N = 20_000, 300
        tr = _csr_trace(shape, rng, K, N, rng.integers(0, 11, size=K))
    elif shape == "every_kernel_wide":
        K, N = 600, 40_000
        tr = _csr_trace(shape, rng, K, N, rng.integers(65, 400, size=K))
    elif shape == "odd_narrow_buckets":
        K, N = 60_000, 100_000
        tr = _csr_trace(shape, rng, K, N, rng.integers(30, 70, size=K))
    elif shape == "odd_wide_buckets":
        K, N = 250_000, 1_500_000
        tr = _csr_trace(shape, rng, K, N, rng.integers(4, 12, size=K))
    else:
        K, N = 50_000, 3_000_000
        tr = _csr_trace(shape, rng, K, N, rng.integers(0, 9, size=K))
    tb = gpu.upload(tr)
    check_vitality(gpu, oracle, tr, tb)
    check_timeline(gpu, oracle, tr, tb)


def test_more_tensors_than_one_pass_of_buckets(gpu, oracle):
    """Vitality on 18 M tensors: more than the 4096 buckets of 4096 tensors one pass of the bucketed formulation takes, so
    the events are walked twice, the second time for the tensors from 16 777 216 on, with the first pass's totals
    carried over.  Events concentrate around the pass boundary (a third of them within 3000 ids of it)."""
    rng = np.random.default_rng(16777216)
    K, N = 400_000, 18_000_000
    deg = rng.integers(0, 9, size=K)
    tr = _csr_trace("two_passes", rng, K, N, deg)
    near = rng.random(tr.E) < 0.33
    tr.kernel_tensors[near] = (16_777_216 + rng.integers(-3000, 3000, size=int(near.sum()))).astype(np.int32)
    tb = gpu.upload(tr)
    check_vitality(gpu, oracle, tr, tb)


def test_inplace_relu_variant(gpu, oracle):
    tr = traces.config1_resnet152(inplace_relu=True)
    full_parity(gpu, oracle, tr)


def test_scaled_stress_dag(gpu, oracle):
    """Several scan tiles and a ragged tail: K = 20 000, N = 80 000 (plain oracle still feasible)."""
    tr = traces.config4_stress_dag(K=20000, N=80000)
    ref = full_parity(gpu, oracle, tr, lazy_oracle=True)
    assert len(ref.migrations) > 1000


def test_iteration_limit_and_host_capacity(gpu, oracle):
    tr = traces.config0_mlp_chain()
    full_parity(gpu, oracle, tr, max_iterations=5)
    full_parity(gpu, oracle, tr, host_capacity=200 << 20)
    tr.capacity_frac = (1, 1)
    ref = full_parity(gpu, oracle, tr)
    assert ref.status == "ALREADY_FITS"
    tr.capacity_frac = None; tr.capacity_bytes = 1 << 63
    full_parity(gpu, oracle, tr)
    tr.capacity_bytes = 0
    full_parity(gpu, oracle, tr)


def test_heavy_tensors(gpu, oracle):
    """Tensors used by very many kernels take the block-wide sort (shared-memory and global-memory variants)."""
    rng = np.random.default_rng(5)
    K, N = 30000, 50
    lists = []
    for k in range(K):
        lst = [int(x) for x in rng.integers(4, N, size=int(rng.integers(0, 3)))]
        if k % 2 == 0: lst.append(0)                 # 15 000 uses: sorted in global memory
        if k % 7 == 0: lst += [1, 1]                 # 4 286 uses, each listed twice: shared-memory sort + repeats
        if k % 400 == 0: lst.append(2)               # 75 uses with long periods
        if rng.random() < 0.002: lst.append(3)
        lists.append(lst)
    size = rng.integers(1 << 10, 1 << 24, size=N)
    dur = rng.integers(1000, 100000, size=K)
    tr = traces.from_lists("heavy", lists, size, dur, (rng.random(N) < 0.2).astype(np.uint8), capacity_frac=(1, 2))
    tb = gpu.upload(tr)
    v, ov = check_vitality(gpu, oracle, tr, tb)
    tl, _ = check_timeline(gpu, oracle, tr, tb)
    check_geometry(gpu, oracle, tr, tb, v, ov, tl)


def test_empty_and_degenerate(gpu, oracle):
    for lists, nb in (([], []), ([[], []], []), ([[], [], []], [5, 7]), ([[0], [0], [0]], [9]), ([[0, 0, 0]], [3])):
        tr = traces.from_lists("e", lists, nb, [3] * len(lists), capacity_bytes=0)
        full_parity(gpu, oracle, tr)


def test_output_capacity_is_reported(gpu):
    import torch
    tr = traces.config0_mlp_chain()
    tb = gpu.upload(tr)
    v = gpu.g10_vitality(tb, uses_cap=10, periods_cap=5)
    torch.cuda.synchronize()
    c = _np(v.counts)
    assert c[0] == 320 and c[1] == 93 and (c[2] & 0x10) and (c[2] & 0x20)
    plan = gpu.g10_plan_migrations(tb, 1 << 20, tr.host_bw, tr.ssd_bw, migrations_cap=3)
    torch.cuda.synchronize()
    s = _np(plan.summary)
    assert s[0] > 3 and (s[7] & 0x40)


def test_bad_trace_sets_status_bits(gpu):
    import torch
    tr = traces.config0_mlp_chain()
    tr.kernel_tensors = tr.kernel_tensors.copy(); tr.kernel_tensors[7] = 1000
    tr.kernel_ns = tr.kernel_ns.copy(); tr.kernel_ns[3] = 0
    tr.tensor_bytes = tr.tensor_bytes.copy(); tr.tensor_bytes[5] = 0
    tb = gpu.upload(tr)
    v = gpu.g10_vitality(tb)
    tl = gpu.g10_pressure_timeline(tb)
    torch.cuda.synchronize()
    assert _np(v.counts)[2] & 0x1
    st = int(tl.status.item())
    assert (st & 0x1) and (st & 0x8) and (st & 0x4)
    vf = gpu.g10_vitality(tb, timeline=True)                 # both analyses from one call: the same bits in both status words
    torch.cuda.synchronize()
    for word in (int(vf.timeline.status.item()), int(_np(vf.counts)[2])):
        assert (word & 0x1) and (word & 0x8) and (word & 0x4)
    assert np.array_equal(_np(vf.timeline.pressure), _np(tl.pressure)) and np.array_equal(_np(vf.first_use), _np(v.first_use))
    # first / last use handed over but wrong (last before first, last beyond the trace): flagged, skipped, in bounds
    good = traces.config0_mlp_chain()
    tbg = gpu.upload(good)
    vg = gpu.g10_vitality(tbg)
    torch.cuda.synchronize()
    first, last = vg.first_use.clone(), vg.last_use.clone()
    last[3] = first[3] - 1 if int(first[3]) > 0 else -5
    last[9] = good.K + 7
    tg = gpu.g10_pressure_timeline(tbg, first_last=(first, last))
    ok = gpu.g10_pressure_timeline(tbg)
    torch.cuda.synchronize()
    assert int(tg.status.item()) == 0x200 and int(ok.status.item()) == 0
    assert int(tg.peak_bytes.item()) <= int(ok.peak_bytes.item())


def test_bad_kernel_ptr_is_flagged(gpu):
    """A kernel_ptr that is not a monotone map onto [0, E]: both calls finish, stay in bounds and say so."""
    import torch
    base = traces.config0_mlp_chain()
    for kind in ("swapped", "beyond", "short"):
        tr = traces.config0_mlp_chain()
        ptr = base.kernel_ptr.copy()
        if kind == "swapped":
            ptr[10], ptr[20] = base.kernel_ptr[20], base.kernel_ptr[10]
        elif kind == "beyond":
            ptr[50:60] = base.E + 1000
        else:
            ptr[-1] = base.E - 7
        tr.kernel_ptr = ptr
        tb = gpu.upload(tr)
        v = gpu.g10_vitality(tb)
        tl = gpu.g10_pressure_timeline(tb)
        torch.cuda.synchronize()
        assert _np(v.counts)[2] & 0x2, kind
        assert int(tl.status.item()) & 0x2, kind
        assert _np(v.counts)[0] == 0 and (_np(v.num_uses) == 0).all()       # nothing is partitioned


def test_host_pointer_mode(gpu, oracle):
    """The same calls with every array in (pinned) host memory: the library stages the copies itself."""
    tr = traces.config1_resnet152()
    tb = gpu.pin(tr)
    v = gpu.g10_vitality(tb)
    ov = oracle.vitality(tr.kernel_ptr, tr.kernel_tensors, tr.N)
    pn = int(v.counts[1])
    assert int(v.counts[2]) == 0 and pn == len(ov.period_tensor)
    e2 = int(v.counts[0])
    assert e2 == len(ov.uses)
    for name, n in (("first_use", None), ("last_use", None), ("num_uses", None), ("use_ptr", None), ("period_ptr", None),
                    ("uses", e2), ("period_tensor", pn), ("period_prev_use", pn), ("period_next_use", pn)):
        assert np.array_equal(getattr(v, name).numpy()[:n], getattr(ov, name)), name
    tl = gpu.g10_pressure_timeline(tb)
    start, P0, peak, slot = oracle.timeline(tr)
    assert np.array_equal(tl.pressure.numpy(), P0) and int(tl.peak_bytes) == peak and int(tl.peak_slot) == slot
    assert np.array_equal(tl.kernel_start_ns.numpy(), start)
    vf = gpu.g10_vitality(tb, timeline=True)                 # both analyses from one call: the trace is staged once
    assert int(vf.counts[2]) == 0 and int(vf.timeline.status) == 0
    for name, n in (("first_use", None), ("last_use", None), ("num_uses", None), ("use_ptr", None), ("period_ptr", None),
                    ("uses", e2), ("period_tensor", pn), ("period_prev_use", pn), ("period_next_use", pn)):
        assert np.array_equal(getattr(vf, name).numpy()[:n], getattr(ov, name)), name
    assert np.array_equal(vf.timeline.pressure.numpy(), P0) and int(vf.timeline.peak_bytes) == peak and int(vf.timeline.peak_slot) == slot
    assert np.array_equal(vf.timeline.kernel_start_ns.numpy(), start)
    ref = oracle.plan(tr, tr.capacity_from_peak(peak))
    plan = gpu.g10_plan_migrations(tb, tr.capacity_from_peak(int(tl.peak_bytes)), tr.host_bw, tr.ssd_bw)
    assert np.array_equal(plan.summary.numpy()[:7], ref.summary[:7]) and int(plan.summary[7]) == 0
    n = int(plan.summary[0])
    assert np.array_equal(plan.migrations[:n * 48].numpy().view(gpu.MIGRATION_DTYPE), ref.migrations)
    assert np.array_equal(plan.final_pressure.numpy(), ref.final_pressure)


def test_full_size_stress_dag_passes(gpu, oracle):
    """Config 4 at full size (K = 1e6, N = 4e6): vitality and timeline element by element; the plan's first
    1000 iterations bit for bit against the oracle's lazy tier, and the invariants of a valid plan on them."""
    import torch
    tr = traces.config4_stress_dag()
    tb = gpu.upload(tr)
    v, ov = check_vitality(gpu, oracle, tr, tb)
    tl, (start, P0, peak, slot) = check_timeline(gpu, oracle, tr, tb)
    cap = tr.capacity_from_peak(peak)
    ref = oracle.plan(tr, cap, lazy=True, max_iterations=1000)
    plan = check_plan(gpu, tr, tb, cap, ref, max_iterations=1000)
    helpers.check_plan_invariants(tr, cap, start, P0, ov, gpu.migrations_numpy(plan), _np(plan.final_pressure),
                                  gpu.STATUS[int(plan.summary[2].item())], tr.host_bw, tr.ssd_bw, check_area=False)
    # the characterisation statistics (Section 3) at the same size, from the vitality just checked
    pn = int(v.counts[1].item())
    st = gpu.g10_characterize(tr.K, tr.N, v.use_ptr, v.uses, tb.tensor_bytes, tl.kernel_start_ns, pn, v.period_tensor,
                              v.period_prev_use, v.period_next_use, tr.host_bw, tr.ssd_bw)
    torch.cuda.synchronize()
    oc = oracle.characterize(tr.K, ov, tr.tensor_bytes, start, tr.host_bw, tr.ssd_bw)
    assert np.array_equal(_np(st.active_bytes)[:tr.K], oc.active_bytes)
    assert np.array_equal(_np(st.len_hist), oc.len_hist)
    assert np.array_equal(_np(st.size_len_hist).reshape(41, 45), oc.size_len_hist)
    assert np.array_equal(_np(st.hide), oc.hide) and np.array_equal(_np(st.summary), oc.summary)


def test_full_size_stress_plan_digest(gpu):
    """The complete plan of config 4 (13 505 migrations), the eager prefetch pass over it and the instruction stream
    emitted from both, against the digests of the CPU oracle's results stored by
    tests/golden/make_config4_plan_digest.py (the oracle needs about ten minutes for the plan)."""
    import hashlib, json, os
    import torch
    path = os.path.join(os.path.dirname(__file__), "golden", "config4_plan_digest.json")
    gold = json.load(open(path))
    tr = traces.config4_stress_dag()
    assert tr.sha256() == gold["trace_sha256"]
    tb = gpu.upload(tr)
    tl = gpu.g10_pressure_timeline(tb)
    torch.cuda.synchronize()
    assert int(tl.peak_bytes.item()) == gold["peak_bytes"] and int(tl.peak_slot.item()) == gold["peak_slot"]
    cap = tr.capacity_from_peak(int(tl.peak_bytes.item()))
    assert cap == gold["capacity_bytes"]
    plan = gpu.g10_plan_migrations(tb, cap, tr.host_bw, tr.ssd_bw)
    torch.cuda.synchronize()
    summary = _np(plan.summary)
    assert summary[7] == 0 and summary[:7].tolist() == gold["summary"]
    mig = gpu.migrations_numpy(plan)
    assert [[int(m[k]) for k in m.dtype.names] for m in mig[:5]] == gold["first_migrations"]
    h = hashlib.sha256()
    h.update(mig.tobytes()); h.update(_np(plan.final_pressure)[:tr.K].tobytes()); h.update(summary[:7].tobytes())
    assert h.hexdigest() == gold["plan_sha256"]
    # the eager prefetch pass over the same plan
    n = int(summary[0])
    pf = gpu.g10_schedule_prefetch(tr.K, n, plan.migrations, tl.kernel_start_ns, tb.tensor_bytes, cap, plan.final_pressure)
    torch.cuda.synchronize()
    assert _np(pf.summary)[:4].tolist() == gold["prefetch_summary"] and int(_np(pf.summary)[4]) == 0
    hp = hashlib.sha256()
    for a in (_np(pf.order)[:n], _np(pf.new_absent_last)[:n], _np(pf.new_prefetch_issue_ns)[:n], _np(pf.pressure)[:tr.K], _np(pf.summary)[:4]):
        hp.update(np.ascontiguousarray(a).tobytes())
    assert hp.hexdigest() == gold["prefetch_sha256"]
    # the instruction stream of that plan with the eager prefetch times (8 M records), field by field
    v = gpu.g10_vitality(tb)
    em = gpu.g10_emit_instructions(tr.K, tr.N, v.first_use, v.last_use, tb.tensor_bytes, tb.tensor_global, tl.kernel_start_ns,
                                   n, plan.migrations, pf.new_prefetch_issue_ns)
    torch.cuda.synchronize()
    assert int(em.counts[1].item()) == 0 and int(em.counts[0].item()) == gold["num_instructions"]
    got = gpu.instructions_numpy(em)
    he = hashlib.sha256()
    he.update(np.ascontiguousarray(_np(em.inst_ptr)).tobytes())
    for name in gold["instruction_fields"]:
        he.update(np.ascontiguousarray(got[name]).tobytes())
    assert he.hexdigest() == gold["instructions_sha256"]


def check_prefetch(gpu, oracle, tr, cap):
    """Eviction plan then the eager prefetch pass (Section 4.4), both sides from their own plan."""
    import torch
    tb = gpu.upload(tr)
    tl = gpu.g10_pressure_timeline(tb)
    plan = gpu.g10_plan_migrations(tb, cap, tr.host_bw, tr.ssd_bw)
    torch.cuda.synchronize()
    n = int(plan.summary[0].item())
    P1 = plan.final_pressure.clone()
    pf = gpu.g10_schedule_prefetch(tr.K, n, plan.migrations, tl.kernel_start_ns, tb.tensor_bytes, cap, plan.final_pressure)
    pf1 = gpu.g10_schedule_prefetch(tr.K, n, plan.migrations, tl.kernel_start_ns, tb.tensor_bytes, cap, P1, one_block=True)
    torch.cuda.synchronize()
    start = oracle.slot_clock(tr.kernel_ns)
    ref = oracle.plan(tr, cap, lazy=True)
    opf = oracle.schedule_prefetch(tr.K, ref.migrations, start, tr.tensor_bytes, cap, ref.final_pressure)
    assert n == len(ref.migrations)
    for got in (pf, pf1):                         # with a workspace (many blocks on a long timeline) and without (one block)
        assert np.array_equal(_np(got.order)[:n], opf.order)
        assert np.array_equal(_np(got.new_absent_last)[:n], opf.new_absent_last)
        assert np.array_equal(_np(got.new_prefetch_issue_ns)[:n], opf.new_prefetch_issue_ns)
        assert np.array_equal(_np(got.pressure)[:tr.K], opf.pressure)
        assert np.array_equal(_np(got.summary)[:4], opf.summary) and int(_np(got.summary)[4]) == 0
    return opf


def test_prefetch_pass(gpu, oracle):
    import json, os
    ex = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "hand_worked_examples.json")))["examples"]["prefetch"]
    tr = traces.from_lists("p", ex["kernel_lists"], ex["tensor_bytes"], ex["kernel_ns"], host_bw=ex["host_bw"], ssd_bw=ex["ssd_bw"])
    opf = check_prefetch(gpu, oracle, tr, ex["capacity"])
    assert opf.pressure.tolist() == ex["prefetch_pass"]["pressure"]
    rng = np.random.default_rng(99)
    for trial in range(40):
        toy = traces.random_toy(rng, int(rng.integers(4, 40)), int(rng.integers(1, 30)), max_deg=5)
        start, P0, peak, slot = oracle.timeline(toy)
        check_prefetch(gpu, oracle, toy, peak * int(rng.integers(1, 10)) // 10)
    moved = 0
    for cfg in (0, 1, 2, 3):
        tr = traces.make_config(cfg)
        start, P0, peak, slot = oracle.timeline(tr)
        moved += int(check_prefetch(gpu, oracle, tr, tr.capacity_from_peak(peak)).summary[0])
        if cfg == 0:
            moved += int(check_prefetch(gpu, oracle, tr, peak * 9 // 10).summary[0])      # ends FIT: room to move
    assert moved > 0
    tr = traces.config4_stress_dag(K=20000, N=80000)
    start, P0, peak, slot = oracle.timeline(tr)
    check_prefetch(gpu, oracle, tr, tr.capacity_from_peak(peak))
    check_prefetch(gpu, oracle, tr, peak * 8 // 10)


def check_emit(gpu, oracle, tr, cap, eager):
    """Instruction stream (Section 4.4, Figure 9) from the GPU's own vitality + plan (+ eager prefetch pass)."""
    import torch
    tb = gpu.upload(tr)
    v = gpu.g10_vitality(tb)
    tl = gpu.g10_pressure_timeline(tb)
    plan = gpu.g10_plan_migrations(tb, cap, tr.host_bw, tr.ssd_bw)
    torch.cuda.synchronize()
    n = int(plan.summary[0].item())
    ni = None
    if eager:
        pf = gpu.g10_schedule_prefetch(tr.K, n, plan.migrations, tl.kernel_start_ns, tb.tensor_bytes, cap, plan.final_pressure)
        ni = pf.new_prefetch_issue_ns
    em = gpu.g10_emit_instructions(tr.K, tr.N, v.first_use, v.last_use, tb.tensor_bytes, tb.tensor_global, tl.kernel_start_ns,
                                   n, plan.migrations, ni)
    torch.cuda.synchronize()
    assert int(em.counts[1].item()) == 0
    ov = oracle.vitality(tr.kernel_ptr, tr.kernel_tensors, tr.N)
    start = oracle.slot_clock(tr.kernel_ns)
    ref = oracle.plan(tr, cap, lazy=True)
    oni = None
    if eager:
        oni = oracle.schedule_prefetch(tr.K, ref.migrations, start, tr.tensor_bytes, cap, ref.final_pressure).new_prefetch_issue_ns
    oe = oracle.emit_instructions(tr.K, ov.first_use, ov.last_use, tr.tensor_bytes, tr.tensor_global, start, ref.migrations, oni)
    assert int(em.counts[0].item()) == len(oe.instructions)
    assert np.array_equal(_np(em.inst_ptr), oe.inst_ptr)
    got = gpu.instructions_numpy(em)
    for name in oe.instructions.dtype.names:
        assert np.array_equal(got[name], oe.instructions[name]), name
    return len(oe.instructions)


def test_instruction_stream(gpu, oracle):
    import json, os
    ex = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "hand_worked_examples.json")))["examples"]["A"]
    tr = traces.from_lists("A", ex["kernel_lists"], ex["tensor_bytes"], ex["kernel_ns"], host_bw=ex["host_bw"], ssd_bw=ex["ssd_bw"])
    assert check_emit(gpu, oracle, tr, ex["capacity"], False) == len(ex["instruction_stream"]["instructions"])
    rng = np.random.default_rng(2024)
    for trial in range(40):
        toy = traces.random_toy(rng, int(rng.integers(1, 40)), int(rng.integers(1, 30)), max_deg=5)
        start, P0, peak, slot = oracle.timeline(toy)
        check_emit(gpu, oracle, toy, peak * int(rng.integers(1, 10)) // 10, bool(trial % 2))
    for cfg in (0, 1, 2, 3):
        tr = traces.make_config(cfg)
        start, P0, peak, slot = oracle.timeline(tr)
        check_emit(gpu, oracle, tr, tr.capacity_from_peak(peak), cfg % 2 == 0)
    tr = traces.config4_stress_dag(K=20000, N=80000)
    start, P0, peak, slot = oracle.timeline(tr)
    assert check_emit(gpu, oracle, tr, tr.capacity_from_peak(peak), True) > 100000
    # very many tensors allocated at one boundary: the bucket is sorted in global memory
    lists = [list(range(6000))] + [[i] for i in range(0, 6000, 7)]
    big = traces.from_lists("wide", lists, [64] * 6000, [100] * len(lists), [1] * 3000 + [0] * 3000, capacity_bytes=10**9)
    check_emit(gpu, oracle, big, 10**9, False)


@pytest.mark.gpu
def test_instruction_stream_in_whole_rounds(gpu, oracle):
    """The stream of allocations and frees of a 200 000-kernel trace (no plan): 1.1 M instructions in more buckets than the
    writing kernel has blocks, so that the buckets are narrowed to whole rounds of its grid (592 buckets of 338 boundaries
    on a 148-SM part: a width that is no power of two)."""
    import torch
    tr = traces.config4_stress_dag(K=200_000, N=800_000)
    tb = gpu.upload(tr)
    v = gpu.g10_vitality(tb)
    tl = gpu.g10_pressure_timeline(tb)
    em = gpu.g10_emit_instructions(tr.K, tr.N, v.first_use, v.last_use, tb.tensor_bytes, tb.tensor_global, tl.kernel_start_ns, 0, None, None)
    torch.cuda.synchronize()
    assert int(em.counts[1].item()) == 0
    ov = oracle.vitality(tr.kernel_ptr, tr.kernel_tensors, tr.N)
    start = oracle.slot_clock(tr.kernel_ns)
    oe = oracle.emit_instructions(tr.K, ov.first_use, ov.last_use, tr.tensor_bytes, tr.tensor_global, start,
                                  np.zeros(0, oracle.MIGRATION_DTYPE), None)
    assert int(em.counts[0].item()) == len(oe.instructions) > 1_000_000
    assert np.array_equal(_np(em.inst_ptr), oe.inst_ptr)
    got = gpu.instructions_numpy(em)
    for name in got.dtype.names:
        assert np.array_equal(got[name], oe.instructions[name]), name


def check_stats(gpu, oracle, tr):
    """Characterisation statistics (Section 3, Figures 2-4) from the GPU's own vitality + slot clock."""
    import torch
    tb = gpu.upload(tr)
    v = gpu.g10_vitality(tb)
    tl = gpu.g10_pressure_timeline(tb)
    torch.cuda.synchronize()
    Pn = int(v.counts[1].item())
    st = gpu.g10_characterize(tr.K, tr.N, v.use_ptr, v.uses, tb.tensor_bytes, tl.kernel_start_ns, Pn, v.period_tensor,
                              v.period_prev_use, v.period_next_use, tr.host_bw, tr.ssd_bw)
    torch.cuda.synchronize()
    ov = oracle.vitality(tr.kernel_ptr, tr.kernel_tensors, tr.N)
    oc = oracle.characterize(tr.K, ov, tr.tensor_bytes, oracle.slot_clock(tr.kernel_ns), tr.host_bw, tr.ssd_bw)
    assert np.array_equal(_np(st.active_bytes)[:tr.K], oc.active_bytes)
    assert np.array_equal(_np(st.len_hist), oc.len_hist)
    assert np.array_equal(_np(st.size_len_hist).reshape(41, 45), oc.size_len_hist)
    assert np.array_equal(_np(st.hide), oc.hide)
    assert np.array_equal(_np(st.summary), oc.summary)
    return int(oc.len_hist.sum())


@pytest.mark.gpu
def test_characterisation_statistics(gpu, oracle):
    rng = np.random.default_rng(77)
    for trial in range(40):
        check_stats(gpu, oracle, traces.random_toy(rng, int(rng.integers(1, 40)), int(rng.integers(1, 30)), max_deg=5))
    for cfg in (0, 1, 2, 3):
        check_stats(gpu, oracle, traces.make_config(cfg))
    assert check_stats(gpu, oracle, traces.config4_stress_dag(K=200000, N=800000)) > 100000
    # one tensor used by thousands of kernels (the warp shares its use list); sizes and lengths at the histogram edges
    lists = [[0, 1 + (k % 5)] for k in range(5000)]
    tr = traces.from_lists("hot", lists, [1 << 44, 1, 2, 3, 1 << 41, 1 << 40], [((1 << 44) - 1) if k % 3 else 1 for k in range(5000)],
                           [1, 0, 0, 0, 0, 0], capacity_bytes=1 << 50)
    check_stats(gpu, oracle, tr)
    # empty trace
    check_stats(gpu, oracle, traces.from_lists("empty", [], [], [], [], capacity_bytes=1))


def check_batch(gpu, oracle, tr, variants, max_iterations=0):
    """Batched re-planning: every variant equals the oracle's plan of the perturbed trace; stability pairs equal."""
    import torch
    tb = gpu.upload(tr)
    dev_variants = []
    for v in variants:
        d = dict(v)
        if v.get("kernel_ns") is not None:
            d["kernel_ns"] = torch.from_numpy(np.ascontiguousarray(v["kernel_ns"], dtype=np.int64)).cuda()
        dev_variants.append(d)
    got = gpu.g10_plan_batch(tb, dev_variants, max_iterations=max_iterations)
    torch.cuda.synchronize()
    ref = oracle.plan_batch(tr, variants, max_iterations=max_iterations)
    summary = _np(got.summary)
    for j, r in enumerate(ref.plans):
        assert summary[j, 7] == 0, "variant %d device status %x" % (j, summary[j, 7])
        assert np.array_equal(summary[j, :7], r.summary[:7]), (j, summary[j], r.summary)
        assert np.array_equal(gpu.batch_migrations_numpy(got, j), r.migrations), j
        assert np.array_equal(_np(got.final_pressure)[j, :tr.K], r.final_pressure), j
    assert np.array_equal(_np(got.stability)[:len(variants)], ref.stability)
    return ref


def _jitter(rng, dur, pct):
    f = rng.uniform(1.0 - pct / 100.0, 1.0 + pct / 100.0, size=len(dur))
    return np.maximum(1, np.rint(np.asarray(dur, dtype=np.float64) * f)).astype(np.int64)


@pytest.mark.gpu
def test_batched_replanning(gpu, oracle):
    rng = np.random.default_rng(4242)
    for trial in range(12):
        tr = traces.random_toy(rng, int(rng.integers(1, 40)), int(rng.integers(1, 30)), max_deg=5)
        start, P0, peak, slot = oracle.timeline(tr)
        cap = peak * int(rng.integers(1, 10)) // 10
        base = dict(gpu_capacity_bytes=cap, host_bw=tr.host_bw, ssd_bw=tr.ssd_bw)
        variants = [base, dict(base, kernel_ns=_jitter(rng, tr.kernel_ns, 25)), dict(base, ssd_bw=tr.ssd_bw * 3),
                    dict(base, host_capacity_bytes=int(rng.integers(1, 200))), dict(base, gpu_capacity_bytes=cap // 2)]
        check_batch(gpu, oracle, tr, variants, max_iterations=int(rng.integers(0, 3)) * 2)
    for cfg in (0, 1, 2):
        tr = traces.make_config(cfg)
        start, P0, peak, slot = oracle.timeline(tr)
        cap = tr.capacity_from_peak(peak)
        base = dict(gpu_capacity_bytes=cap, host_bw=tr.host_bw, ssd_bw=tr.ssd_bw)
        variants = [base] + [dict(base, kernel_ns=_jitter(rng, tr.kernel_ns, pct)) for pct in (5, 10, 15, 20, 25)]
        variants += [dict(base, ssd_bw=bw) for bw in (12_800_000_000, 19_200_000_000, 32_000_000_000)]
        variants += [dict(base, host_capacity_bytes=hc << 30) for hc in (1, 32, 256)]
        ref = check_batch(gpu, oracle, tr, variants)
        assert ref.stability[0, 0] == ref.stability[0, 1] == len(ref.plans[0].migrations)
    # a variant with an invalid duration reports it in its own status word, the others stay clean
    import torch
    tr = traces.config0_mlp_chain()
    tb = gpu.upload(tr)
    start, P0, peak, slot = oracle.timeline(tr)
    base = dict(gpu_capacity_bytes=tr.capacity_from_peak(peak), host_bw=tr.host_bw, ssd_bw=tr.ssd_bw)
    bad = tr.kernel_ns.copy(); bad[5] = 0
    got = gpu.g10_plan_batch(tb, [base, dict(base, kernel_ns=torch.from_numpy(bad).cuda()), base])
    torch.cuda.synchronize()
    s7 = _np(got.summary)[:, 7]
    assert s7[0] == 0 and (s7[1] & 0x8) and s7[2] == 0
    # a trace too large for one SM: the variants are planned one after the other by the planners that use the whole GPU
    tr = traces.make_config(3)
    start, P0, peak, slot = oracle.timeline(tr)
    base = dict(gpu_capacity_bytes=tr.capacity_from_peak(peak), host_bw=tr.host_bw, ssd_bw=tr.ssd_bw)
    variants = [base, dict(base, kernel_ns=_jitter(rng, tr.kernel_ns, 10)), dict(base, ssd_bw=4 * tr.ssd_bw),
                dict(base, gpu_capacity_bytes=base["gpu_capacity_bytes"] * 3 // 4, host_capacity_bytes=64 << 30),
                dict(base, kernel_ns=_jitter(rng, tr.kernel_ns, 25), host_bw=2 * tr.host_bw)]
    ref = check_batch(gpu, oracle, tr, variants)
    assert ref.stability[0, 0] == ref.stability[0, 1] == len(ref.plans[0].migrations) > 1000
    ref = check_batch(gpu, oracle, tr, variants[:2], max_iterations=50)
    assert len(ref.plans[1].migrations) == 50


def check_cyclic(gpu, oracle, tr, cap, host_capacity=0, max_iterations=0):
    """Steady-state plan on the cyclic timeline against the oracle's (plain tier)."""
    import torch
    tb = gpu.upload(tr)
    plan = gpu.g10_plan_cyclic(tb, cap, tr.host_bw, tr.ssd_bw, host_capacity_bytes=host_capacity, max_iterations=max_iterations)
    torch.cuda.synchronize()
    ref = oracle.plan_cyclic(tr, cap, host_capacity_bytes=host_capacity, max_iterations=max_iterations)
    summary = _np(plan.summary)
    assert summary[7] == 0, "device status %x" % summary[7]
    assert np.array_equal(summary[:7], ref.summary[:7]), (summary, ref.summary)
    assert np.array_equal(gpu.migrations_numpy(plan), ref.migrations)
    assert np.array_equal(_np(plan.final_pressure)[:tr.K], ref.final_pressure)
    # the calls behind the plan take the steady-state plan as it is (Section 4.4): eager prefetch pass (with the plan's
    # capacity and with more room, so that wrap-around prefetches move too), then the instruction stream of one iteration
    if tr.K > 0 and len(ref.migrations) > 0 and max_iterations == 0:
        n = len(ref.migrations)
        tl = gpu.g10_pressure_timeline(tb)
        v = gpu.g10_vitality(tb)
        ov = oracle.vitality(tr.kernel_ptr, tr.kernel_tensors, tr.N)
        start = oracle.slot_clock(tr.kernel_ns)
        for cap2 in (cap, cap + int(tr.tensor_bytes.max())):
            P = plan.final_pressure.clone()
            pf = gpu.g10_schedule_prefetch(tr.K, n, plan.migrations, tl.kernel_start_ns, tb.tensor_bytes, cap2, P)
            em = gpu.g10_emit_instructions(tr.K, tr.N, v.first_use, v.last_use, tb.tensor_bytes, tb.tensor_global, tl.kernel_start_ns,
                                           n, plan.migrations, pf.new_prefetch_issue_ns)
            torch.cuda.synchronize()
            opf = oracle.schedule_prefetch(tr.K, ref.migrations, start, tr.tensor_bytes, cap2, ref.final_pressure)
            assert np.array_equal(_np(pf.order)[:n], opf.order) and np.array_equal(_np(pf.new_absent_last)[:n], opf.new_absent_last)
            assert np.array_equal(_np(pf.new_prefetch_issue_ns)[:n], opf.new_prefetch_issue_ns)
            assert np.array_equal(_np(P)[:tr.K], opf.pressure) and np.array_equal(_np(pf.summary)[:4], opf.summary) and int(_np(pf.summary)[4]) == 0
            oe = oracle.emit_instructions(tr.K, ov.first_use, ov.last_use, tr.tensor_bytes, tr.tensor_global, start, ref.migrations,
                                          opf.new_prefetch_issue_ns)
            assert int(em.counts[1].item()) == 0 and int(em.counts[0].item()) == len(oe.instructions)
            assert np.array_equal(_np(em.inst_ptr), oe.inst_ptr)
            got = gpu.instructions_numpy(em)
            for name in oe.instructions.dtype.names:
                assert np.array_equal(got[name], oe.instructions[name]), name
    return ref


@pytest.mark.gpu
def synthetic_prefetch_records(gpu, rng, K, n, wrap, long_share=0.3):
    """Seeded records over a random pressure curve: absent ranges that are short or (a share of them) as long as most of
    the timeline, capacity such that about one slot in sixteen cannot take a mid-sized tensor."""
    dur = rng.integers(1, 1000, size=K).astype(np.int64)
    start = np.concatenate([[0], np.cumsum(dur)]).astype(np.int64)
    T = int(start[K])
    N = 64
    nbytes = rng.integers(1, 1 << 20, size=N).astype(np.int64)
    P = rng.integers(0, 1 << 22, size=K).astype(np.int64)
    mig = np.zeros(n, dtype=gpu.MIGRATION_DTYPE)
    a = rng.integers(0, K, size=n)
    length = np.where(rng.random(n) < long_share, rng.integers(1, K - 1, size=n), rng.integers(1, 64, size=n))
    b = np.minimum(a + length - 1, a + K - 2)
    if not wrap:
        b = np.minimum(b, K - 1)
    mig["absent_first"], mig["absent_last"] = a, b
    mig["tensor"] = rng.integers(0, N, size=n)
    issue = np.where(b + 1 <= K, start[np.minimum(b + 1, K)], start[(b + 1) % K] + T) - rng.integers(0, 2, size=n)
    mig["prefetch_issue_ns"] = issue
    mig["period"] = np.arange(n)
    return mig, start, nbytes, P


def check_prefetch_records(gpu, oracle, K, mig, start, nbytes, cap, P, **kw):
    import torch
    n = len(mig)
    dm = torch.from_numpy(mig.view(np.uint8).copy()).cuda()
    dP = torch.from_numpy(P.copy()).cuda()
    pf = gpu.g10_schedule_prefetch(K, n, dm, torch.from_numpy(start).cuda(), torch.from_numpy(nbytes).cuda(), cap, dP, **kw)
    torch.cuda.synchronize()
    opf = oracle.schedule_prefetch(K, mig, start, nbytes, cap, P)
    assert np.array_equal(_np(pf.order)[:n], opf.order)
    assert np.array_equal(_np(pf.new_absent_last)[:n], opf.new_absent_last)
    assert np.array_equal(_np(pf.new_prefetch_issue_ns)[:n], opf.new_prefetch_issue_ns)
    assert np.array_equal(_np(dP), opf.pressure)
    assert np.array_equal(_np(pf.summary)[:4], opf.summary) and int(_np(pf.summary)[4]) == 0
    return opf


@pytest.mark.gpu
def test_prefetch_pass_on_wrapping_records(gpu, oracle):
    """The eager prefetch pass on synthetic records whose absent ranges reach into the next iteration, for every kernel the
    call can choose: pressure curve in shared memory (K = 5000), per-tile bounds in shared memory (K = 40 000, several
    tiles and a ragged last one) -- called without a workspace, and with one (the many-block form then hands such
    records to the one-block form behind it)."""
    rng = np.random.default_rng(60221023)
    for K, n in ((5000, 400), (40000, 1500), (40000, 6000)):
        mig, start, nbytes, P = synthetic_prefetch_records(gpu, rng, K, n, wrap=True)
        assert (mig["absent_last"] >= K).sum() > 20
        for one_block in (True, False):
            opf = check_prefetch_records(gpu, oracle, K, mig, start, nbytes, int(1 << 22), P, one_block=one_block)
        assert int(opf.summary[0]) > n // 10


@pytest.mark.gpu
def test_prefetch_pass_in_slices(gpu, oracle):
    """The many-block form of the eager prefetch pass (timeline cut into one slice per thread block) on synthetic records
    that do not wrap: short and very long absent ranges mixed, so that searches start everywhere at once, run through many
    slices and wait for one another; slice counts from a handful to every block the GPU holds, ragged last slice; a curve
    where nothing blocks (every search runs to absent_first) and one where everything does; empty ranges."""
    rng = np.random.default_rng(2310094431)
    for K, n, long_share in ((15361, 300, 0.3), (40000, 6000, 0.3), (151552 + 77, 9000, 0.1), (400003, 12000, 0.02), (1200007, 5000, 0.01)):
        mig, start, nbytes, P = synthetic_prefetch_records(gpu, rng, K, n, wrap=False, long_share=long_share)
        opf = check_prefetch_records(gpu, oracle, K, mig, start, nbytes, int(1 << 22), P)
        assert int(opf.summary[0]) > n // 10
    K, n = 60000, 3000
    mig, start, nbytes, P = synthetic_prefetch_records(gpu, rng, K, n, wrap=False, long_share=0.5)
    check_prefetch_records(gpu, oracle, K, mig, start, nbytes, int(1 << 62), P)          # nothing ever blocks
    check_prefetch_records(gpu, oracle, K, mig, start, nbytes, 0, P)                     # every slot blocks: nothing moves
    mig2 = mig.copy()
    empty = rng.random(n) < 0.2
    mig2["absent_first"] = np.where(empty, mig2["absent_last"] + 1, mig2["absent_first"])   # ranges without a slot
    check_prefetch_records(gpu, oracle, K, mig2, start, nbytes, int(1 << 22), P)
    # equal prefetch times: the visiting order falls back to the record index
    mig3 = mig.copy()
    mig3["prefetch_issue_ns"] = (mig3["prefetch_issue_ns"] // 100000) * 100000
    check_prefetch_records(gpu, oracle, K, mig3, start, nbytes, int(1 << 22), P)


@pytest.mark.gpu
def test_cyclic_planning(gpu, oracle):
    import json, os, torch
    ex = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "cyclic_example.json")))
    tr = traces.from_lists("cyc", ex["kernel_lists"], ex["tensor_bytes"], ex["kernel_ns"], ex["tensor_global"],
                           host_bw=ex["host_bw"], ssd_bw=ex["ssd_bw"], capacity_bytes=ex["capacity"])
    ref = check_cyclic(gpu, oracle, tr, ex["capacity"])
    assert ref.final_pressure.tolist() == ex["final_pressure"]
    rng = np.random.default_rng(1618)
    wrapped = 0
    for trial in range(60):
        toy = traces.random_toy(rng, int(rng.integers(1, 40)), int(rng.integers(1, 30)), max_deg=5)
        if trial % 3 == 0:
            toy.tensor_global = np.ones(toy.N, np.uint8)
        start, P0, peak, slot = oracle.timeline(toy)
        hc = int(rng.integers(0, 3)) * int(rng.integers(1, 80))
        ref = check_cyclic(gpu, oracle, toy, peak * int(rng.integers(0, 10)) // 10, host_capacity=hc, max_iterations=int(rng.integers(0, 2)) * 3)
        wrapped += int((ref.migrations["absent_last"] >= toy.K).sum())
    assert wrapped > 10
    for cfg in (0, 1, 2):
        tr = traces.make_config(cfg)
        start, P0, peak, slot = oracle.timeline(tr)
        ref = check_cyclic(gpu, oracle, tr, tr.capacity_from_peak(peak))
        plain = oracle.plan(tr, tr.capacity_from_peak(peak), lazy=True)
        assert ref.summary[3] <= plain.summary[3]            # the weights' wrap-around periods only add options here
    for lists, nb in (([], []), ([[], []], []), ([[0], [0], [0]], [9])):
        tr = traces.from_lists("e", lists, nb, [3] * len(lists), [1] * len(nb), capacity_bytes=0)
        check_cyclic(gpu, oracle, tr, 0)
    # too large for one SM: the multi-block planner behind the single-block one takes over (Algorithm 1 as printed, on
    # the cycle).  The oracle's plain tier needs most of a minute for the whole plan of this trace, so the first 400
    # iterations are compared record by record, and a shorter ViT-shaped trace (two iterations) to the end.
    tr = traces.make_config(3)
    start, P0, peak, slot = oracle.timeline(tr)
    ref = check_cyclic(gpu, oracle, tr, tr.capacity_from_peak(peak), max_iterations=400)
    assert len(ref.migrations) == 400 and int((ref.migrations["absent_last"] >= tr.K).sum()) > 0
    tr = traces.config3_vit_huge(iterations=2)
    start, P0, peak, slot = oracle.timeline(tr)
    ref = check_cyclic(gpu, oracle, tr, tr.capacity_from_peak(peak))
    assert int((ref.migrations["absent_last"] >= tr.K).sum()) > 10
    # host-pointer form of the call (the library stages the copies itself)
    tr = traces.make_config(1)
    start, P0, peak, slot = oracle.timeline(tr)
    cap = tr.capacity_from_peak(peak)
    ref = oracle.plan_cyclic(tr, cap)
    plan = gpu.g10_plan_cyclic(gpu.pin(tr), cap, tr.host_bw, tr.ssd_bw)
    assert np.array_equal(plan.summary.numpy()[:7], ref.summary[:7]) and int(plan.summary[7]) == 0
    n = int(plan.summary[0])
    assert np.array_equal(plan.migrations[:n * 48].numpy().view(gpu.MIGRATION_DTYPE), ref.migrations)
    assert np.array_equal(plan.final_pressure.numpy(), ref.final_pressure)


@pytest.mark.gpu
def test_crowded_ties_and_conflicts(gpu, oracle):
    """Thousands of identical periods: every commit makes all the others stale with equal bounds and blocks their
    transfer windows, so the planners' rarely used paths run (rounds beyond their size limits, lists used up and
    published again, very many destinations re-chosen at once).  All planners against the oracle."""
    K = 60
    for n, size, dur in ((1500, 1 << 20, 1000000), (700, 3 << 20, 2000000)):
        lists = [[] for _ in range(K)]
        for i in range(n):
            lists[i % 20].append(i)                      # twenty groups of identical periods, all overlapping in the middle
            lists[K - 1 - (i % 7)].append(i)
        sizes = [size + (i % 4) for i in range(n)]       # a few distinct sizes: near-ties next to exact ties
        tr = traces.from_lists("crowd", lists, sizes, [dur] * K, capacity_frac=(1, 3))
        tb = gpu.upload(tr)
        start, P0, peak, slot = oracle.timeline(tr)
        cap = tr.capacity_from_peak(peak)
        ref = oracle.plan(tr, cap, lazy=True)
        assert np.array_equal(ref.migrations, oracle.plan(tr, cap).migrations) and len(ref.migrations) > 100
        for flags in (0, gpu.FLAG_GLOBAL_STATE, gpu.FLAG_MULTI_BLOCK, gpu.FLAG_RESCORE_ALL):
            check_plan(gpu, tr, tb, cap, ref, flags=flags)
        check_cyclic(gpu, oracle, tr, cap)


@pytest.mark.gpu
def test_analysis_call_in_a_cuda_graph(gpu, oracle):
    """The device-mode calls only enqueue work on the caller's stream (kernels, memsets; programmatic dependencies between
    them): they can be captured in a CUDA graph and replayed.  The one-call analysis of config 1, captured once, replayed
    three times into cleared outputs, against the oracle."""
    import torch
    tr = traces.config1_resnet152()
    tb = gpu.upload(tr)
    ws = torch.empty(gpu.g10_workspace_bytes(gpu.WS_ANALYSIS, tb.K, tb.N, tb.E), dtype=torch.uint8, device="cuda")
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        v = gpu.g10_vitality(tb, ws=ws, timeline=True, stream=s)             # (first call outside the capture: attributes get set)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            gpu.g10_vitality(tb, ws=ws, out=v, timeline=v.timeline, stream=torch.cuda.current_stream())
    torch.cuda.synchronize()
    ov = oracle.vitality(tr.kernel_ptr, tr.kernel_tensors, tr.N)
    start, P0, peak, slot = oracle.timeline(tr)
    for _ in range(3):
        for t in (v.first_use, v.last_use, v.period_tensor, v.timeline.pressure, v.counts, v.timeline.peak_bytes):
            t.zero_()
        g.replay()
        torch.cuda.synchronize()
        pn = int(v.counts[1].item())
        assert int(v.counts[2].item()) == 0 and int(v.timeline.status.item()) == 0 and pn == len(ov.period_tensor)
        assert np.array_equal(_np(v.first_use), ov.first_use) and np.array_equal(_np(v.last_use), ov.last_use)
        assert np.array_equal(_np(v.period_tensor)[:pn], ov.period_tensor)
        assert np.array_equal(_np(v.timeline.pressure)[:tr.K], P0) and int(v.timeline.peak_bytes.item()) == peak
