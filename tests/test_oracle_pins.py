"""Pins for the CPU oracle: each test ties an oracle function to something other than itself --
hand-worked examples, dense brute force on toy traces, closed forms, invariants, special cases."""
import json
import os

import numpy as np
import pytest

import helpers
from paper_2310_09443_b200 import traces

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_worked_examples.json")


def _example(name):
    ex = json.load(open(GOLDEN))["examples"][name]
    tr = traces.from_lists(name, ex["kernel_lists"], ex["tensor_bytes"], ex["kernel_ns"],
                           host_bw=ex["host_bw"], ssd_bw=ex["ssd_bw"])
    return ex, tr


def test_example_A_vitality_pressure_geometry(oracle):
    ex, tr = _example("A")
    v = oracle.vitality(tr.kernel_ptr, tr.kernel_tensors, tr.N)
    assert v.first_use.tolist() == ex["first_use"] and v.last_use.tolist() == ex["last_use"]
    got = list(zip(v.period_tensor.tolist(), v.period_prev_use.tolist(), v.period_next_use.tolist()))
    assert got == [tuple(p) for p in ex["periods"]]
    start, P, peak, slot = oracle.timeline(tr)
    assert start.tolist() == ex["start"] and P.tolist() == ex["pressure"] and [peak, slot] == ex["peak"]
    g = oracle.geometry(start, tr.tensor_bytes, v.period_tensor, v.period_prev_use, v.period_next_use,
                        tr.host_bw, tr.ssd_bw)
    for X, key in ((0, "geometry_ssd"), (1, "geometry_host")):
        got = [[int(g.transfer_ns[X, p]), int(g.absent_first[X, p]), int(g.absent_last[X, p])] for p in range(2)]
        assert got == ex[key]


@pytest.mark.parametrize("name", ["A", "A_prime", "B"])
@pytest.mark.parametrize("lazy", [False, True])
def test_hand_worked_plans(oracle, name, lazy):
    ex, tr = _example(name)
    r = oracle.plan(tr, ex["capacity"], lazy=lazy)
    assert r.status == ex["status"]
    assert len(r.migrations) == len(ex["migrations"])
    for j, (m, e) in enumerate(zip(r.migrations, ex["migrations"])):
        for key in ("period", "tensor", "dest", "absent_first", "absent_last", "iteration", "evict_issue_ns",
                    "prefetch_issue_ns", "transfer_ns"):
            assert int(m[key]) == e[key], (j, key)
        assert r.win_benefit[j] == e["benefit"] and int(r.win_cost[j]) == e["cost"]
    assert r.final_pressure.tolist() == ex["final_pressure"]
    assert [int(r.summary[3]), int(r.summary[4])] == ex["final_peak"]
    assert int(r.summary[0]) == len(ex["migrations"])


def test_brute_force_agrees_with_hand_worked():
    """The dense checker itself is pinned to the same hand-worked numbers."""
    for name in ("A", "A_prime", "B"):
        ex, tr = _example(name)
        b = helpers.brute_plan(tr, ex["capacity"], ex["host_bw"], ex["ssd_bw"])
        assert b["status"] == ex["status"] and b["final_pressure"] == ex["final_pressure"]
        assert [{k: m[k] for k in e} for m, e in zip(b["plan"], ex["migrations"])] == ex["migrations"]


def test_vitality_pressure_exhaustive_small():
    """All 2^(K*N) use patterns for K*N <= 12: vitality and pressure against the dense definition."""
    from oracle import g10_oracle as O
    for K, N in ((4, 3), (6, 2), (3, 4), (12, 1)):
        for bits in range(1 << (K * N)):
            lists = [[i for i in range(N) if (bits >> (k * N + i)) & 1] for k in range(K)]
            tr = traces.from_lists("x", lists, [3 + 5 * i for i in range(N)], [1 + k for k in range(K)],
                                   [(i % 2) for i in range(N)])
            uses, first, last, periods = helpers.brute_vitality(tr)
            v = O.vitality(tr.kernel_ptr, tr.kernel_tensors, N)
            assert v.first_use.tolist() == first and v.last_use.tolist() == last
            assert v.uses.tolist() == [k for u in uses for k in u]
            assert list(zip(v.period_tensor.tolist(), v.period_prev_use.tolist(), v.period_next_use.tolist())) == periods
            P, peak, slot = O.pressure(K, tr.tensor_bytes, tr.tensor_global, v.first_use, v.last_use)
            bp = helpers.brute_pressure(tr, uses)
            assert P.tolist() == bp and peak == max(bp) and slot == bp.index(max(bp))


def test_random_toy_full_path(oracle):
    """Random toy traces (empty kernels, in-kernel repeats, unused tensors, globals): every stage and the
    whole plan against the dense big-integer restatement; lazy tier equals plain tier."""
    rng = np.random.default_rng(12345)
    n_plans = 0
    for trial in range(400):
        K = int(rng.integers(1, 15)); N = int(rng.integers(1, 9))
        tr = traces.random_toy(rng, K, N)
        uses, first, last, periods = helpers.brute_vitality(tr)
        v = oracle.vitality(tr.kernel_ptr, tr.kernel_tensors, N)
        assert v.first_use.tolist() == first and v.last_use.tolist() == last
        assert v.num_uses.tolist() == [len(u) for u in uses]
        assert v.use_ptr.tolist() == np.concatenate([[0], np.cumsum([len(u) for u in uses])]).tolist()
        assert list(zip(v.period_tensor.tolist(), v.period_prev_use.tolist(), v.period_next_use.tolist())) == periods
        start, P, peak, slot = oracle.timeline(tr)
        assert start.tolist() == helpers.brute_start(tr)
        bp = helpers.brute_pressure(tr, uses)
        assert P.tolist() == bp
        g = oracle.geometry(start, tr.tensor_bytes, v.period_tensor, v.period_prev_use, v.period_next_use,
                            tr.host_bw, tr.ssd_bw)
        for X, bw in ((0, tr.ssd_bw), (1, tr.host_bw)):
            for p, per in enumerate(periods):
                bg = helpers.brute_geometry(tr, start.tolist(), per, bw)
                assert int(g.transfer_ns[X, p]) == bg["t"]
                if bg["valid"]:
                    assert (int(g.absent_first[X, p]), int(g.absent_last[X, p])) == (bg["a_abs"], bg["b_abs"])
                else:
                    assert (int(g.absent_first[X, p]), int(g.absent_last[X, p])) == (-1, -2)
        for frac in ((1, 2), (1, 5), (0, 1)):
            cap = peak * frac[0] // frac[1]
            hc = int(rng.integers(0, 3)) * int(rng.integers(1, 80))
            b = helpers.brute_plan(tr, cap, tr.host_bw, tr.ssd_bw, host_capacity=hc)
            for lazy in (False, True):
                r = oracle.plan(tr, cap, host_capacity_bytes=hc, lazy=lazy)
                assert r.status == b["status"]
                got = [{k: int(m[k]) for k in m.dtype.names} for m in r.migrations]
                exp = [{k: m[k] for k in r.migrations.dtype.names} for m in b["plan"]]
                assert got == exp
                assert r.win_benefit == [m["benefit"] for m in b["plan"]]
                assert r.final_pressure.tolist() == b["final_pressure"]
                assert (int(r.summary[3]), int(r.summary[4])) == b["final_peak"]
                assert int(r.summary[1]) == b["rounds"]
            n_plans += len(b["plan"])
    assert n_plans > 200      # the sweep really exercises the loop


def test_config0_closed_forms(oracle):
    """MLP chain: fwd_l = l-1, bwd_l = 32 + 2(32-l), opt_l = 33 + 2(32-l).  A_{l-1} and W_l each have one
    period fwd_l -> bwd_l for l <= 31; dA_l (l = 1..31) has one 1-slot period; nothing else: 93 periods."""
    tr = traces.config0_mlp_chain()
    assert (tr.K, tr.N, tr.E) == (96, 130, 320)
    L = 32
    v = oracle.vitality(tr.kernel_ptr, tr.kernel_tensors, tr.N)
    fwd = lambda l: l - 1
    bwd = lambda l: 32 + 2 * (L - l)
    opt = lambda l: 33 + 2 * (L - l)
    exp = []
    for l in range(1, L):                      # A_{l-1}: id l-1
        exp.append((l - 1, fwd(l), bwd(l)))
    for l in range(1, L):                      # dA_l: id 33 + l, written by bwd_{l+1}, read by bwd_l
        exp.append((33 + l, bwd(l + 1), bwd(l)))
    for l in range(1, L):                      # W_l: id 66 + l - 1
        exp.append((66 + l - 1, fwd(l), bwd(l)))
    got = list(zip(v.period_tensor.tolist(), v.period_prev_use.tolist(), v.period_next_use.tolist()))
    assert got == sorted(exp) and len(got) == 93
    for l in range(1, L + 1):
        assert v.first_use[66 + l - 1] == fwd(l) and v.last_use[66 + l - 1] == opt(l)
        assert v.num_uses[98 + l - 1] == 2
    # the 1-slot dA periods can never host a migration
    start = oracle.slot_clock(tr.kernel_ns)
    g = oracle.geometry(start, tr.tensor_bytes, v.period_tensor, v.period_prev_use, v.period_next_use,
                        tr.host_bw, tr.ssd_bw)
    short = (v.period_next_use - v.period_prev_use) < 4
    assert short.sum() == 31 and np.all(g.absent_first[:, short] == -1)


def _replay(oracle, tr, cap, r, host_capacity=0):
    v = oracle.vitality(tr.kernel_ptr, tr.kernel_tensors, tr.N)
    start, P0, peak, slot = oracle.timeline(tr)
    return helpers.check_plan_invariants(tr, cap, start, P0, v, r.migrations, r.final_pressure, r.status,
                                         tr.host_bw, tr.ssd_bw, win_benefit=r.win_benefit,
                                         host_capacity=host_capacity), v, start


@pytest.mark.parametrize("cfg", [0, 1, 2])
def test_plan_invariants_on_configs(oracle, cfg):
    tr = traces.make_config(cfg)
    start, P0, peak, slot = oracle.timeline(tr)
    # conservation: sum of pressure over slots = sum over tensors of size * live slots
    v = oracle.vitality(tr.kernel_ptr, tr.kernel_tensors, tr.N)
    live = np.where(v.first_use < 0, 0, np.where(tr.tensor_global == 1, tr.K, v.last_use - v.first_use + 1))
    assert int(P0.astype(object).sum()) == int((tr.tensor_bytes.astype(object) * live.astype(object)).sum())
    cap = tr.capacity_from_peak(peak)
    r = oracle.plan(tr, cap)
    (P, busy, hocc), v, start = _replay(oracle, tr, cap, r)
    assert np.all(busy <= tr.kernel_ns[None, :])
    r2 = oracle.plan(tr, cap, lazy=True)
    assert np.array_equal(r.migrations, r2.migrations) and np.array_equal(r.final_pressure, r2.final_pressure)
    assert np.array_equal(r.summary, r2.summary)
    if r.status == "EXHAUSTED":
        # nothing left: every remaining period is inadmissible or relieves nothing (checked with numpy)
        done = set(r.migrations["period"].tolist())
        g = oracle.geometry(start, tr.tensor_bytes, v.period_tensor, v.period_prev_use, v.period_next_use,
                            tr.host_bw, tr.ssd_bw)
        ex = np.maximum(P - cap, 0)
        for p in range(len(v.period_tensor)):
            if p in done:
                continue
            u, w = int(v.period_prev_use[p]), int(v.period_next_use[p])
            a, b = u + 1, w - 1
            for X in (0, 1):
                ap, bp, t = int(g.absent_first[X, p]), int(g.absent_last[X, p]), int(g.transfer_ns[X, p])
                if ap < 0:
                    continue
                ks = np.arange(a, ap)
                ov = np.minimum(start[a] + t, start[ks + 1]) - np.maximum(start[a], start[ks])
                ok = np.all(busy[2 * X, a:ap] + ov <= tr.kernel_ns[a:ap])
                ks = np.arange(bp + 1, b + 1)
                ov = np.minimum(start[w], start[ks + 1]) - np.maximum(start[w] - t, start[ks])
                ok = ok and np.all(busy[2 * X + 1, bp + 1:b + 1] + ov <= tr.kernel_ns[bp + 1:b + 1])
                if ok:
                    assert ex[ap:bp + 1].max() == 0, "an admissible beneficial candidate was left behind"
                    break


def test_special_cases(oracle):
    tr = traces.config0_mlp_chain()
    start, P0, peak, slot = oracle.timeline(tr)
    r = oracle.plan(tr, peak)                       # capacity >= peak: nothing to do
    assert r.status == "ALREADY_FITS" and len(r.migrations) == 0 and np.array_equal(r.final_pressure, P0)
    r = oracle.plan(tr, 1 << 63)
    assert r.status == "ALREADY_FITS"
    r = oracle.plan(tr, peak // 2, host_bw=1, ssd_bw=1)   # transfers far longer than any period
    assert r.status == "EXHAUSTED" and len(r.migrations) == 0
    # enormous bandwidth: t = 1 ns, so a' = a + 1 and b' = b - 1 for every migration
    r = oracle.plan(tr, peak // 2, host_bw=1 << 62, ssd_bw=1 << 62)
    v = oracle.vitality(tr.kernel_ptr, tr.kernel_tensors, tr.N)
    assert len(r.migrations) > 0
    for m in r.migrations:
        p = int(m["period"])
        assert m["transfer_ns"] == 1
        assert m["absent_first"] == v.period_prev_use[p] + 2 and m["absent_last"] == v.period_next_use[p] - 2
    # iteration limit
    r3 = oracle.plan(tr, peak * 2 // 5, max_iterations=3)
    full = oracle.plan(tr, peak * 2 // 5)
    assert r3.status == "ITERATION_LIMIT" and np.array_equal(r3.migrations, full.migrations[:3])
    # empty traces
    for lists, nb in (([], []), ([[], []], []), ([[], []], [5, 7])):
        e = traces.from_lists("e", lists, nb, [3] * len(lists))
        r = oracle.plan(e, 0)
        assert r.status == "ALREADY_FITS" and len(r.migrations) == 0
        assert int(r.summary[3]) == 0 and int(r.summary[4]) == (0 if lists else -1)


def test_single_period_closed_form(oracle):
    """One tensor, used by kernels 0 and 9, equal slots of 100 ns, SSD only fast enough for one slot each way:
    absent slots 2..7, benefit = min(size, peak - cap) * 600, cost = 2 t."""
    lists = [[0]] + [[] for _ in range(8)] + [[0]]
    tr = traces.from_lists("one", lists, [50], [100] * 10, ssd_bw=500_000_000, host_bw=500_000_000)
    r = oracle.plan(tr, 20)
    assert r.status == "EXHAUSTED"             # slots 0, 1, 8, 9 still hold the tensor
    m = r.migrations[0]
    assert (m["absent_first"], m["absent_last"], m["transfer_ns"], m["dest"]) == (2, 7, 100, 0)
    assert r.win_benefit[0] == 30 * 600 and r.win_cost[0] == 200
    assert r.final_pressure.tolist() == [50, 50, 0, 0, 0, 0, 0, 0, 50, 50]


def test_host_capacity_limits_host_migrations(oracle):
    ex, tr = _example("B")
    r = oracle.plan(tr, ex["capacity"], host_capacity_bytes=7)     # the 8-byte tensor does not fit
    assert len(r.migrations) == 1 and r.migrations[0]["dest"] == 0
    r = oracle.plan(tr, ex["capacity"], host_capacity_bytes=8)
    assert len(r.migrations) == 2 and r.migrations[1]["dest"] == 1


def test_lazy_equals_plain_scaled_stress(oracle):
    tr = traces.config4_stress_dag(K=3000, N=12000)
    start, P0, peak, slot = oracle.timeline(tr)
    cap = tr.capacity_from_peak(peak)
    a = oracle.plan(tr, cap)
    b = oracle.plan(tr, cap, lazy=True)
    assert len(a.migrations) > 50
    assert np.array_equal(a.migrations, b.migrations) and np.array_equal(a.summary, b.summary)
    assert np.array_equal(a.final_pressure, b.final_pressure)
    _replay(oracle, tr, cap, a)


def _same_plan(a, b):
    return (np.array_equal(a.migrations, b.migrations) and np.array_equal(a.summary, b.summary)
            and np.array_equal(a.final_pressure, b.final_pressure))


def test_lazy_equals_plain_config3(oracle):
    """The lazy tier backs the GPU parity checks of the ViT-shaped trace: it has to give Algorithm 1's plan there."""
    tr = traces.make_config(3)
    start, P0, peak, slot = oracle.timeline(tr)
    cap = tr.capacity_from_peak(peak)
    a = oracle.plan(tr, cap)
    b = oracle.plan(tr, cap, lazy=True)
    assert len(a.migrations) > 1000 and _same_plan(a, b)


def test_lazy_equals_plain_stress_20k(oracle):
    """... and on the stress trace at K = 2*10^4, N = 8*10^4 (several scan tiles, periods hundreds of slots long),
    before it stands in for the plain tier at full size."""
    tr = traces.config4_stress_dag(K=20000, N=80000)
    start, P0, peak, slot = oracle.timeline(tr)
    cap = tr.capacity_from_peak(peak)
    a = oracle.plan(tr, cap)
    b = oracle.plan(tr, cap, lazy=True)
    assert len(a.migrations) > 1000 and _same_plan(a, b)
    _replay(oracle, tr, cap, a)


@pytest.mark.parametrize("cfg,ssd_bw,host_bw,cap_num,host_cap", [
    (1, 102_400_000_000, 32_000_000_000, 1, 0),
    (1, 6_400_000_000, 512_000_000_000, 1, 8 << 30),
    (2, 102_400_000_000, 512_000_000_000, 2, 0),
    (2, 3_200_000_000, 32_000_000_000, 1, 8 << 30),
    (2, 12_800_000_000, 512_000_000_000, 2, 8 << 30),
])
def test_lazy_equals_plain_on_the_sweep(oracle, cfg, ssd_bw, host_bw, cap_num, host_cap):
    """Points of the bandwidth / capacity / host-memory sweep that the GPU parity test checks against the lazy tier
    (fast SSD, fast host link, finite host memory, half the usual capacity): same plan from both tiers."""
    tr = traces.make_config(cfg)
    cap = tr.capacity_from_peak(0) // cap_num
    a = oracle.plan(tr, cap, host_bw=host_bw, ssd_bw=ssd_bw, host_capacity_bytes=host_cap)
    b = oracle.plan(tr, cap, host_bw=host_bw, ssd_bw=ssd_bw, host_capacity_bytes=host_cap, lazy=True)
    assert len(a.migrations) > 100 and _same_plan(a, b)
