"""Pins for the oracle's eager prefetch pass (Section 4.4): hand-worked example, dense restatement on toy traces,
invariants on the DNN-shaped configs."""
import json
import os

import numpy as np

import helpers
from paper_2310_09443_b200 import traces

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_worked_examples.json")


def test_hand_worked_prefetch_example(oracle):
    ex = json.load(open(GOLDEN))["examples"]["prefetch"]
    tr = traces.from_lists("p", ex["kernel_lists"], ex["tensor_bytes"], ex["kernel_ns"], host_bw=ex["host_bw"], ssd_bw=ex["ssd_bw"])
    start, P0, peak, slot = oracle.timeline(tr)
    assert P0.tolist() == ex["pressure"]
    r = oracle.plan(tr, ex["capacity"])
    assert r.status == ex["status"] and r.final_pressure.tolist() == ex["final_pressure"]
    assert [int(r.migrations[0][k]) for k in ("absent_first", "absent_last", "prefetch_issue_ns")] == [2, 5, 62]
    pf = oracle.schedule_prefetch(tr.K, r.migrations, start, tr.tensor_bytes, ex["capacity"], r.final_pressure)
    g = ex["prefetch_pass"]
    assert pf.order.tolist() == g["order"] and pf.new_absent_last.tolist() == g["new_absent_last"]
    assert pf.new_prefetch_issue_ns.tolist() == g["new_prefetch_issue_ns"]
    assert pf.pressure.tolist() == g["pressure"] and pf.summary.tolist() == g["summary"]


def test_prefetch_random_toys_against_dense(oracle):
    rng = np.random.default_rng(4242)
    moved = 0
    for trial in range(300):
        K = int(rng.integers(4, 18)); N = int(rng.integers(1, 9))
        tr = traces.random_toy(rng, K, N)
        start, P0, peak, slot = oracle.timeline(tr)
        for cap in (peak * 3 // 4, peak // 2, peak):
            b = helpers.brute_plan(tr, cap, tr.host_bw, tr.ssd_bw)
            r = oracle.plan(tr, cap)
            assert [int(m["period"]) for m in r.migrations] == [m["period"] for m in b["plan"]]
            order, nl, ni, P = helpers.brute_prefetch(b["plan"], b["final_pressure"], helpers.brute_start(tr), tr.tensor_bytes, cap)
            pf = oracle.schedule_prefetch(tr.K, r.migrations, start, tr.tensor_bytes, cap, r.final_pressure)
            assert pf.order.tolist() == order and pf.new_absent_last.tolist() == nl
            assert pf.new_prefetch_issue_ns.tolist() == ni and pf.pressure.tolist() == P
            moved += int(pf.summary[0])
    assert moved > 50


def _invariants(tr, cap, start, mig, P_before, pf):
    P_after = pf.pressure
    assert np.all(P_after >= P_before)
    changed = P_after != P_before
    assert np.all(P_after[changed] <= cap)                       # nothing is pushed above capacity
    nl = pf.new_absent_last
    assert np.all(nl <= mig["absent_last"]) and np.all(nl >= mig["absent_first"] - 1)
    s = tr.tensor_bytes[mig["tensor"]]
    assert int((P_after - P_before).astype(object).sum()) == int(((mig["absent_last"] - nl).astype(object) * s.astype(object)).sum())
    moved = nl < mig["absent_last"]
    assert np.array_equal(pf.new_prefetch_issue_ns[moved], start[nl[moved] + 1])
    assert np.array_equal(pf.new_prefetch_issue_ns[~moved], mig["prefetch_issue_ns"][~moved])
    assert np.all(pf.new_prefetch_issue_ns <= mig["prefetch_issue_ns"])
    key = mig["prefetch_issue_ns"][pf.order]
    assert np.all(np.diff(key) >= 0) and sorted(pf.order.tolist()) == list(range(len(mig)))


def test_prefetch_invariants_on_configs(oracle):
    for cfg in (0, 1, 2):
        tr = traces.make_config(cfg)
        start, P0, peak, slot = oracle.timeline(tr)
        cap = tr.capacity_from_peak(peak)
        r = oracle.plan(tr, cap, lazy=True)
        pf = oracle.schedule_prefetch(tr.K, r.migrations, start, tr.tensor_bytes, cap, r.final_pressure)
        _invariants(tr, cap, start, r.migrations, r.final_pressure, pf)
        # a plan that ends FIT leaves room: use a capacity well above the need on config 0 and see prefetches move
        if cfg == 0:
            r2 = oracle.plan(tr, peak * 9 // 10)
            pf2 = oracle.schedule_prefetch(tr.K, r2.migrations, start, tr.tensor_bytes, peak * 9 // 10, r2.final_pressure)
            _invariants(tr, peak * 9 // 10, start, r2.migrations, r2.final_pressure, pf2)
            assert r2.status == "FIT" and pf2.summary[0] > 0
