"""Pins for the oracle's steady-state (cyclic) planner: a hand-worked example with a wrap-around period, the dense
per-nanosecond restatement on toy traces, and the reduction to the ordinary planner when nothing is global."""
import json
import os

import numpy as np

import helpers
from paper_2310_09443_b200 import traces

FIELDS = ("period", "tensor", "dest", "absent_first", "absent_last", "iteration", "evict_issue_ns", "prefetch_issue_ns", "transfer_ns")


def test_hand_worked_wrap_around(oracle):
    ex = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "cyclic_example.json")))
    tr = traces.from_lists("cyc", ex["kernel_lists"], ex["tensor_bytes"], ex["kernel_ns"], ex["tensor_global"],
                           host_bw=ex["host_bw"], ssd_bw=ex["ssd_bw"], capacity_bytes=ex["capacity"])
    start, P0, peak, slot = oracle.timeline(tr)
    assert P0.tolist() == ex["unplanned_pressure"]
    r = oracle.plan_cyclic(tr, ex["capacity"])
    assert r.periods.tolist() == ex["periods"]
    assert [{f: int(m[f]) for f in FIELDS} for m in r.migrations] == ex["migrations"]
    assert r.final_pressure.tolist() == ex["final_pressure"] and r.summary[:7].tolist() == ex["summary"]
    # the ordinary planner cannot touch the weight: one migration only
    assert len(oracle.plan(tr, ex["capacity"]).migrations) == 1


def test_toys_against_dense_cycle(oracle):
    rng = np.random.default_rng(2718)
    wrapped = 0
    for trial in range(300):
        K = int(rng.integers(2, 12)); N = int(rng.integers(1, 7))
        tr = traces.random_toy(rng, K, N, max_bytes=3000, max_ns=300)
        if trial % 3 == 0:
            tr.tensor_global = np.ones(N, np.uint8)
        start, P0, peak, slot = oracle.timeline(tr)
        cap = peak * int(rng.integers(1, 10)) // 10
        hc = int(rng.integers(0, 2)) * int(rng.integers(1, 6000))
        mi = int(rng.integers(0, 2)) * int(rng.integers(1, 4))
        ref = helpers.brute_plan_cyclic(tr, cap, tr.host_bw, tr.ssd_bw, hc, mi)
        got = oracle.plan_cyclic(tr, cap, host_capacity_bytes=hc, max_iterations=mi)
        assert got.periods.tolist() == [list(p) for p in ref["periods"]]
        assert [{f: int(m[f]) for f in FIELDS} for m in got.migrations] == ref["plan"]
        assert got.final_pressure.tolist() == ref["final_pressure"] and got.status == ref["status"]
        assert int(got.summary[1]) == ref["rounds"] and (int(got.summary[3]), int(got.summary[4])) == ref["final_peak"]
        wrapped += sum(1 for m in ref["plan"] if m["absent_last"] >= K or m["prefetch_issue_ns"] >= int(start[K]))
    assert wrapped > 20          # the toys do exercise periods that reach into the next iteration


def test_without_global_tensors_it_is_the_ordinary_plan(oracle):
    rng = np.random.default_rng(99)
    for trial in range(40):
        tr = traces.random_toy(rng, int(rng.integers(1, 30)), int(rng.integers(1, 20)), max_deg=4)
        tr.tensor_global = np.zeros(tr.N, np.uint8)
        start, P0, peak, slot = oracle.timeline(tr)
        cap = peak * int(rng.integers(1, 10)) // 10
        a = oracle.plan(tr, cap); c = oracle.plan_cyclic(tr, cap)
        assert np.array_equal(a.migrations, c.migrations) and np.array_equal(a.final_pressure, c.final_pressure)
        assert np.array_equal(a.summary, c.summary)
    tr = traces.config0_mlp_chain()                      # with globals the cycle offers more: never a worse final peak here
    start, P0, peak, slot = oracle.timeline(tr)
    cap = tr.capacity_from_peak(peak)
    assert oracle.plan_cyclic(tr, cap).summary[3] <= oracle.plan(tr, cap).summary[3]
