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


# ------------------------------------------------------------------------------------------------
# The calls behind the plan (Section 4.4) on steady-state plans: eager prefetch pass and instruction stream.
# ------------------------------------------------------------------------------------------------
def _stream_rows(oracle, e, K):
    rows = []
    for b in range(K + 1):
        for j in range(int(e.inst_ptr[b]), int(e.inst_ptr[b + 1])):
            i = e.instructions[j]
            rows.append([b, oracle.OPCODES[int(i["opcode"])], int(i["tensor"]), int(i["target"]), int(i["record"]),
                         int(i["bytes"]), int(i["time_ns"])])
    return rows


def test_hand_worked_wrap_around_downstream(oracle):
    ex = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "cyclic_example.json")))
    tr = traces.from_lists("cyc", ex["kernel_lists"], ex["tensor_bytes"], ex["kernel_ns"], ex["tensor_global"],
                           host_bw=ex["host_bw"], ssd_bw=ex["ssd_bw"], capacity_bytes=ex["capacity"])
    start, P0, peak, slot = oracle.timeline(tr)
    v = oracle.vitality(tr.kernel_ptr, tr.kernel_tensors, tr.N)
    r = oracle.plan_cyclic(tr, ex["capacity"])
    pf = oracle.schedule_prefetch(tr.K, r.migrations, start, tr.tensor_bytes, ex["capacity"], r.final_pressure)
    assert pf.order.tolist() == ex["prefetch"]["order"] and pf.new_absent_last.tolist() == ex["prefetch"]["new_absent_last"]
    assert pf.new_prefetch_issue_ns.tolist() == ex["prefetch"]["new_prefetch_issue_ns"] and pf.summary.tolist() == ex["prefetch"]["summary"]
    e = oracle.emit_instructions(tr.K, v.first_use, v.last_use, tr.tensor_bytes, tr.tensor_global, start, r.migrations, pf.new_prefetch_issue_ns)
    assert e.inst_ptr.tolist() == ex["instruction_stream"]["inst_ptr"]
    assert _stream_rows(oracle, e, tr.K) == ex["instruction_stream"]["instructions"]


def _mirror_prefetch(plan, pressure, start, tensor_bytes, cap, K):
    """Dense restatement on a timeline unrolled twice: slot k and slot k + K are kept equal by writing both, so that
    no index is ever reduced modulo K; the visiting order comes from the position of the prefetch inside the iteration."""
    T = start[K]
    P2 = list(pressure) + list(pressure)
    start2 = list(start) + [start[k] + T for k in range(1, K + 1)]
    order = sorted(range(len(plan)), key=lambda i: (plan[i]["prefetch_issue_ns"] - (T if plan[i]["prefetch_issue_ns"] >= T else 0), i))
    new_last, new_issue = [None] * len(plan), [None] * len(plan)
    for i in order:
        m = plan[i]
        s = int(tensor_bytes[m["tensor"]])
        j = m["absent_last"] + 1
        while j - 1 >= m["absent_first"] and P2[j - 1] + s <= cap:
            j -= 1
        for k in range(j, m["absent_last"] + 1):
            P2[k] += s
            P2[k + K if k < K else k - K] += s
        new_last[i] = j - 1
        new_issue[i] = start2[j] if j <= m["absent_last"] else m["prefetch_issue_ns"]
    assert P2[:K] == P2[K:]
    return order, new_last, new_issue, P2[:K]


def _dense_stream(tr, uses, start, plan, issue):
    """Boundary by boundary, kind by kind, tensor by tensor: does this instruction stand here?"""
    K, T = tr.K, start[tr.K]
    rows = []
    for b in range(K + 1):
        for op in (0, 1, 2, 3):                                   # FREE, PRE_EVICT, ALLOC, PREFETCH
            for i in range(tr.N):
                glob = bool(tr.tensor_global[i])
                if op == 2 and uses[i] and b == (0 if glob else uses[i][0]):
                    rows.append((b, 2, i, -1, -1, int(tr.tensor_bytes[i]), start[b]))
                if op == 0 and uses[i] and not glob and b == uses[i][-1] + 1:
                    rows.append((b, 0, i, -1, -1, int(tr.tensor_bytes[i]), start[b]))
                for r, m in enumerate(plan):
                    if m["tensor"] != i:
                        continue
                    if op == 1 and start[b] == m["evict_issue_ns"]:
                        rows.append((b, 1, i, m["dest"], r, int(tr.tensor_bytes[i]), m["evict_issue_ns"]))
                    if op == 3:
                        t = issue[r] - T if issue[r] >= T else issue[r]
                        if start[b] <= t and (b == K or start[b + 1] > t):
                            rows.append((b, 3, i, -1, r, int(tr.tensor_bytes[i]), t))
    return rows


def test_downstream_of_cyclic_plans_against_dense(oracle):
    rng = np.random.default_rng(4242)
    wrapped = moved = 0
    for trial in range(300):
        K = int(rng.integers(2, 12)); N = int(rng.integers(1, 7))
        tr = traces.random_toy(rng, K, N, max_bytes=3000, max_ns=300)
        if trial % 3 != 1:
            tr.tensor_global = np.ones(N, np.uint8)
        start, P0, peak, slot = oracle.timeline(tr)
        v = oracle.vitality(tr.kernel_ptr, tr.kernel_tensors, tr.N)
        uses = helpers.brute_vitality(tr)[0]
        cap = peak * int(rng.integers(3, 10)) // 10
        r = oracle.plan_cyclic(tr, cap)
        plan = [{f: int(m[f]) for f in FIELDS} for m in r.migrations]
        st = [int(x) for x in start]
        # (the pass is also run with more room than the plan had, so that prefetches, wrap-around ones too, do move)
        for cap2 in (cap, cap + int(tr.tensor_bytes.max())):
            pf = oracle.schedule_prefetch(tr.K, r.migrations, start, tr.tensor_bytes, cap2, r.final_pressure)
            order, new_last, new_issue, P = _mirror_prefetch(plan, [int(x) for x in r.final_pressure], st, tr.tensor_bytes, cap2, K)
            assert pf.order.tolist() == order and pf.new_absent_last.tolist() == new_last and pf.new_prefetch_issue_ns.tolist() == new_issue
            assert pf.pressure.tolist() == P
            for issue in (None, pf.new_prefetch_issue_ns):
                e = oracle.emit_instructions(tr.K, v.first_use, v.last_use, tr.tensor_bytes, tr.tensor_global, start, r.migrations, issue)
                ref = _dense_stream(tr, uses, st, plan, [m["prefetch_issue_ns"] for m in plan] if issue is None else new_issue)
                got = [(b, int(i["opcode"]), int(i["tensor"]), int(i["target"]), int(i["record"]), int(i["bytes"]), int(i["time_ns"]))
                       for b in range(K + 1) for i in e.instructions[int(e.inst_ptr[b]):int(e.inst_ptr[b + 1])]]
                assert got == ref and int(e.inst_ptr[K + 1]) == len(ref)
            moved += sum(1 for i, m in enumerate(plan) if new_last[i] < m["absent_last"] and m["absent_last"] >= K)
        wrapped += sum(1 for m in plan if m["absent_last"] >= K or m["prefetch_issue_ns"] >= st[K])
    assert wrapped > 20 and moved > 3        # wrap-around periods occur, and some of their prefetches do move
