"""Pins for the oracle's instruction-stream emission (Section 4.4, Figure 9): the hand-worked stream of example A,
a dense restatement on toy traces, and structural invariants on the DNN-shaped configs."""
import json
import os

import numpy as np

import helpers
from paper_2310_09443_b200 import traces

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_worked_examples.json")


def _stream(oracle, e, K):
    rows = []
    for b in range(K + 1):
        for j in range(int(e.inst_ptr[b]), int(e.inst_ptr[b + 1])):
            i = e.instructions[j]
            rows.append([b, oracle.OPCODES[int(i["opcode"])], int(i["tensor"]), int(i["target"]), int(i["record"]),
                         int(i["bytes"]), int(i["time_ns"])])
    return rows


def test_hand_worked_stream(oracle):
    ex = json.load(open(GOLDEN))["examples"]["A"]
    tr = traces.from_lists("A", ex["kernel_lists"], ex["tensor_bytes"], ex["kernel_ns"], host_bw=ex["host_bw"], ssd_bw=ex["ssd_bw"])
    start, P0, peak, slot = oracle.timeline(tr)
    v = oracle.vitality(tr.kernel_ptr, tr.kernel_tensors, tr.N)
    r = oracle.plan(tr, ex["capacity"])
    e = oracle.emit_instructions(tr.K, v.first_use, v.last_use, tr.tensor_bytes, tr.tensor_global, start, r.migrations)
    assert e.inst_ptr.tolist() == ex["instruction_stream"]["inst_ptr"]
    assert _stream(oracle, e, tr.K) == ex["instruction_stream"]["instructions"]


def brute_stream(tr, uses, start, plan, new_issue=None):
    rows = []
    for i, u in enumerate(uses):
        if not u:
            continue
        glob = bool(tr.tensor_global[i])
        rows.append((0 if glob else u[0], 2, i, -1, -1, int(tr.tensor_bytes[i]), start[0 if glob else u[0]]))
        if not glob:
            rows.append((u[-1] + 1, 0, i, -1, -1, int(tr.tensor_bytes[i]), start[u[-1] + 1]))
    for r, m in enumerate(plan):
        b = start.index(m["evict_issue_ns"])
        rows.append((b, 1, m["tensor"], m["dest"], r, int(tr.tensor_bytes[m["tensor"]]), m["evict_issue_ns"]))
        t = m["prefetch_issue_ns"] if new_issue is None else new_issue[r]
        b = max(k for k in range(len(start)) if start[k] <= t)
        rows.append((b, 3, m["tensor"], -1, r, int(tr.tensor_bytes[m["tensor"]]), t))
    rows.sort(key=lambda x: (x[0], x[1], x[2]))
    return rows


def test_random_toys_against_dense(oracle):
    rng = np.random.default_rng(31337)
    total = 0
    for trial in range(200):
        K = int(rng.integers(2, 16)); N = int(rng.integers(1, 9))
        tr = traces.random_toy(rng, K, N)
        start, P0, peak, slot = oracle.timeline(tr)
        v = oracle.vitality(tr.kernel_ptr, tr.kernel_tensors, tr.N)
        uses, first, last, periods = helpers.brute_vitality(tr)
        cap = peak // 2
        b = helpers.brute_plan(tr, cap, tr.host_bw, tr.ssd_bw)
        r = oracle.plan(tr, cap)
        for eager in (False, True):
            ni = None
            bni = None
            if eager:
                pf = oracle.schedule_prefetch(tr.K, r.migrations, start, tr.tensor_bytes, cap, r.final_pressure)
                ni = pf.new_prefetch_issue_ns
                bni = helpers.brute_prefetch(b["plan"], b["final_pressure"], helpers.brute_start(tr), tr.tensor_bytes, cap)[2]
            e = oracle.emit_instructions(tr.K, v.first_use, v.last_use, tr.tensor_bytes, tr.tensor_global, start, r.migrations, ni)
            exp = brute_stream(tr, uses, helpers.brute_start(tr), b["plan"], bni)
            got = []
            for bd in range(tr.K + 1):
                for j in range(int(e.inst_ptr[bd]), int(e.inst_ptr[bd + 1])):
                    i = e.instructions[j]
                    got.append((bd, int(i["opcode"]), int(i["tensor"]), int(i["target"]), int(i["record"]), int(i["bytes"]), int(i["time_ns"])))
            assert got == exp
            assert int(e.inst_ptr[tr.K + 1]) == len(exp)
            total += len(exp)
    assert total > 2000


def test_stream_invariants_on_configs(oracle):
    for cfg in (0, 1, 2):
        tr = traces.make_config(cfg)
        start, P0, peak, slot = oracle.timeline(tr)
        v = oracle.vitality(tr.kernel_ptr, tr.kernel_tensors, tr.N)
        cap = tr.capacity_from_peak(peak)
        r = oracle.plan(tr, cap, lazy=True)
        e = oracle.emit_instructions(tr.K, v.first_use, v.last_use, tr.tensor_bytes, tr.tensor_global, start, r.migrations)
        ins = e.instructions
        used = v.first_use >= 0
        n_alloc = int((ins["opcode"] == 2).sum()); n_free = int((ins["opcode"] == 0).sum())
        assert n_alloc == int(used.sum()) and n_free == int((used & (tr.tensor_global == 0)).sum())
        assert int((ins["opcode"] == 1).sum()) == len(r.migrations) == int((ins["opcode"] == 3).sum())
        assert np.all(np.diff(e.inst_ptr) >= 0) and e.inst_ptr[0] == 0 and e.inst_ptr[-1] == len(ins)
        boundary = np.repeat(np.arange(tr.K + 1), np.diff(e.inst_ptr[:tr.K + 2]))
        # every tensor is allocated before (at the boundary of) its first use and freed right after its last
        al = ins["opcode"] == 2
        fu = v.first_use[ins["tensor"][al]]
        assert np.all(boundary[al] <= fu)
        fr = ins["opcode"] == 0
        assert np.array_equal(boundary[fr], v.last_use[ins["tensor"][fr]] + 1)
        # a pre-eviction sits at its period start, the matching prefetch later and before the next use
        ev = ins["opcode"] == 1; pf = ins["opcode"] == 3
        bev = np.zeros(len(r.migrations), np.int64); bpf = np.zeros(len(r.migrations), np.int64)
        bev[ins["record"][ev]] = boundary[ev]; bpf[ins["record"][pf]] = boundary[pf]
        assert np.all(bev < r.migrations["absent_first"]) and np.all(bpf == r.migrations["absent_last"] + 1)
        # order inside a boundary
        key = boundary.astype(np.int64) * (1 << 34) + ins["opcode"].astype(np.int64) * (1 << 31) + ins["tensor"]
        assert np.all(np.diff(key) > 0)
