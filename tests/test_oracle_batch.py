"""Pins for the oracle's batched re-planning (the planner side of the paper's sensitivity studies, Section 5):
every variant must be the plan of the perturbed trace on its own (checked against the dense brute force), and the
stability pairs must obey the set identities."""
import copy

import numpy as np

import helpers
from paper_2310_09443_b200 import traces


def jitter(rng, dur, pct):
    f = rng.uniform(1.0 - pct / 100.0, 1.0 + pct / 100.0, size=len(dur))
    return np.maximum(1, np.rint(np.asarray(dur, dtype=np.float64) * f)).astype(np.int64)


def test_variants_are_independent_plans(oracle):
    rng = np.random.default_rng(31337)
    for trial in range(25):
        K = int(rng.integers(3, 14)); N = int(rng.integers(2, 8))
        tr = traces.random_toy(rng, K, N, max_bytes=4000, max_ns=3000)
        start, P0, peak, slot = oracle.timeline(tr)
        cap = peak * int(rng.integers(2, 9)) // 10
        variants = [dict(gpu_capacity_bytes=cap, host_bw=tr.host_bw, ssd_bw=tr.ssd_bw)]
        for pct in (5, 25):
            variants.append(dict(gpu_capacity_bytes=cap, host_bw=tr.host_bw, ssd_bw=tr.ssd_bw, kernel_ns=jitter(rng, tr.kernel_ns, pct)))
        variants.append(dict(gpu_capacity_bytes=cap, host_bw=tr.host_bw, ssd_bw=tr.ssd_bw * 5))
        variants.append(dict(gpu_capacity_bytes=cap, host_bw=tr.host_bw, ssd_bw=tr.ssd_bw, host_capacity_bytes=int(rng.integers(1, 6000))))
        variants.append(dict(gpu_capacity_bytes=max(cap // 2, 1), host_bw=tr.host_bw * 2, ssd_bw=tr.ssd_bw))
        for lazy in (False, True):
            got = oracle.plan_batch(tr, variants, lazy=lazy)
            sets = []
            for v, r in zip(variants, got.plans):
                tv = copy.copy(tr)
                if v.get("kernel_ns") is not None:
                    tv.kernel_ns = v["kernel_ns"]
                ref = helpers.brute_plan(tv, v["gpu_capacity_bytes"], v["host_bw"], v["ssd_bw"], v.get("host_capacity_bytes", 0))
                assert [m["period"] for m in ref["plan"]] == r.migrations["period"].tolist()
                assert [m["dest"] for m in ref["plan"]] == r.migrations["dest"].tolist()
                assert ref["final_pressure"] == r.final_pressure.tolist() and ref["status"] == r.status
                sets.append(set(m["period"] for m in ref["plan"]))
            for j, s in enumerate(sets):
                assert got.stability[j].tolist() == [len(s & sets[0]), len(s | sets[0])]


def test_stability_identities_on_config0(oracle):
    tr = traces.config0_mlp_chain()
    start, P0, peak, slot = oracle.timeline(tr)
    cap = tr.capacity_from_peak(peak)
    rng = np.random.default_rng(9)
    base = dict(gpu_capacity_bytes=cap, host_bw=tr.host_bw, ssd_bw=tr.ssd_bw)
    variants = [base, dict(base), dict(base, kernel_ns=jitter(rng, tr.kernel_ns, 10)), dict(base, ssd_bw=tr.host_bw)]
    got = oracle.plan_batch(tr, variants)
    n = [len(r.migrations) for r in got.plans]
    assert got.stability[0].tolist() == [n[0], n[0]] and got.stability[1].tolist() == [n[0], n[0]]      # an identical variant
    for j in range(len(variants)):
        inter, union = got.stability[j]
        assert inter <= min(n[0], n[j]) and union == n[0] + n[j] - inter
    # the pair is symmetric in the two plans: swap base and variant
    swapped = oracle.plan_batch(tr, [variants[2], variants[0]])
    assert swapped.stability[1].tolist() == got.stability[2].tolist()
