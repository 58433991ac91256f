"""Independent checkers used by the tests: a dense brute-force restatement of the planning path for
toy traces (Python big integers, per-nanosecond bookkeeping, Fractions for ratios) and a plan
replayer that checks the invariants a valid plan must satisfy at any size.  Neither imports the
oracle nor the CUDA package."""
from __future__ import annotations

from fractions import Fraction

import numpy as np

SSD, HOST = 0, 1


# ------------------------------------------------------------------------------------------------
# Dense brute force (toy sizes only)
# ------------------------------------------------------------------------------------------------
def dense_matrix(tr):
    """used[k][i] = True iff kernel k lists tensor i (Section 4.2: inputs and outputs are active)."""
    used = [[False] * tr.N for _ in range(tr.K)]
    for k in range(tr.K):
        for e in range(int(tr.kernel_ptr[k]), int(tr.kernel_ptr[k + 1])):
            used[k][int(tr.kernel_tensors[e])] = True
    return used


def brute_vitality(tr):
    used = dense_matrix(tr)
    uses = [[k for k in range(tr.K) if used[k][i]] for i in range(tr.N)]
    first = [u[0] if u else -1 for u in uses]
    last = [u[-1] if u else -1 for u in uses]
    periods = []
    for i in range(tr.N):
        for u, v in zip(uses[i], uses[i][1:]):
            # inactive and not dead in every slot strictly between u and v; needs at least one slot
            if any(True for _ in range(u + 1, v)):
                periods.append((i, u, v))
    return uses, first, last, periods


def brute_pressure(tr, uses):
    P = []
    for k in range(tr.K):
        tot = 0
        for i in range(tr.N):
            if not uses[i]:
                continue
            if tr.tensor_global[i] or uses[i][0] <= k <= uses[i][-1]:
                tot += int(tr.tensor_bytes[i])
        P.append(tot)
    return P


def brute_start(tr):
    st = [0]
    for d in tr.kernel_ns:
        st.append(st[-1] + int(d))
    return st


def brute_geometry(tr, start, period, bw):
    """Per-nanosecond: mark which slots the eviction window [t_r, t_r+t) and the prefetch window
    [t_end-t, t_end) touch; absent slots are the slots of the period strictly between them."""
    i, u, v = period
    s = int(tr.tensor_bytes[i])
    t = -((-s * 10 ** 9) // bw)
    t_r, t_end = start[u + 1], start[v]
    if 2 * t > t_end - t_r:
        return dict(t=t, valid=False)

    def slot_of(ns):
        for k in range(tr.K):
            if start[k] <= ns < start[k + 1]:
                return k
        raise AssertionError

    ev = {}
    for ns in range(t_r, t_r + t):
        ev[slot_of(ns)] = ev.get(slot_of(ns), 0) + 1
    pf = {}
    for ns in range(t_end - t, t_end):
        pf[slot_of(ns)] = pf.get(slot_of(ns), 0) + 1
    absent = [k for k in range(u + 1, v) if k > max(ev) and k < min(pf)]
    if not absent:
        return dict(t=t, valid=False)
    return dict(t=t, valid=True, a_abs=absent[0], b_abs=absent[-1], ev=ev, pf=pf)


def brute_plan(tr, cap, host_bw, ssd_bw, host_capacity=0, max_iterations=0):
    """Algorithm 1 restated with dense loops."""
    uses, first, last, periods = brute_vitality(tr)
    start = brute_start(tr)
    P = brute_pressure(tr, uses)
    dur = [int(d) for d in tr.kernel_ns]
    K = tr.K
    geo = [[brute_geometry(tr, start, p, ssd_bw) for p in periods],
           [brute_geometry(tr, start, p, host_bw) for p in periods]]
    booked = {(X, d): [0] * K for X in (SSD, HOST) for d in ("out", "in")}
    hocc = [0] * K
    alive = [True] * len(periods)
    plan = []
    limit = len(periods) if max_iterations <= 0 else min(max_iterations, len(periods))
    it = 0
    rounds = 0
    while True:
        if max(P, default=0) <= cap:
            status = "ALREADY_FITS" if not plan else "FIT"
            break
        if it >= limit:
            status = "ITERATION_LIMIT" if limit < len(periods) else "EXHAUSTED"
            break
        rounds += 1
        best = None
        for p, (i, u, v) in enumerate(periods):
            if not alive[p]:
                continue
            s = int(tr.tensor_bytes[i])
            dest = None
            for X in (SSD, HOST):
                g = geo[X][p]
                if not g["valid"]:
                    continue
                if any(booked[(X, "out")][k] + n > dur[k] for k, n in g["ev"].items()):
                    continue
                if any(booked[(X, "in")][k] + n > dur[k] for k, n in g["pf"].items()):
                    continue
                if X == HOST and host_capacity and any(hocc[k] + s > host_capacity for k in range(u + 1, v)):
                    continue
                dest = X
                break
            if dest is None:
                continue
            g = geo[dest][p]
            benefit = sum(min(s, max(0, P[k] - cap)) * dur[k] for k in range(g["a_abs"], g["b_abs"] + 1))
            if benefit <= 0:
                continue
            ratio = Fraction(benefit, 2 * g["t"])
            if best is None or ratio > best[0]:
                best = (ratio, p, dest, benefit)
        if best is None:
            status = "EXHAUSTED"
            break
        _, p, dest, benefit = best
        i, u, v = periods[p]
        g = geo[dest][p]
        s = int(tr.tensor_bytes[i])
        for k in range(g["a_abs"], g["b_abs"] + 1):
            P[k] -= s
        for k, n in g["ev"].items():
            booked[(dest, "out")][k] += n
        for k, n in g["pf"].items():
            booked[(dest, "in")][k] += n
        if dest == HOST:
            for k in range(u + 1, v):
                hocc[k] += s
        alive[p] = False
        plan.append(dict(period=p, tensor=i, dest=dest, absent_first=g["a_abs"], absent_last=g["b_abs"], iteration=it,
                         evict_issue_ns=start[u + 1], prefetch_issue_ns=start[v] - g["t"], transfer_ns=g["t"],
                         benefit=benefit, cost=2 * g["t"]))
        it += 1
    pk = max(P, default=0)
    return dict(plan=plan, final_pressure=P, status=status, rounds=rounds,
                final_peak=(pk, P.index(pk) if P else -1), periods=periods)


# ------------------------------------------------------------------------------------------------
# Plan replay: invariants that hold at any size (numpy, exact Python ints where products get large)
# ------------------------------------------------------------------------------------------------
def check_plan_invariants(tr, cap, start, P0, vit, migrations, final_pressure, status, host_bw, ssd_bw,
                          win_benefit=None, host_capacity=0, check_area=True):
    """vit: object with period_tensor / period_prev_use / period_next_use; migrations: structured array."""
    K = tr.K
    dur = np.asarray(tr.kernel_ns, dtype=np.int64)
    start = np.asarray(start, dtype=np.int64)
    P = np.asarray(P0, dtype=np.int64).copy()
    busy = np.zeros((4, K), dtype=np.int64)
    hocc = np.zeros(K, dtype=np.int64)
    seen = set()

    def area(Pv):
        ex = np.maximum(Pv - cap, 0)
        return int(np.dot(ex.astype(object), dur.astype(object))) if K else 0

    A = area(P) if check_area else None
    for j, m in enumerate(migrations):
        p = int(m["period"]); X = int(m["dest"])
        assert p not in seen, "period migrated twice"
        seen.add(p)
        i = int(vit.period_tensor[p]); u = int(vit.period_prev_use[p]); v = int(vit.period_next_use[p])
        assert int(m["tensor"]) == i
        assert int(m["iteration"]) == j
        s = int(tr.tensor_bytes[i])
        bw = ssd_bw if X == SSD else host_bw
        t = -((-s * 10 ** 9) // bw)
        assert int(m["transfer_ns"]) == t
        a, b = u + 1, v - 1
        ap, bp = int(m["absent_first"]), int(m["absent_last"])
        # eviction slots [a, a'-1], absent slots [a', b'], prefetch slots [b'+1, b] tile the period
        assert u < a < ap <= bp < b < v
        t_r, t_end = int(start[a]), int(start[v])
        assert int(m["evict_issue_ns"]) == t_r and int(m["prefetch_issue_ns"]) == t_end - t
        assert t_r + t <= t_end - t
        # the windows end / begin exactly around the absent range
        assert start[ap - 1] < t_r + t <= start[ap]
        assert start[bp + 1] <= t_end - t < start[bp + 2]
        ks = np.arange(a, ap)
        ov = np.minimum(t_r + t, start[ks + 1]) - np.maximum(t_r, start[ks])
        assert ov.sum() == t
        busy[2 * X, a:ap] += ov
        ks = np.arange(bp + 1, b + 1)
        ov = np.minimum(t_end, start[ks + 1]) - np.maximum(t_end - t, start[ks])
        assert ov.sum() == t
        busy[2 * X + 1, bp + 1:b + 1] += ov
        assert np.all(busy[2 * X, a:ap] <= dur[a:ap]) and np.all(busy[2 * X + 1, bp + 1:b + 1] <= dur[bp + 1:b + 1])
        if X == HOST:
            hocc[a:b + 1] += s
            if host_capacity:
                assert hocc[a:b + 1].max() <= host_capacity
        if check_area or win_benefit is not None:
            ex = np.minimum(np.maximum(P[ap:bp + 1] - cap, 0), s)
            ben = int(np.dot(ex.astype(object), dur[ap:bp + 1].astype(object)))
            assert ben > 0, "a committed migration must relieve pressure above capacity"
            if win_benefit is not None:
                assert int(win_benefit[j]) == ben
        P[ap:bp + 1] -= s
        if check_area:
            A2 = area(P)
            assert A2 == A - ben, "excess-area identity"
            A = A2
        assert P[ap:bp + 1].min() >= 0
    assert np.array_equal(P, np.asarray(final_pressure, dtype=np.int64))
    if status == "FIT":
        assert len(migrations) > 0 and (P.max() if K else 0) <= cap
    if status == "ALREADY_FITS":
        assert len(migrations) == 0 and (P.max() if K else 0) <= cap
    if status in ("EXHAUSTED", "ITERATION_LIMIT"):
        assert (P.max() if K else 0) > cap
    return P, busy, hocc


# ------------------------------------------------------------------------------------------------
# Eager prefetch pass (Section 4.4), dense restatement
# ------------------------------------------------------------------------------------------------
def brute_prefetch(plan, pressure, start, tensor_bytes, cap):
    """plan: list of dicts as returned by brute_plan; returns (order, new_absent_last, new_issue, new pressure)."""
    P = list(pressure)
    order = sorted(range(len(plan)), key=lambda i: (plan[i]["prefetch_issue_ns"], i))
    new_last = [None] * len(plan)
    new_issue = [None] * len(plan)
    for i in order:
        m = plan[i]
        s = int(tensor_bytes[m["tensor"]])
        # earliest slot j such that the tensor fits in every slot j .. absent_last
        j = m["absent_last"] + 1
        while j - 1 >= m["absent_first"] and P[j - 1] + s <= cap:
            j -= 1
        for k in range(j, m["absent_last"] + 1):
            P[k] += s
        new_last[i] = j - 1
        new_issue[i] = start[j] if j <= m["absent_last"] else m["prefetch_issue_ns"]
    return order, new_last, new_issue, P


# ------------------------------------------------------------------------------------------------
# Steady-state (cyclic) planning, dense restatement for toy traces: the iteration repeats unchanged, a used global
# tensor has one more period from its last use to its first use one iteration later; every nanosecond of a transfer
# window is charged to the physical slot it falls in.
# ------------------------------------------------------------------------------------------------
def brute_plan_cyclic(tr, cap, host_bw, ssd_bw, host_capacity=0, max_iterations=0):
    uses, first, last, periods = brute_vitality(tr)
    K = tr.K
    periods = list(periods)
    for i in range(tr.N):
        if tr.tensor_global[i] and uses[i] and first[i] + K - last[i] >= 2:
            periods.append((i, last[i], first[i] + K))
    start = brute_start(tr)
    T = start[K] if K else 0
    dur = [int(d) for d in tr.kernel_ns]
    P = brute_pressure(tr, uses)

    def when(k):                                  # unrolled start time of unrolled slot k (k <= 2K)
        return start[k] if k <= K else start[k - K] + T

    def slot_at(ns):                              # unrolled slot holding unrolled nanosecond ns
        it, r = divmod(ns, T)
        for k in range(K):
            if start[k] <= r < start[k + 1]:
                return k + it * K
        raise AssertionError

    def geometry(period, bw):
        i, u, v = period
        s = int(tr.tensor_bytes[i])
        t = -((-s * 10 ** 9) // bw)
        t_r, t_end = when(u + 1), when(v)
        if 2 * t > t_end - t_r:
            return dict(t=t, valid=False)
        ev, pf = {}, {}
        for ns in range(t_r, t_r + t):
            ev[slot_at(ns)] = ev.get(slot_at(ns), 0) + 1
        for ns in range(t_end - t, t_end):
            pf[slot_at(ns)] = pf.get(slot_at(ns), 0) + 1
        absent = [k for k in range(u + 1, v) if k > max(ev) and k < min(pf)]
        if not absent:
            return dict(t=t, valid=False)
        return dict(t=t, valid=True, a_abs=absent[0], b_abs=absent[-1], ev=ev, pf=pf)

    geo = [[geometry(p, ssd_bw) for p in periods], [geometry(p, host_bw) for p in periods]]
    booked = {(X, d): [0] * K for X in (SSD, HOST) for d in ("out", "in")}
    hocc = [0] * K
    alive = [True] * len(periods)
    plan = []
    limit = len(periods) if max_iterations <= 0 else min(max_iterations, len(periods))
    it = rounds = 0
    while True:
        if max(P, default=0) <= cap:
            status = "ALREADY_FITS" if not plan else "FIT"
            break
        if it >= limit:
            status = "ITERATION_LIMIT" if limit < len(periods) else "EXHAUSTED"
            break
        rounds += 1
        best = None
        for p, (i, u, v) in enumerate(periods):
            if not alive[p]:
                continue
            s = int(tr.tensor_bytes[i])
            dest = None
            for X in (SSD, HOST):
                g = geo[X][p]
                if not g["valid"]:
                    continue
                if any(booked[(X, "out")][k % K] + n > dur[k % K] for k, n in g["ev"].items()):
                    continue
                if any(booked[(X, "in")][k % K] + n > dur[k % K] for k, n in g["pf"].items()):
                    continue
                if X == HOST and host_capacity and any(hocc[k % K] + s > host_capacity for k in range(u + 1, v)):
                    continue
                dest = X
                break
            if dest is None:
                continue
            g = geo[dest][p]
            benefit = sum(min(s, max(0, P[k % K] - cap)) * dur[k % K] for k in range(g["a_abs"], g["b_abs"] + 1))
            if benefit <= 0:
                continue
            ratio = Fraction(benefit, 2 * g["t"])
            if best is None or ratio > best[0]:
                best = (ratio, p, dest)
        if best is None:
            status = "EXHAUSTED"
            break
        _, p, dest = best
        i, u, v = periods[p]
        g = geo[dest][p]
        s = int(tr.tensor_bytes[i])
        for k in range(g["a_abs"], g["b_abs"] + 1):
            P[k % K] -= s
        for k, n in g["ev"].items():
            booked[(dest, "out")][k % K] += n
        for k, n in g["pf"].items():
            booked[(dest, "in")][k % K] += n
        if dest == HOST:
            for k in range(u + 1, v):
                hocc[k % K] += s
        alive[p] = False
        plan.append(dict(period=p, tensor=i, dest=dest, absent_first=g["a_abs"], absent_last=g["b_abs"], iteration=it,
                         evict_issue_ns=when(u + 1), prefetch_issue_ns=when(v) - g["t"], transfer_ns=g["t"]))
        it += 1
    pk = max(P, default=0)
    return dict(plan=plan, final_pressure=P, status=status, rounds=rounds, periods=periods,
                final_peak=(pk, P.index(pk) if P else -1))
