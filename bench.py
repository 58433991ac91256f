#!/usr/bin/env python
"""Benchmark of the G10 planning path on B200.

Headline (`value`): trace events per second through the analysis passes S1-S3 -- slot clock, tensor vitality
and pressure timeline, i.e. one g10_vitality call with its timeline output (the e2e leg: the same call through host pointers) -- on the
1M-kernel / 4M-tensor stress trace (config 4), the largest single-GPU workload and the only one whose arrays are large enough
for an HBM fraction to mean something.  A step is one such pass with the trace resident in HBM; the L2 is flushed
between steps.  Second headline (`plan_ms`): one whole g10_plan_migrations call (S1-S7) on the ResNet-152-shaped
trace (config 1).  The same line carries the plan of every configuration (`plans`), the two analysis calls on a
trace four and eight times the size (`scale`), the calls behind the plan (prefetch pass, instruction stream, batched and
cyclic planning), the roofline of the passes and the CPU oracle timed beside them.  Prints ONE JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--quick | --passes-only]

With N > 1 (torchrun) every rank works on its own replica of the trace (the path does not shard: the greedy loop
is a strict sequence); value is the aggregate over ranks, time the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2310_09443_b200 import traces  # noqa: E402

WORKLOAD = "config4_stress_dag"
PLAN_WORKLOAD = "config1_resnet152_b256"
L2_FLUSH_BYTES = 512 << 20
# DRAM bytes per call on the stress trace (dram__bytes_read.sum + dram__bytes_write.sum summed over the call's kernels), from
# the one-pass ncu capture whose command and table are in profiles/passes_config4_stress.md (the capture that leaves the
# caches alone between launches, as this program does: the write-back of the L2 flush's dirty lines is part of it).
# "sources_sha256" is the hash of the kernel sources at the time of the capture: when the sources have changed since, the
# bench line says so ("traffic_stale") instead of passing old traffic off as current, and a CPU test warns.
TRAFFIC = {"vitality": 227_100_000, "timeline": 117_800_000, "timeline_given": 135_500_000, "fused": 337_200_000, "captured_at": "2026-11-25",
           "sources_sha256": "ebb78cb31457e2e2a3b2906af1e995c64e1459826260a1eb9c5a0bb878efadf8"}


PASS_SOURCES = ("g10_passes.cu", "g10_vitality_buckets.cu")     # the kernels of g10_vitality and g10_pressure_timeline


def kernel_sources_sha256():
    """Hash of the sources that hold the kernels of the two analysis calls (what the stored traffic was measured on)."""
    import hashlib
    h = hashlib.sha256()
    d = os.path.join(ROOT, "paper_2310_09443_b200", "csrc")
    for f in PASS_SOURCES:
        h.update(f.encode())
        with open(os.path.join(d, f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi (every 20 ms, a process of its own: a sampling thread in this
    process would delay the launches) from some untimed steps before the timed region to its end.  The timed region of the
    default run lasts a few milliseconds, less than nvidia-smi needs to come up: it is started a moment earlier, the same
    step runs untimed until it has answered a few times, and the timed steps follow at once."""

    def __init__(self, gpu_index: int):
        self.rows = []
        self.proc = None
        self.gpu_index = gpu_index

    def start(self):
        q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + q,
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def count(self) -> int:
        return len(self.rows)

    def stop(self, first_timed_row: int = 0):
        """first_timed_row: how many rows there were when the timed region began (the rest came during it)."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        in_timed = len(self.rows) - first_timed_row
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0])); mx = float(r[1])
            except ValueError:
                continue
            for nm, val in zip(names, r[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm), "samples_in_timed_region": max(0, in_timed),
                "window": "untimed steps right before the timed region and the timed region itself"}




def pass_bytes(K, N, E, uses, periods):
    """Algorithmic bytes of the two analysis calls.  Vitality reads kernel_ptr (8K) and kernel_tensors (4E) and writes
    first/last/num_uses (12N), use_ptr (8N), uses (4E'), period_ptr (8N) and the periods (12 Pn); the timeline reads
    kernel_ns (8K), tensor_bytes (8N), first/last (8N), the global flag (N) and writes start (8K) and pressure (8K)."""
    return 8 * K + 4 * E + 28 * N + 4 * uses + 12 * periods, 24 * K + 17 * N


def oracle_s123(O, tr):
    """One pass S1-S3 of the CPU oracle: vitality, slot clock and the plain definition of the pressure."""
    v = O.vitality(tr.kernel_ptr, tr.kernel_tensors, tr.N)
    start, P0, peak, slot = O.timeline(tr)
    return v, peak


def run_reference(args):
    """The CPU oracle as it stands, timed on the host cores (rank 0 only): the same metric on the same workload.
    A step is one whole pass S1-S3 over the stress trace (about five seconds on one core)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import g10_oracle as O
    O.build()
    tr = traces.config4_stress_dag()
    steps, warm = max(1, min(args.steps, 12)), max(0, min(args.warmup, 1))      # bounded: the whole run ends within minutes
    for _ in range(warm):
        oracle_s123(O, tr)
    t0 = time.perf_counter()
    for _ in range(steps):
        v, peak = oracle_s123(O, tr)
    dt = time.perf_counter() - t0
    value = tr.E * steps / dt
    t1 = time.perf_counter()
    tr1 = traces.config1_resnet152()
    r = O.plan(tr1, tr1.capacity_from_peak(0))
    plan_ms = (time.perf_counter() - t1) * 1e3
    line = {
        "impl": "reference", "metric": "trace_events_per_s", "value": value, "unit": "events/s", "n_gpus": args.gpus,
        "steps": steps, "warmup": warm, "ms_per_step": dt / steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "trace_sha256": tr.sha256(), "K": tr.K, "N": tr.N, "E": tr.E,
                   "uses": int(len(v.uses)), "periods": int(len(v.period_tensor)),
                   "steps_note": "steps and warm-up bounded to 12 and 1: a step takes seconds on one core"},
        "cpu_baseline": {"value": value, "unit": "events/s", "cores": 1, "kind": "oracle",
                         "sample": "%d whole passes S1-S3 over config 4" % steps, "cpu_model": cpu_model()},
        "e2e": {"value": value, "unit": "events/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "plan_ms": plan_ms, "plan_workload": PLAN_WORKLOAD, "plan_migrations": int(r.summary[0]),
    }
    print(json.dumps(line))


def max_over_ranks(torch, dist, world, ms, device):
    """Per-rank device time (ms) -> the slowest rank's (the job's time)."""
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_events_per_s(world, events_per_step, steps, total_ms):
    """Replicas only: every rank processes its own copy of the trace, so the job's throughput is the sum."""
    return world * events_per_step * steps / (total_ms / 1e3)


def timed(torch, fn, steps, warmup, flush):
    """CUDA-event times (ms) of `steps` calls of fn on the current stream; `flush` (a buffer larger than the L2, or
    None) is rewritten before every call, outside the event pair."""
    for _ in range(warmup):
        if flush is not None:
            flush.fill_(1)
        fn()
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in evs:
        if flush is not None:
            flush.fill_(1)
        a.record()
        fn()
        b.record()
    torch.cuda.synchronize()
    return [a.elapsed_time(b) for a, b in evs]


def time_calls(torch, fn, steps, warmup, flush):
    """Sum of the timed calls, in seconds."""
    return sum(timed(torch, fn, steps, warmup, flush)) / 1e3


def roofline(nbytes, seconds, peak, peak_kind, **extra):
    gbs = nbytes / seconds / 1e9
    d = {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak, "frac_of_nominal_8000": gbs / 8000.0,
         "algorithmic_bytes": nbytes, "peak_kind": peak_kind}
    d.update(extra)
    return d


def replicate_trace(torch, binding, tb, times):
    """The same trace `times` times back to back on the device (kernels, tensors and events of copy r follow those of copy
    r - 1; tensor ids shifted by r * N): the stress trace scaled up for the roofline measurement."""
    K, N, E = tb.K, tb.N, tb.E
    kptr = torch.cat([tb.kernel_ptr[:-1] + r * E for r in range(times)] + [torch.tensor([times * E], dtype=torch.int64, device=tb.kernel_ptr.device)])
    kt = torch.cat([tb.kernel_tensors + r * N for r in range(times)])
    nbytes = tb.tensor_bytes.repeat(times)
    ns = tb.kernel_ns.repeat(times)
    glob = tb.tensor_global.repeat(times) if tb.tensor_global is not None else None
    return binding.TraceBuffers(kptr, kt, nbytes, ns, glob, K=times * K, N=times * N, E=times * E)


def scaled_passes(torch, binding, tb, times, flush, hbm_peak, peak_kind, reps=5):
    """g10_vitality and g10_pressure_timeline alone on the stress trace replicated `times` times: with the fixed cost of
    a call (launches, phase chains of tens of microseconds) spread over `times` as many events, what is left is throughput."""
    big = replicate_trace(torch, binding, tb, times)
    ws = torch.empty(binding.g10_workspace_bytes(binding.WS_PLAN, big.K, big.N, big.E), dtype=torch.uint8, device=tb.kernel_ptr.device)
    v = binding.g10_vitality(big, ws=ws)
    tl = binding.g10_pressure_timeline(big, ws=ws)
    torch.cuda.synchronize()
    uses, periods = int(v.counts[0].item()), int(v.counts[1].item())
    vb, tlb = pass_bytes(big.K, big.N, big.E, uses, periods)
    out = {"times": times, "K": big.K, "N": big.N, "E": big.E, "uses": uses, "periods": periods,
           "device_status": int(v.counts[2].item()) | int(tl.status.item()), "repetitions": reps,
           "peak_bytes_is_that_of_one_copy": True}
    fl = (v.first_use.clone(), v.last_use.clone())          # (as in the headline step: first / last use handed over to the timeline call)
    del v, tl
    for name, fn, nb in (("vitality", lambda: binding.g10_vitality(big, ws=ws), vb),
                         ("timeline", lambda: binding.g10_pressure_timeline(big, ws=ws, first_last=fl), tlb)):
        cold = float(np.median(timed(torch, fn, reps, 2, flush)))
        warm = float(np.median(timed(torch, fn, reps, 2, None)))
        out[name + "_ms"] = cold
        out[name + "_ms_warm_l2"] = warm
        out[name + "_roofline"] = roofline(nb, cold / 1e3, hbm_peak, peak_kind)
    # both analyses from one call, as in the headline step
    vf = binding.g10_vitality(big, ws=ws, timeline=True)
    fused = float(np.median(timed(torch, lambda: binding.g10_vitality(big, ws=ws, out=vf, timeline=vf.timeline), reps, 2, flush)))
    out["s123_one_call_ms"] = fused
    out["events_per_s"] = big.E / (fused / 1e3)
    out["roofline"] = roofline(vb + tlb, fused / 1e3, hbm_peak, peak_kind)
    out["timeline_note"] = "timeline_ms: first / last use handed over from an earlier vitality call; events_per_s and roofline: both analyses from one g10_vitality call, as in the headline step"
    del big, ws, fl, vf
    torch.cuda.empty_cache()
    return out


def plan_stats(torch, binding, tr, dev, flush, steps, warm, stage=False):
    """Whole g10_plan_migrations calls on one trace (capacity from the trace's own recipe, applied to the peak this
    library computed): median and spread of `steps` timed calls after `warm` warm-up calls."""
    tb = binding.upload(tr, dev)
    ws = torch.empty(binding.g10_workspace_bytes(binding.WS_PLAN, tb.K, tb.N, tb.E), dtype=torch.uint8, device=dev)
    tl = binding.g10_pressure_timeline(tb, ws=ws)
    torch.cuda.synchronize()
    cap = tr.capacity_from_peak(int(tl.peak_bytes.item()))
    plan = binding.g10_plan_migrations(tb, cap, tr.host_bw, tr.ssd_bw, ws=ws)
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(5)] if stage else None
    if ev:
        for e in ev:
            e.record()                      # (an event owns a handle only once it has been recorded)
    loop_ms = []

    def call():
        binding.g10_plan_migrations(tb, cap, tr.host_bw, tr.ssd_bw, ws=ws, out=plan, stage_events=ev)

    ms = []
    for i in range(warm + steps):
        flush.fill_(1)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); call(); b.record(); b.synchronize()
        if i >= warm:
            ms.append(a.elapsed_time(b))
            if stage:
                loop_ms.append(ev[3].elapsed_time(ev[4]))
    s = plan.summary.cpu().numpy()
    out = {"K": tr.K, "N": tr.N, "E": tr.E, "plan_ms": float(np.median(ms)), "plan_ms_min": float(min(ms)), "plan_ms_max": float(max(ms)),
           "timed_calls": steps, "warmup_calls": warm, "migrations": int(s[0]), "iterations": int(s[1]), "status": binding.STATUS.get(int(s[2]), "?"),
           "device_status": int(s[7]), "capacity_bytes": int(cap), "us_per_iteration": float(np.median(ms)) * 1e3 / max(int(s[1]), 1)}
    if stage:
        out["greedy_loop_ms"] = float(np.median(loop_ms))
        out["greedy_loop_us_per_iteration"] = float(np.median(loop_ms)) * 1e3 / max(int(s[1]), 1)
    return out, (tb, ws, plan, tl, cap)


def run_ours(args):
    import torch
    from paper_2310_09443_b200 import binding, build

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the planner has no CPU path")
    torch.cuda.set_device(local)
    dev = "cuda:%d" % local
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl")
        if local == 0:
            build.build()                   # one build per node; the others wait for it
        dist.barrier()
    build.build()
    binding.load_library()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    hbm_peak, peak_kind = measured_peaks()
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)

    # ---- the headline: S1-S3 (one g10_vitality + one g10_pressure_timeline call) on the stress trace, device-resident
    tr = traces.config4_stress_dag()
    tb = binding.upload(tr, dev)
    ws = torch.empty(binding.g10_workspace_bytes(binding.WS_PLAN, tb.K, tb.N, tb.E), dtype=torch.uint8, device=dev)
    v = binding.g10_vitality(tb, ws=ws)
    tl = binding.g10_pressure_timeline(tb, ws=ws)
    torch.cuda.synchronize()
    assert int(v.counts[2].item()) == 0 and int(tl.status.item()) == 0, "device status"
    uses, periods = int(v.counts[0].item()), int(v.counts[1].item())
    K, N, E = tr.K, tr.N, tr.E
    vit_bytes, tl_bytes = pass_bytes(K, N, E, uses, periods)

    def step():
        # (one call gives both analyses: the vitality kernel that writes first / last use books every tensor's size on its
        # way, so that the events are walked once and only the slot clock and the pressure scan are left; the e2e leg
        # below and `passes.vitality_ms` / `passes.timeline_ms` time the two calls on their own)
        binding.g10_vitality(tb, ws=ws, out=v, timeline=tl)

    for _ in range(args.warmup):
        flush.fill_(1)
        step()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    # (more untimed steps, paced by the GPU, until the sampler has answered a few times -- at most half a second; every rank
    # does the same so that the ranks stay under the same load)
    t_settle = time.time()
    while time.time() - t_settle < 0.5 and (rank != 0 or sampler.proc is None or sampler.count() < 4 or time.time() - t_settle < 0.1):
        flush.fill_(1)
        step()
        torch.cuda.synchronize()
        if rank == 0 and sampler.proc is None:
            break
    barrier()
    first_timed_row = sampler.count()
    launches0 = binding.g10_launch_count()
    total_ms = 0.0
    for _ in range(args.steps):
        flush.fill_(1)                      # L2 flush between timed iterations (outside the event pair)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        step()
        b.record()
        b.synchronize()
        total_ms += a.elapsed_time(b)
    gpu_launches = binding.g10_launch_count() - launches0
    barrier()
    clocks = sampler.stop(first_timed_row) if rank == 0 else None
    total_ms = max_over_ranks(torch, dist, world, total_ms, dev)
    value = aggregate_events_per_s(world, E, args.steps, total_ms)
    step_s = total_ms / args.steps / 1e3

    # ---- the same pass end to end through the host-pointer form of the calls: the library stages the trace (H2D) and
    # copies every output back (D2H) inside the timed region
    tbh = binding.pin(tr)
    wsh = torch.empty(binding.g10_workspace_bytes(binding.WS_PLAN, K, N, E, binding.MEM_HOST), dtype=torch.uint8, device=dev)

    outs = [None, None]                                               # pinned result buffers, allocated by the first call

    def step_host():
        # (synchronous: results are in host memory on return; one call, as in the device-resident step: the trace is staged once)
        outs[0] = binding.g10_vitality(tbh, ws=wsh, device=dev, out=outs[0], timeline=outs[1] if outs[1] is not None else True)
        outs[1] = outs[0].timeline
        return outs[0], outs[1]

    e2e_steps = max(3, args.steps // 4)
    for _ in range(2):
        step_host()
    barrier()
    e2e_ms = 0.0
    for _ in range(e2e_steps):
        flush.fill_(1)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        vh, th = step_host()
        b.record()
        b.synchronize()
        e2e_ms += a.elapsed_time(b)
    assert int(vh.counts[0]) == uses and int(th.peak_bytes) == int(tl.peak_bytes.item())
    e2e_ms = max_over_ranks(torch, dist, world, e2e_ms, dev)
    e2e_value = aggregate_events_per_s(world, E, e2e_steps, e2e_ms)
    h2d = tbh.nbytes()                                                # the one call stages the trace once
    d2h = (12 * N + 16 * (N + 1) + 4 * uses + 12 * periods + 24) + (8 * (K + 1) + 8 * K + 8 + 4 + 8)
    del tbh, wsh, vh, th, outs

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- each call on its own (cold and warm L2), for the per-call rooflines
    reps = max(5, args.steps)
    vit_cold = float(np.median(timed(torch, lambda: binding.g10_vitality(tb, ws=ws), reps, 3, flush)))
    tl_cold = float(np.median(timed(torch, lambda: binding.g10_pressure_timeline(tb, ws=ws), reps, 3, flush)))
    tlg_cold = float(np.median(timed(torch, lambda: binding.g10_pressure_timeline(tb, ws=ws, first_last=(v.first_use, v.last_use)), reps, 3, flush)))
    fused_cold = float(np.median(timed(torch, lambda: binding.g10_vitality(tb, ws=ws, out=v, timeline=tl), reps, 3, flush)))
    vit_warm = float(np.median(timed(torch, lambda: binding.g10_vitality(tb, ws=ws), reps, 3, None)))
    tl_warm = float(np.median(timed(torch, lambda: binding.g10_pressure_timeline(tb, ws=ws), reps, 3, None)))
    sha = kernel_sources_sha256()
    stale = sha != TRAFFIC["sources_sha256"]
    traffic_note = {"captured_at": TRAFFIC["captured_at"], "sources_sha256_at_capture": TRAFFIC["sources_sha256"],
                    "sources_sha256_now": sha, "traffic_stale": stale}
    roof = roofline(vit_bytes + tl_bytes, step_s, hbm_peak, peak_kind,
                    kernel="S1-S3 in one call, g10_vitality with its timeline output: k_seg_scan<0> (slot clock), k_bk_hist, k_bk_scatter, "
                           "k_bk_emit<true> (uses, periods and the bookings of the tensors' sizes), k_seg_scan<1> (pressure, peak)",
                    dominant_kernel="k_bk_emit", traffic=TRAFFIC["fused"], traffic_note=traffic_note,
                    ms=step_s * 1e3, algorithmic_bytes_per_event=(vit_bytes + tl_bytes) / E,
                    roofline_events_per_s=E / ((vit_bytes + tl_bytes) / (hbm_peak * 1e9)),
                    note="random accesses of the passes are bound by the L2's rate of scattered 32-byte sector requests "
                         "(about 170 G/s measured on this part), not by HBM bytes")
    passes = {"vitality_ms": vit_cold, "timeline_ms": tl_cold, "vitality_ms_warm_l2": vit_warm, "timeline_ms_warm_l2": tl_warm,
              "vitality_roofline": roofline(vit_bytes, vit_cold / 1e3, hbm_peak, peak_kind, traffic=TRAFFIC["vitality"]),
              "timeline_roofline": roofline(tl_bytes, tl_cold / 1e3, hbm_peak, peak_kind, traffic=TRAFFIC["timeline"]),
              "timeline_after_vitality_ms": tlg_cold,
              "s123_one_call_ms": fused_cold,
              "timeline_after_vitality_roofline": roofline(tl_bytes, tlg_cold / 1e3, hbm_peak, peak_kind, traffic=TRAFFIC["timeline_given"]),
              "timeline_note": "timeline_ms: first / last use derived from the trace (k_first_last_pairs); timeline_after_vitality_ms: "
                               "handed over from an earlier vitality call; the timed step gets both analyses from one g10_vitality call",
              "repetitions": reps, "l2": "flushed between timed calls (the *_warm_l2 figures: not flushed)"}

    if args.passes_only:                   # (small profiling target: the headline and the per-call figures only)
        print(json.dumps({"metric": "trace_events_per_s", "value": value, "unit": "events/s", "ms_per_step": step_s * 1e3, "steps": args.steps,
                          "config": {"workload": WORKLOAD, "K": K, "N": N, "E": E}, "passes": passes, "roofline": roof, "gpu_launches": gpu_launches}))
        return

    # ---- whole plans, every configuration (median of >= 3 timed calls after warm-up; config 1 with stage events)
    plans = {}
    kept = None
    for cfg in range(5):
        trc = tr if cfg == 4 else traces.make_config(cfg)
        n_t, n_w = (3, 1) if cfg == 4 else (max(5, args.steps) if cfg == 1 else 5, 3)
        st, state = plan_stats(torch, binding, trc, dev, flush, n_t, n_w, stage=(cfg == 1))
        plans["config%d" % cfg] = st
        if cfg in (1, 4):
            kept = kept or {}
            kept[cfg] = (trc,) + state
        else:
            del state
    plan1 = plans["config1"]

    extras = {}
    if not args.quick:
        # ---- the calls behind the plan (Section 4.4) on the finished plans of config 1 and config 4
        for cfg in (1, 4):
            trc, tbc, wsc, planc, tlc, capc = kept[cfg]
            n_mig = int(planc.summary[0].item())
            pws = torch.empty(max(256, binding.g10_workspace_bytes(binding.WS_PREFETCH, trc.K, 0, n_mig)), dtype=torch.uint8, device=dev)
            pf_ms = []
            for _ in range(4):                                        # (the pass rewrites the pressure curve it is given: a fresh copy per call)
                P = planc.final_pressure.clone()
                flush.fill_(1)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                pf = binding.g10_schedule_prefetch(trc.K, n_mig, planc.migrations, tlc.kernel_start_ns, tbc.tensor_bytes, capc, P, ws=pws)
                b.record()
                torch.cuda.synchronize()
                pf_ms.append(a.elapsed_time(b))
            assert int(pf.summary[4].item()) == 0, "device status of the prefetch pass"
            vc = binding.g10_vitality(tbc, ws=wsc)
            torch.cuda.synchronize()

            def emit():
                return binding.g10_emit_instructions(trc.K, trc.N, vc.first_use, vc.last_use, tbc.tensor_bytes, tbc.tensor_global,
                                                     tlc.kernel_start_ns, n_mig, planc.migrations, pf.new_prefetch_issue_ns)

            em_ms = float(np.median(timed(torch, emit, 3, 1, flush)))
            em = emit()
            torch.cuda.synchronize()
            n_inst = int(em.counts[0].item())
            em_bytes = 17 * trc.N + 56 * n_mig + 32 * n_inst + 8 * (trc.K + 2)
            extras["config%d" % cfg] = {
                "prefetch_pass": {"ms": float(np.median(pf_ms[1:])), "moved": int(pf.summary[0].item()), "slots_regained": int(pf.summary[1].item()),
                                  "records": n_mig, "note": "median of 3 calls after one warm-up, L2 flushed, each on a fresh copy of the plan's pressure curve"},
                "instruction_stream": {"ms": em_ms, "instructions": n_inst, "device_status": int(em.counts[1].item()),
                                       "roofline": roofline(em_bytes, em_ms / 1e3, hbm_peak, peak_kind),
                                       "note": "the binding allocates the record buffer inside the timed call"}}
            del pf, em, vc, P, pws
        # ---- batched re-planning of config 1: one variant per SM, kernel durations jittered by +-10 % (seeded), variant 0 unperturbed
        trc, tbc, wsc, planc, tlc, capc = kept[1]
        sms = torch.cuda.get_device_properties(dev).multi_processor_count
        rng = np.random.default_rng(20231009)
        base_v = dict(gpu_capacity_bytes=capc, host_bw=trc.host_bw, ssd_bw=trc.ssd_bw)
        variants = [base_v]
        for _ in range(sms - 1):
            f = rng.uniform(0.9, 1.1, size=trc.K)
            dur = np.maximum(1, np.rint(trc.kernel_ns.astype(np.float64) * f)).astype(np.int64)
            variants.append(dict(base_v, kernel_ns=torch.from_numpy(dur).to(dev)))
        wsb = torch.empty(binding.g10_workspace_bytes(binding.WS_BATCH, tbc.K, tbc.N, tbc.E), dtype=torch.uint8, device=dev)
        mcap = int(planc.summary[0].item()) + 64
        b_ms = float(np.median(timed(torch, lambda: binding.g10_plan_batch(tbc, variants, ws=wsb, migrations_cap=mcap), 5, 3, flush)))
        bo = binding.g10_plan_batch(tbc, variants, ws=wsb, migrations_cap=mcap)
        torch.cuda.synchronize()
        stab = bo.stability.cpu().numpy().astype(np.float64)
        extras["batch_replan"] = {"workload": PLAN_WORKLOAD, "variants": len(variants), "ms": b_ms, "plans_per_s": len(variants) / (b_ms / 1e3),
                                  "trace_events_per_s": len(variants) * trc.E / (b_ms / 1e3), "jitter": "+-10 % per kernel, seeded",
                                  "mean_jaccard_vs_unperturbed": float(np.mean(stab[1:, 0] / np.maximum(stab[1:, 1], 1))),
                                  "device_status_or": int(np.bitwise_or.reduce(bo.summary.cpu().numpy()[:, 7]))}
        del wsb, bo, variants
        # ---- steady-state (cyclic) plan of config 1
        c_ms = float(np.median(timed(torch, lambda: binding.g10_plan_cyclic(tbc, capc, trc.host_bw, trc.ssd_bw, ws=wsc), 5, 3, flush)))
        cp = binding.g10_plan_cyclic(tbc, capc, trc.host_bw, trc.ssd_bw, ws=wsc)
        torch.cuda.synchronize()
        cs = cp.summary.cpu().numpy()
        extras["cyclic_plan"] = {"workload": PLAN_WORKLOAD, "plan_ms": c_ms, "migrations": int(cs[0]), "status": binding.STATUS.get(int(cs[2]), "?"),
                                 "final_peak_bytes": int(cs[3]), "final_peak_bytes_acyclic": int(planc.summary[3].item()), "device_status": int(cs[7])}
        del cp
    kept = None
    torch.cuda.empty_cache()

    # ---- the two analysis calls on the stress trace eight (and four) times over: fixed cost against throughput
    scale = {}
    if not args.quick:
        for times in (4, 8):
            scale["x%d" % times] = scaled_passes(torch, binding, tb, times, flush, hbm_peak, peak_kind)

    line = {
        "metric": "trace_events_per_s", "value": value, "unit": "events/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": step_s * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "step": "S1-S3: one g10_vitality call with its timeline output (uses, periods, slot clock, pressure, peak), trace resident in HBM",
                   "trace_sha256": tr.sha256(), "K": K, "N": N, "E": E, "uses": uses, "periods": periods,
                   "l2": "flushed between timed iterations (%d MiB write)" % (L2_FLUSH_BYTES >> 20),
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "plan_ms": plan1["plan_ms"], "plan_workload": PLAN_WORKLOAD,
        "plan_greedy_loop": {"kernel": "k_plan_one", "bound": "latency", "ms": plan1.get("greedy_loop_ms"),
                             "us_per_iteration": plan1.get("greedy_loop_us_per_iteration"), "iterations": plan1["iterations"],
                             "note": "the planner state of this workload lives in the shared memory of one SM: a chain of dependent "
                                     "iterations (search, rescore, commit); reported per iteration, an HBM fraction would mean nothing"},
        "plans": plans,
        "passes": passes,
        "e2e": {"value": e2e_value, "unit": "events/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms / e2e_steps, "steps": e2e_steps,
                "note": "host-pointer form of the same one call: it stages the trace (pinned host memory) and copies every output of both analyses back"},
        "gpu_launches": gpu_launches,
        "gpu_launches_note": "counted by the library itself (g10_launch_count before and after the timed region): its own kernels only, "
                             "%d per step; memset nodes and the L2 flush are not counted" % (gpu_launches // max(args.steps, 1)),
        "clocks": clocks,
        "roofline": roof,
        "behind_the_plan": extras,
        "scale": scale,
    }
    line["cpu_baseline"] = cpu_baseline(tr)
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def cpu_model():
    try:
        with open("/proc/cpuinfo") as f:
            for ln in f:
                if ln.lower().startswith("model name"):
                    return ln.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def cpu_baseline(tr):
    """The oracle on the same workload, one thread: three whole passes S1-S3 over the stress trace (about fifteen seconds),
    then the config-1 plan with both of its tiers."""
    from oracle import g10_oracle as O
    O.build()
    t0 = time.perf_counter()
    reps = 3
    for _ in range(reps):
        oracle_s123(O, tr)
    dt = time.perf_counter() - t0
    tr1 = traces.config1_resnet152()
    cap = tr1.capacity_from_peak(0)
    ts, tl_ = [], []
    for _ in range(3):
        t1 = time.perf_counter(); O.plan(tr1, cap); ts.append(time.perf_counter() - t1)
        t1 = time.perf_counter(); O.plan(tr1, cap, lazy=True); tl_.append(time.perf_counter() - t1)
    return {"value": tr.E * reps / dt, "unit": "events/s", "cores": 1, "kind": "oracle",
            "sample": "%d whole passes S1-S3 (vitality, slot clock, plain-definition pressure) over config 4 in %.1f s" % (reps, dt),
            "ms_per_step": dt / reps * 1e3, "plan_ms_config1_plain_tier": sorted(ts)[1] * 1e3, "plan_ms_config1_lazy_tier": sorted(tl_)[1] * 1e3,
            "host_cores_available": os.cpu_count(), "cpu_model": cpu_model()}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)      # (0.3 ms each with the L2 flush: long enough for a few clock samples)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--quick", action="store_true", help="headline, plans and per-call rooflines only")
    ap.add_argument("--passes-only", action="store_true", help="headline and per-call rooflines only (small profiling target)")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
