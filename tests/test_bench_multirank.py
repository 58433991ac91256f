"""The N > 1 bookkeeping of bench.py ("replicas only": every rank plans its own copy of the trace, no data-path
collective): max over ranks of the per-rank time and the aggregate throughput, run as two gloo ranks on CPU."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    import torch, torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    ms = 10.0 * (rank + 1)                       # rank 1 is the slow one
    total = bench.max_over_ranks(torch, dist, world, ms, "cpu")
    value = bench.aggregate_events_per_s(world, 5268, 4, total)
    assert abs(total - 20.0) < 1e-9, total
    assert abs(value - world * 5268 * 4 / 0.020) < 1e-6, value
    dist.barrier()
    dist.destroy_process_group()
    print("rank", rank, "ok")
""") % ROOT


def test_two_rank_aggregation(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29577")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                          "--master-addr", "127.0.0.1", "--master-port", "29577", str(script)],
                         env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stdout + out.stderr
    assert out.stdout.count("ok") == 2


def test_reference_arm_runs_on_cpu():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "3"],
                         capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr
    import json
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == "trace_events_per_s" and line["value"] > 0
    assert line["config"]["workload"] == "config4_stress_dag" and line["plan_workload"] == "config1_resnet152_b256" and line["cpu_baseline"]["kind"] == "oracle"


def test_traffic_constants_carry_the_hash_of_the_sources_they_were_captured_on():
    """The DRAM traffic in the bench line is a stored ncu figure: it is tagged with the hash of the kernel sources it was
    captured on, and a bench line on other sources says "traffic_stale".  A stale tag is reported here as a warning."""
    import warnings

    sys.path.insert(0, ROOT)
    import bench

    now = bench.kernel_sources_sha256()
    assert len(now) == 64 and int(now, 16) >= 0
    assert set(bench.TRAFFIC) == {"vitality", "timeline", "timeline_given", "fused", "captured_at", "sources_sha256"}
    assert len(bench.TRAFFIC["sources_sha256"]) == 64, "the traffic constants carry no source hash"
    assert bench.TRAFFIC["vitality"] > 0 and bench.TRAFFIC["timeline"] > 0
    if now != bench.TRAFFIC["sources_sha256"]:
        warnings.warn("kernel sources changed since the DRAM traffic in bench.py was captured: re-capture it "
                      "(profiles/passes_config4_stress.md has the command)")
