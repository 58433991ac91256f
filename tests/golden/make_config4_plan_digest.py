"""Writes tests/golden/config4_plan_digest.json: a digest of the CPU oracle's complete plan for the
full-size stress trace (config 4: 1e6 kernels, 4e6 tensors), of the eager prefetch pass over it and of the
instruction stream emitted from both.  The oracle's lazy tier needs about ten
minutes for it, too long for a test, so the GPU parity test compares its own plan with this digest.
Calls only the trace generator and the oracle.  Usage: python tests/golden/make_config4_plan_digest.py"""
import hashlib
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import g10_oracle as O  # noqa: E402
from paper_2310_09443_b200 import traces  # noqa: E402


def digest(migrations, final_pressure, summary):
    h = hashlib.sha256()
    h.update(migrations.tobytes())
    h.update(final_pressure.tobytes())
    h.update(summary[:7].tobytes())
    return h.hexdigest()


def main():
    tr = traces.config4_stress_dag()
    start, P0, peak, slot = O.timeline(tr)
    cap = tr.capacity_from_peak(peak)
    r = O.plan(tr, cap, lazy=True)
    pf = O.schedule_prefetch(tr.K, r.migrations, start, tr.tensor_bytes, cap, r.final_pressure)
    hp = hashlib.sha256()
    for a in (pf.order, pf.new_absent_last, pf.new_prefetch_issue_ns, pf.pressure, pf.summary):
        hp.update(a.tobytes())
    # the instruction stream (Section 4.4) of that plan with the eager prefetch times, field by field
    ov = O.vitality(tr.kernel_ptr, tr.kernel_tensors, tr.N)
    oe = O.emit_instructions(tr.K, ov.first_use, ov.last_use, tr.tensor_bytes, tr.tensor_global, start, r.migrations,
                             pf.new_prefetch_issue_ns)
    he = hashlib.sha256()
    he.update(np.ascontiguousarray(oe.inst_ptr).tobytes())
    for name in oe.instructions.dtype.names:
        he.update(np.ascontiguousarray(oe.instructions[name]).tobytes())
    out = {
        "_source": "oracle/g10_oracle.c, lazy tier, on paper_2310_09443_b200.traces.config4_stress_dag() (seed 4)",
        "trace_sha256": tr.sha256(), "peak_bytes": int(peak), "peak_slot": int(slot), "capacity_bytes": int(cap),
        "summary": [int(x) for x in r.summary[:7]], "status": r.status,
        "first_migrations": [[int(m[k]) for k in m.dtype.names] for m in r.migrations[:5]],
        "plan_sha256": digest(r.migrations, r.final_pressure, r.summary),
        "prefetch_summary": [int(x) for x in pf.summary], "prefetch_sha256": hp.hexdigest(),
        "num_instructions": int(len(oe.instructions)), "instruction_fields": list(oe.instructions.dtype.names),
        "instructions_sha256": he.hexdigest(),
    }
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "config4_plan_digest.json")
    with open(path, "w") as f:
        json.dump(out, f, indent=1)
    print(json.dumps(out))


if __name__ == "__main__":
    main()
