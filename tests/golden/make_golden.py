"""Write the stored expected values under tests/golden/.  Calls only the CPU oracle.

The paper prints no worked numeric example for this path (no table, and its figures carry
no values), so nothing here is the paper's; these files freeze the oracle's own output on
the smallest workload so that a later change to its arithmetic is seen, and so that the
GPU tests have one fixed reference that does not depend on rebuilding the oracle.

    python tests/golden/make_golden.py
"""

import json
import sys
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parents[2]
sys.path.insert(0, str(ROOT))

import oracle  # noqa: E402
from workloads import make_workload  # noqa: E402


def main():
    wl = make_workload(0)
    out = oracle.schedule(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, wl.epoch_seconds, wl.total_cores,
                          wl.max_cores_per_job)
    doc = {
        "source": "oracle/slaq_oracle.cpp on workloads.make_workload(0); written by tests/golden/make_golden.py",
        "alloc": out["alloc"].tolist(),
        "family": out["family"].tolist(),
        "M": [float.hex(v) for v in out["M"]],
        "R": [float.hex(v) for v in out["R"]],
        "gain_first_core": [float.hex(v) for v in out["gain"][:, 0]],
    }
    (Path(__file__).parent / "config0_oracle.json").write_text(json.dumps(doc, indent=1) + "\n")


if __name__ == "__main__":
    main()
