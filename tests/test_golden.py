"""The oracle must keep reproducing its stored output on the 8-job workload."""

import json
from pathlib import Path

import numpy as np

from workloads import make_workload


def test_oracle_reproduces_stored_config0(oracle_mod):
    doc = json.loads((Path(__file__).parent / "golden" / "config0_oracle.json").read_text())
    wl = make_workload(0)
    out = oracle_mod.schedule(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, wl.epoch_seconds, wl.total_cores,
                              wl.max_cores_per_job)
    assert out["alloc"].tolist() == doc["alloc"]
    assert out["family"].tolist() == doc["family"]
    np.testing.assert_array_equal(out["M"], [float.fromhex(v) for v in doc["M"]])
    # libm may differ by an ulp between machines in exp/log: allow 1e-12 on derived values
    np.testing.assert_allclose(out["R"], [float.fromhex(v) for v in doc["R"]], rtol=1e-12)
    np.testing.assert_allclose(out["gain"][:, 0], [float.fromhex(v) for v in doc["gain_first_core"]], rtol=1e-12)
