"""The two forms of the fit's sweep agree on the GPU: the library's (powers of x by running sums, one change of basis per
sweep) against the one kept in the timing program (powers of x multiplied out point by point).  They share the model
evaluation and nothing of the accumulation, so a wrong coefficient of the change of basis, a wrong origin of a lane or a
row walked twice shows as a difference far above rounding."""

import re
import subprocess
import sys
from pathlib import Path

import pytest

pytestmark = pytest.mark.gpu

ROOT = Path(__file__).resolve().parent.parent


def test_running_sums_equal_the_multiplied_out_sums():
    sys.path.insert(0, str(ROOT / "bench_probes"))
    import build_probes
    build_probes.build_probes()
    out = subprocess.run([str(ROOT / "bench_probes" / "fit_sweep_probe"), "8"], check=True, capture_output=True,
                         text=True, timeout=300).stdout
    worst = [float(x) for x in re.findall(r"largest relative difference of a sum from the library's sweep: (\S+)", out)]
    assert len(worst) == 5, out            # one per lanes-per-job setting (2, 4, 8, 16, 32)
    # measured: 6e-16 to 6e-14 (the library steps x by one addition per row, the other form multiplies the running
    # index out, so the two evaluate the model a few 1e-15 apart in x); a wrong coefficient shows as 1e-3 or more
    assert max(worst) < 1e-11, worst
