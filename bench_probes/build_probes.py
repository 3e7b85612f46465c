"""Compile the stand-alone measurement programs that back the roofline figures (sm_100a, nvcc).

    python bench_probes/build_probes.py

fp64_issue_probe   issue rate of the fp64 pipe by operand pattern (the roofline's denominator)
fit_sweep_probe    the fit kernel's sweep function in a loop of its own (what the instruction mix allows)
"""

from __future__ import annotations

import subprocess
from pathlib import Path

HERE = Path(__file__).resolve().parent
ROOT = HERE.parent
CSRC = ROOT / "paper_1802_04819_b200" / "csrc"
PROGRAMS = ["fp64_issue_probe", "fit_sweep_probe"]


def build_probes(verbose_ptxas: bool = False) -> list[Path]:
    out = []
    for name in PROGRAMS:
        cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-I", str(CSRC),
               "-o", str(HERE / name), str(HERE / f"{name}.cu")]
        if verbose_ptxas:
            cmd += ["-Xptxas", "-v"]
        subprocess.run(cmd, check=True)
        out.append(HERE / name)
    return out


if __name__ == "__main__":
    for path in build_probes(verbose_ptxas=True):
        print(path)
