"""Compile the CUDA library in-tree with nvcc for sm_100a."""

from __future__ import annotations

import subprocess
from pathlib import Path

PKG = Path(__file__).resolve().parent
ROOT = PKG.parent
CSRC = PKG / "csrc"
LIB = PKG / "libslaq.so"
SOURCES = ["slaq_api.cu", "slaq_fit.cu", "slaq_gain.cu", "slaq_alloc.cu"]


def nvcc_command(verbose_ptxas: bool = False) -> list[str]:
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-I", str(ROOT / "include"), "-Xcompiler", "-fPIC", "-shared", "-o", str(LIB)]
    if verbose_ptxas:
        cmd += ["-Xptxas", "-v"]
    return cmd + [str(CSRC / s) for s in SOURCES]


PROBE = PKG / "fp64_issue_probe"


def build_probe() -> Path:
    """Compile the stand-alone fp64 issue-rate probe (csrc/fp64_issue_probe.cu) next to the library."""
    subprocess.run(["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
                    "-o", str(PROBE), str(CSRC / "fp64_issue_probe.cu")], check=True)
    return PROBE


def is_stale() -> bool:
    if not LIB.exists():
        return True
    built = LIB.stat().st_mtime
    deps = list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + [ROOT / "include" / "slaq.h"]
    return any(d.stat().st_mtime > built for d in deps)


def build(force: bool = False, verbose_ptxas: bool = False) -> Path:
    if force or verbose_ptxas or is_stale():
        subprocess.run(nvcc_command(verbose_ptxas), check=True)
    return LIB


if __name__ == "__main__":
    build(force=True, verbose_ptxas=True)
    build_probe()
