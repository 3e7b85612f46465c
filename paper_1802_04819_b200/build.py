"""Compile the CUDA library in-tree with nvcc for sm_100a."""

from __future__ import annotations

import subprocess
from pathlib import Path

PKG = Path(__file__).resolve().parent
ROOT = PKG.parent
CSRC = PKG / "csrc"
LIB = PKG / "libslaq.so"
SOURCES = ["slaq_api.cu", "slaq_fit.cu", "slaq_gain.cu", "slaq_alloc.cu", "slaq_select_free.cu"]


# Instrumented builds of the same sources, each a library of its own beside libslaq.so.
VARIANTS = {
    "clocks": ["-DSLAQ_PHASE_CLOCKS"],     # the fit kernel times its phases (slaq_get_fit_phase_cycles)
    "bounds": ["-DSLAQ_DEBUG_BOUNDS"],     # every ring, pool, gain, segment and shared-slice index is checked
}


def variant_path(name: str) -> Path:
    return PKG / f"libslaq_{name}.so"


def nvcc_command(verbose_ptxas: bool = False, out: Path = LIB, defines=()) -> list[str]:
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-I", str(ROOT / "include"), "-Xcompiler", "-fPIC", "-shared", "-o", str(out), *defines]
    if verbose_ptxas:
        cmd += ["-Xptxas", "-v"]
    return cmd + [str(CSRC / s) for s in SOURCES]


def build_variant(name: str, force: bool = False) -> Path:
    """Compile an instrumented build (see VARIANTS) to libslaq_<name>.so."""
    out = variant_path(name)
    if force or is_stale(out):
        subprocess.run(nvcc_command(out=out, defines=VARIANTS[name]), check=True)
    return out


def is_stale(lib: Path = LIB) -> bool:
    if not lib.exists():
        return True
    built = lib.stat().st_mtime
    deps = list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + [ROOT / "include" / "slaq.h"]
    return any(d.stat().st_mtime > built for d in deps)


def build(force: bool = False, verbose_ptxas: bool = False) -> Path:
    if force or verbose_ptxas or is_stale():
        subprocess.run(nvcc_command(verbose_ptxas), check=True)
    return LIB


if __name__ == "__main__":
    build(force=True, verbose_ptxas=True)
