"""The stand-alone measurement programs and the instrumented library builds must compile (nvcc cross-compiles for
sm_100a without a GPU); nothing is run here."""

import sys
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent


def test_measurement_programs_compile():
    sys.path.insert(0, str(ROOT / "bench_probes"))
    import build_probes
    built = build_probes.build_probes()
    assert {p.name for p in built} == {"fp64_issue_probe", "fit_sweep_probe"}
    assert all(p.exists() and p.stat().st_size > 0 for p in built)


def test_instrumented_builds_compile_and_export_the_same_symbols():
    import ctypes
    import paper_1802_04819_b200 as slaq
    from paper_1802_04819_b200.build import VARIANTS, build_variant
    assert set(VARIANTS) == {"bounds", "clocks"}
    for name in VARIANTS:
        lib = ctypes.CDLL(str(build_variant(name)))
        for symbol in slaq.EXPORTED_SYMBOLS:
            assert hasattr(lib, symbol), f"{symbol} missing from the {name} build"
