"""CPU-side checks of the CUDA library: it builds, loads and exports the whole C ABI."""

import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    import paper_1802_04819_b200 as slaq
    slaq.build()
    return slaq.load_library()


def test_every_declared_symbol_is_exported(lib):
    import paper_1802_04819_b200 as slaq
    header = (ROOT / "include" / "slaq.h").read_text()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(slaq_[a-z_]+)\s*\(", header))
    assert declared, "no declarations found"
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} is declared in slaq.h but not exported"
    assert declared == set(slaq.EXPORTED_SYMBOLS)


def test_binding_constants_match_the_header():
    """Parameter keys, job states and warning codes are typed twice (C header, Python binding)."""
    from paper_1802_04819_b200 import binding
    header = (ROOT / "include" / "slaq.h").read_text()
    values = {name: int(v) for name, v in re.findall(r"\b(SLAQ_[A-Z_]+)\s*=\s*(-?\d+)", header)}
    keys = [n for n in values if n.startswith("SLAQ_P_")]
    assert len(keys) >= 7
    for name in keys:
        assert getattr(binding, name[len("SLAQ_"):]) == values[name], name
    for name in [n for n in values if n.startswith("SLAQ_JOB_") or n.startswith("SLAQ_W_")]:
        assert getattr(binding, name[len("SLAQ_"):]) == values[name], name


def test_workspace_size_is_host_arithmetic(lib):
    import paper_1802_04819_b200 as slaq
    small = slaq.workspace_bytes(8, 20, 16)
    big = slaq.workspace_bytes(100_000, 1000, 64)
    assert 0 < small < big
    assert big >= 100_000 * 1000 * 8          # the ring pool alone
    assert slaq.workspace_bytes(0, 20, 16) == 0   # invalid sizes give 0
    assert slaq.workspace_bytes(8, 100_000, 16) == 0


def test_no_cpu_fallback(lib):
    import torch
    import paper_1802_04819_b200 as slaq
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(slaq.SlaqError):
        slaq.Scheduler(8, 20, 16)


def test_product_does_not_import_the_oracle():
    for path in (ROOT / "paper_1802_04819_b200").rglob("*"):
        if path.suffix in {".py", ".cu", ".cuh", ".h"}:
            text = path.read_text()
            assert "oracle" not in text.lower(), f"{path} mentions the oracle"
