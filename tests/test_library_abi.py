"""CPU-side checks of the boundary: the shared library builds, loads and exports every symbol the
public header declares, and the binding refuses to run without a GPU instead of falling back."""
import re
from pathlib import Path

import pytest
import torch

from paper_2405_19715_b200 import specdec

ROOT = Path(__file__).resolve().parent.parent


def _declared_symbols():
    text = (ROOT / "include" / "specdec.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(specdec_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = specdec.load_library()
    names = _declared_symbols()
    assert set(names) == set(specdec.EXPORTS), names
    for n in names:
        assert hasattr(lib, n), n


def test_no_cpu_fallback():
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    with pytest.raises(RuntimeError):
        specdec.Context(4, 4)


def test_product_path_does_not_import_the_oracle():
    for f in (ROOT / "paper_2405_19715_b200").rglob("*"):
        if f.suffix in (".py", ".cu", ".cuh", ".h"):
            assert not re.search(r"^\s*(from|import)\s+oracle|oracle/|#include.*oracle", f.read_text(), flags=re.M), f
    assert "paper_2405_19715_b200" not in (ROOT / "oracle" / "specdec_oracle.py").read_text()
