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


def test_every_context_entry_point_makes_the_contexts_gpu_current():
    """Source-level check of the rule stated in specdec.h: every exported call that takes a context and touches
    the GPU selects the context's device first (directly or through its argument checker)."""
    csrc = ROOT / "paper_2405_19715_b200" / "csrc"
    text = "\n".join((csrc / f).read_text() for f in ("api.cu", "head.cu"))
    exempt = {"specdec_create", "specdec_destroy", "specdec_last_error", "specdec_launch_count", "specdec_last_kernel",
              "specdec_set_phase_stamps", "specdec_head_launch_mode", "specdec_use_device", "specdec_verify_correct_topk_forward"}
    found = 0
    for m in re.finditer(r"^(?:extern \"C\" )?(?:int|uint64_t|const char\*) (specdec_[a-z_]+)\(([^)]*)\)\s*\{", text, flags=re.M):
        name, args = m.group(1), m.group(2)
        if name in exempt or "specdec_ctx* ctx" not in args:
            continue
        depth, i = 1, m.end()
        while depth and i < len(text):
            depth += {"{": 1, "}": -1}.get(text[i], 0)
            i += 1
        body = text[m.end():i]
        assert re.search(r"specdec_use_device\(ctx\)|check_verify_args\(ctx|check_shard_args\(ctx|specdec_verify_correct\(ctx", body), name
        found += 1
    assert found >= 12
