"""CPU checks of the boundary: the library loads and exports every symbol the header declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "matkv.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(matkv_[a-z0-9_]+)\s*\(", src)))


def test_header_symbols_are_exported_and_bound():
    import __graft_entry__ as ge
    ge.build()
    import paper_2512_22195_b200 as mk
    names = _declared()
    assert len(names) >= 21
    lib = ctypes.CDLL(mk.binding.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/matkv.h but not exported"
        assert hasattr(mk, n), f"{n} has no Python binding of the same name"
    assert sorted(mk.binding.EXPORTS) == names


def test_no_gpu_means_a_loud_error_not_a_fallback():
    import torch
    import paper_2512_22195_b200 as mk
    if torch.cuda.is_available():
        return
    try:
        mk.matkv_create(1, 8, 2, 64, 1, 1, 8)
    except mk.MatkvError as e:
        assert e.code == mk.E_CUDA
    else:
        raise AssertionError("matkv_create succeeded without a GPU")


def test_product_code_never_touches_the_oracle():
    pkg = os.path.join(ROOT, "paper_2512_22195_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".h", ".cuh")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f"{f} mentions the oracle"
