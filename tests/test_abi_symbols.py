"""The C-ABI library loads without a GPU and exports every function the header declares."""
import ctypes
import os
import re

from paper_1202_3173_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "strassen_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(strassen_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_three_named_calls():
    names = _declared()
    for must in ("strassen_plan_create", "strassen_dgemm", "strassen_plan_destroy"):
        assert must in names


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(binding.LIB_PATH)
    names = _declared()
    assert len(names) >= 15
    for name in names:
        assert hasattr(lib, name), name


def test_binding_covers_the_header_one_to_one():
    assert sorted(n for n, _, _ in binding.SYMBOLS) == _declared()
    for n, _, _ in binding.SYMBOLS:
        assert callable(getattr(binding, n)), n


def test_no_torch_types_in_the_boundary():
    text = open(os.path.join(ROOT, "include", "strassen_b200.h")).read()
    assert "torch" not in text and "at::" not in text and "#include <cuda" not in text


def test_product_does_not_reach_into_the_oracle():
    pkg = os.path.join(ROOT, "paper_1202_3173_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cpp", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.lower(), os.path.join(dirpath, f)
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            assert "paper_1202_3173_b200" not in open(os.path.join(ROOT, "oracle", f)).read()
