"""The C-ABI library builds, loads without a GPU and exports every function include/dcut.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "dcut.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(dcut_[a-z_0-9]+)\s*\(", src)))


@pytest.fixture(scope="module")
def lib():
    from paper_2607_14647_b200 import build
    return ctypes.CDLL(build.build_lib())


def test_header_declares_the_hot_path():
    names = _declared()
    for n in ("dcut_select", "dcut_verify_attn", "dcut_accept", "dcut_create", "dcut_destroy"):
        assert n in names


def test_every_declared_symbol_is_exported(lib):
    for name in _declared():
        assert hasattr(lib, name), f"{name} declared in dcut.h but not exported"


def test_binding_lists_the_same_entry_points(lib):
    from paper_2607_14647_b200 import binding
    declared = _declared()
    assert sorted(binding.EXPORTS) == [n for n in declared if n in binding.EXPORTS]
    for n in ("dcut_select", "dcut_verify_attn", "dcut_accept"):
        assert n in binding.EXPORTS


def test_budget_from_ratio_host_only(lib):
    k = ctypes.c_int(0)
    for (B, g, num, den), want in [((64, 15, 1, 4), 256), ((64, 15, 3, 4), 768), ((1, 15, 1, 4), 4),
                                   ((3, 4, 1, 4), 4), ((3, 4, 1, 2), 8), ((10, 3, 1, 100), 10)]:
        assert lib.dcut_budget_from_ratio(B, g, num, den, ctypes.byref(k)) == 0 and k.value == want
    assert lib.dcut_budget_from_ratio(4, 4, 1, 0, ctypes.byref(k)) == 1


def test_product_path_does_not_touch_the_oracle():
    """No file of the package imports, opens or links anything under oracle/."""
    pkg = os.path.join(ROOT, "paper_2607_14647_b200")
    for dirpath, _, files in os.walk(pkg):
        if os.path.basename(dirpath) == "build":
            continue
        for f in files:
            if f.endswith((".py", ".cu", ".h", ".cuh")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"(import|from)\s+oracle|oracle/|liboracle|dcut_oracle|oracle_[a-z]+\(", text), f
