"""The C-ABI library loads and exports every symbol the public header declares (no GPU needed)."""
import ctypes
import os
import re

import paper_2510_07535_b200 as pkg
from paper_2510_07535_b200 import build as owl_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "owlverify.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(owl_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported():
    owl_build.build()
    lib = pkg.load_library()
    names = declared_functions()
    assert {"owl_create", "owl_destroy", "owl_verify_attn", "owl_tree_accept", "owl_get_status"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in owlverify.h but not exported"


def test_status_strings_and_dims_layout():
    assert pkg.status_string(0) == "ok"
    for code in range(-7, 0):
        assert pkg.status_string(code) not in ("", "unknown status")
    assert pkg.status_string(-99) == "unknown status"
    # owl_dims is 11 int32 + 1 float, no padding
    assert ctypes.sizeof(pkg.OwlDims) == 48


def test_binding_has_the_same_names_as_the_abi():
    for n in ("owl_verify_attn", "owl_tree_accept", "owl_get_status"):
        assert hasattr(pkg.OwlContext, n)


def test_product_path_does_not_import_the_oracle():
    pk = os.path.join(ROOT, "paper_2510_07535_b200")
    for dirpath, _, files in os.walk(pk):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in src and "from oracle" not in src and "liboracle" not in src, f
