"""The C-ABI library builds, loads without a GPU and exports what the header declares."""
import os
import re

import paper_2009_09271_b200 as sc
from paper_2009_09271_b200 import build as scbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "sparsecomm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sc_[a-z_]+)\s*\(", text)))


def test_header_symbols_are_exported():
    scbuild.build()
    lib = sc.load_library()
    names = declared_functions()
    assert len(names) >= 12
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(sc.EXPORTS) == names


def test_strerror_needs_no_gpu():
    assert sc.strerror(0) == "ok"
    assert "timed out" in sc.strerror(-5)
