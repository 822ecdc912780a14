"""The C-ABI library builds, loads and exports every symbol the header declares (no GPU needed)."""
import ctypes
import os
import re

import paper_2606_18394_b200 as jet
from paper_2606_18394_b200 import build as jet_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        text = open(os.path.join(ROOT, "include", fn)).read()
        names += re.findall(r"JET_API\s+[\w\s\*]+?\b(jet_\w+)\s*\(", text)
    return sorted(set(names))


def test_library_builds_and_exports_every_declared_symbol():
    path = jet_build.build()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    declared = _declared()
    assert len(declared) >= 8
    for name in declared:
        assert hasattr(lib, name), name
    assert set(declared) == set(jet.exported_symbols())


def test_status_strings_and_workspace_queries():
    assert jet.status_string(0) == "JET_OK"
    assert jet.status_string(-5) == "JET_ERR_TIMEOUT"
    assert jet.jet_tree_build_workspace_bytes(1, 8, 151936, 7) % 256 == 0
    assert jet.jet_tree_accept_workspace_bytes(32, 64, 151936) >= 32 * 64 * 8
    assert jet.jet_tree_build_workspace_bytes(0, 8, 10, 7) == 0
