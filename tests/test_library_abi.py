"""The C-ABI library exists, loads without a GPU, and exports every symbol include/lantern.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "lantern.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lantern_[a-z_]+)\s*\(", text)))


def test_header_declares_the_entry_points():
    names = declared_functions()
    for must in ("lantern_build_neighbors", "lantern_verify", "lantern_build_workspace_bytes",
                 "lantern_verify_workspace_bytes"):
        assert must in names


def test_library_builds_loads_and_exports_all_symbols():
    from paper_2410_03355_b200 import build
    path = build.build()
    lib = ctypes.CDLL(path)
    for name in declared_functions():
        assert hasattr(lib, name), name


def test_host_side_queries_need_no_gpu():
    import paper_2410_03355_b200 as lt
    assert lt.status_string(0) == "ok"
    assert "workspace" in lt.status_string(-4)
    assert lt.verify_workspace_bytes(32, 7) >= 32 * 8 * 16
    assert lt.verify_workspace_bytes(1, 5000) == 0            # N beyond the supported range
    assert lt.build_workspace_bytes(16384, 8, 1000) == 0
    assert lt.build_workspace_bytes(16384, 256, 1000) == 1024 * 16384 * 4


def test_cpu_tensors_are_refused():
    import torch
    import paper_2410_03355_b200 as lt
    with pytest.raises(ValueError):
        lt.build_neighbors(torch.zeros(16, 8), 4)
