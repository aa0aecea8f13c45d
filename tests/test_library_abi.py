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
                 "lantern_verify_workspace_bytes", "lantern_last_status", "lantern_status_string"):
        assert must in names


def test_header_keeps_the_interface_sketch():
    """Status codes and the workspace query as the boundary was specified: OK, NULL, SHAPE, PARAM, WORKSPACE,
    CUDA, DATA, UNIMPLEMENTED = 0, -1 ... -7; the workspace query takes (B, N, V, k, dtype)."""
    text = open(os.path.join(ROOT, "include", "lantern.h")).read()
    for name, val in [("LANTERN_OK", 0), ("LANTERN_E_NULL", -1), ("LANTERN_E_SHAPE", -2), ("LANTERN_E_PARAM", -3),
                      ("LANTERN_E_WORKSPACE", -4), ("LANTERN_E_CUDA", -5), ("LANTERN_E_DATA", -6),
                      ("LANTERN_E_UNIMPLEMENTED", -7)]:
        assert re.search(rf"\b{name}\s*=\s*{val}\b", text), name
    assert re.search(r"lantern_verify_workspace_bytes\(int B, int N, int V, int k, int dtype\)", text)
    assert re.search(r"lantern_last_status\(const void\* workspace, void\* cuda_stream, int32_t\* out_bits\)", text)


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
    assert lt.verify_workspace_bytes(32, 7, 16384, 1000, lt.BF16) >= 32 * 8 * 16
    assert lt.verify_workspace_bytes(1, 5000) == 0            # N beyond the supported range
    assert lt.verify_workspace_bytes(4, 4, V=12) == 0         # V not a multiple of 8
    assert lt.verify_workspace_bytes(4, 4, V=64, k=65) == 0   # k > V
    assert lt.verify_workspace_bytes(4, 4, top_k=100) > lt.verify_workspace_bytes(4, 4)   # room for the thresholds
    assert lt.verify_launch_count() == 5 and lt.verify_launch_count(False, True) == 6
    assert lt.verify_launch_count(True, True) == 6
    assert "device" in lt.status_string(-6)
    assert lt.build_workspace_bytes(16384, 8, 1000) == 0
    assert lt.build_workspace_bytes(16384, 256, 1000) == 1024 * 16384 * 4


def test_cpu_tensors_are_refused():
    import torch
    import paper_2410_03355_b200 as lt
    with pytest.raises(ValueError):
        lt.build_neighbors(torch.zeros(16, 8), 4)
