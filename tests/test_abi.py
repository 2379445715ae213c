"""The C-ABI library loads without a GPU and exports exactly what include/d2d.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "d2d.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2310_04361_b200 import build
    return ctypes.CDLL(build.build())


def _declared():
    text = open(HEADER).read()
    return sorted(set(re.findall(r"D2D_API[^;(]*?\b(d2d_\w+)\s*\(", text)))


def test_header_declares_the_named_entry_points():
    names = _declared()
    for required in ("d2d_router_fwd", "d2d_select_dynk", "d2d_moe_ffn_fwd", "d2d_layer_fwd", "d2d_layer_create"):
        assert required in names


def test_library_exports_every_declared_symbol(lib):
    for name in _declared():
        assert hasattr(lib, name), name


def test_binding_lists_the_same_symbols():
    from paper_2310_04361_b200 import api
    assert sorted(api.EXPORTS) == _declared()


def test_status_strings_and_host_side_validation(lib):
    lib.d2d_status_str.restype = ctypes.c_char_p
    assert lib.d2d_status_str(0) == b"ok"
    assert b"tau" not in lib.d2d_status_str(1) and lib.d2d_status_str(1)
    assert lib.d2d_status_str(99) == b"unknown status"
    lib.d2d_select_workspace_bytes.restype = ctypes.c_size_t
    assert lib.d2d_select_workspace_bytes(1, 16) >= 64
    assert lib.d2d_select_workspace_bytes(25216, 192) >= 25 * 192 * 4
    assert lib.d2d_select_workspace_bytes(-1, 16) == 0
    # argument errors are reported before any CUDA call is made
    assert lib.d2d_layer_create(None, None, None, None) == 1
    assert lib.d2d_layer_destroy(None) == 0
    lib.d2d_workspace_bytes.restype = ctypes.c_size_t
    assert lib.d2d_workspace_bytes(None, 128) == 0
    assert lib.d2d_router_fwd(None, None, 4, None, None, 0, None) == 1
    assert lib.d2d_select_dynk(None, 4, 16, ctypes.c_float(0.5), None, None, 0, None) == 1
    assert lib.d2d_moe_ffn_fwd(None, None, 4, None, None, None, 0, None) == 1
    assert lib.d2d_group_create(None, 3, None, None) == 1
    assert lib.d2d_group_destroy(None) == 0
    lib.d2d_group_workspace_bytes.restype = ctypes.c_size_t
    assert lib.d2d_group_workspace_bytes(None, 16) == 0
    assert lib.d2d_group_fwd(None, None, 4, ctypes.c_float(0.5), None, None, None, 0, None) == 1


def test_product_does_not_reach_the_oracle():
    """Nothing under the package or the boundary may import, link or execute oracle/."""
    pkg = os.path.join(ROOT, "paper_2310_04361_b200")
    for base, _, files in os.walk(pkg):
        if os.path.basename(base) in ("build", "__pycache__"):
            continue
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h", ".cpp")):
                text = open(os.path.join(base, f)).read()
                assert not re.search(r"^\s*(import|from)\s+oracle\b", text, flags=re.M), f
                assert "d2d_oracle" not in text, f
