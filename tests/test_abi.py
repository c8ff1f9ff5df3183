"""The C-ABI library builds, loads and exports every symbol include/tra.h declares (no GPU needed)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "tra.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tra_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2608_02504_b200 import build
    lib = ctypes.CDLL(build.build())
    names = declared_functions()
    assert {"tra_entropy_attn", "tra_budget_radius", "tra_build_block_mask", "tra_sparse_attn"} <= set(names)
    for name in names:
        assert hasattr(lib, name), name


def test_binding_lists_the_same_symbols():
    from paper_2608_02504_b200 import build
    build.build()
    from paper_2608_02504_b200 import api
    assert sorted(api.EXPORTS) == declared_functions()


def test_status_strings_and_null_arguments():
    from paper_2608_02504_b200 import build
    lib = ctypes.CDLL(build.build())
    lib.tra_status_string.restype = ctypes.c_char_p
    assert lib.tra_status_string(0) == b"ok"
    assert b"capacity" in lib.tra_status_string(-3)
    # host-side argument validation happens before any CUDA call
    assert lib.tra_plan_create(None, None, None) == -1
    assert lib.tra_plan_destroy(None) == -1
    assert lib.tra_budget_radius(None, None, None, None, None, 1, 1, None) == -1
    assert lib.tra_sparse_attn(None, None, None, None, None, None, None, None, None, None, 1, 1, ctypes.c_float(1.0),
                               None) == -1
    assert lib.tra_entropy_attn(None, None, None, None, None, None, None, 1, 1, ctypes.c_float(1.0), None) == -1
    lib.tra_hot_path_host_workspace_bytes.restype = ctypes.c_size_t
    assert lib.tra_hot_path_host_workspace_bytes(None, 8) == 0
    assert lib.tra_hot_path_host(None, None, None, None, None, None, ctypes.c_size_t(0), 1, 1, 1,
                                 ctypes.c_float(1.0), None) == -1
