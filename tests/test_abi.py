"""The C-ABI library builds, loads, and exports every symbol include/twig.h declares.
Host-side argument checks are exercised without launching anything (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2503_14075_b200 import build
    return ctypes.CDLL(build.build())


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "twig.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(?:twig_status|size_t|const char \*)\s*\*?\s*(\w+)\s*\(", text)
    return sorted(set(names))


def test_header_functions_are_exported(lib):
    names = _declared_functions()
    assert {"ttp_score_topk_compact", "tree_verify_attention", "tree_accept_compact", "ttp_score",
            "ttp_topk", "ttp_compact", "twig_workspace_bytes", "twig_status_str"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_binding_lists_the_same_entry_points():
    src = open(os.path.join(ROOT, "paper_2503_14075_b200", "twig.py")).read()
    for n in _declared_functions():
        assert f'"{n}"' in src and f"def {n}(" in src or n == "twig_status_str", n


def test_host_side_errors_launch_nothing(lib):
    lib.twig_status_str.restype = ctypes.c_char_p
    assert lib.twig_status_str(0) == b"ok"
    assert lib.twig_status_str(4) == b"workspace too small"
    lib.twig_workspace_bytes.restype = ctypes.c_size_t
    need = lib.twig_workspace_bytes(2, 32, 128, 675, 64)
    assert need >= 2 * 32 * 675 * 4
    assert lib.twig_workspace_bytes(0, 32, 128, 675, 64) == 0
    # NULL pointers are refused before any CUDA call
    vp = ctypes.c_void_p
    lib.ttp_topk.argtypes = [vp, vp, vp, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, vp, vp, vp]
    assert lib.ttp_topk(None, None, None, 1, 16, 4, None, None, None) == 1        # TWIG_ERR_NULL
    lib.tree_accept_compact.argtypes = [vp] * 4 + [ctypes.c_int32] * 2 + [vp] * 9
    assert lib.tree_accept_compact(*([None] * 4), 8, 8, *([None] * 9)) == 1
    lib.tree_verify_attention.argtypes = [vp] * 4 + [ctypes.c_int32] + [vp] * 3 + [ctypes.c_int32] * 2 + \
        [ctypes.c_float] + [vp] * 4 + [ctypes.c_size_t, vp]
    assert lib.tree_verify_attention(None, None, None, None, 0, None, None, None, 8, 4, 0.0, None, None,
                                     None, None, 0, None) == 1
