"""The C-ABI library builds for sm_100a, loads without a GPU, and exports every
symbol that include/cast.h declares (no compute call is made here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib_path():
    from paper_2510_26577_b200 import build
    return build.build()


def _declared():
    text = open(os.path.join(ROOT, "include", "cast.h")).read()
    return sorted(set(re.findall(r"CAST_API[^;(]*?\b(cast_\w+)\s*\(", text)))


def test_header_declares_the_five_calls():
    names = _declared()
    for n in ("cast_tree_expand", "cast_select_nodes", "cast_tree_attention", "cast_accept", "cast_compact_kv"):
        assert n in names


def test_library_exports_every_declared_symbol(lib_path):
    lib = ctypes.CDLL(lib_path)
    for name in _declared():
        assert hasattr(lib, name), name


def test_binding_lists_every_declared_symbol(lib_path):
    from paper_2510_26577_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()
    lib = binding.load_library()
    assert lib.cast_status_string(3) == b"capacity exceeded"


def test_config_struct_matches_header_layout():
    from paper_2510_26577_b200.binding import CastConfig
    # 3 doubles + 14 int32 = 80 bytes, no padding (doubles first)
    assert ctypes.sizeof(CastConfig) == 80
    assert CastConfig.max_batch.offset == 24 and CastConfig.rerank_per_row.offset == 76
