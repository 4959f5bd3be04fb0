"""The C-ABI library loads without a GPU and exports every symbol include/dgq.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "dgq.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(dgq_[a-z0-9_]+)\s*\(", src)))


def test_header_symbols_exported():
    from paper_2501_04304_b200 import build, binding
    build.build()
    lib = ctypes.CDLL(build.LIB)
    names = _declared()
    assert len(names) >= 16
    for n in names:
        assert hasattr(lib, n), n
    assert set(binding.EXPORTS) == set(names)


def test_status_strings_and_arg_checks():
    from paper_2501_04304_b200 import binding as b
    assert b.status_string(0) == "ok"
    assert "unknown" in b.status_string(99)
    # argument validation runs before any CUDA call
    n = ctypes.c_size_t(0)
    assert b.lib().dgq_cross_attn_workspace_bytes(2, 8, 4096, 77, 40, ctypes.byref(n)) == 0
    # one partial maximum per block of 128 query rows of every head + (row max, log2 row sum) per row
    assert n.value == 2 * 8 * (4096 // 128) * 4 + 2 * 8 * 4096 * 8
    assert b.lib().dgq_cross_attn_workspace_bytes(2, 8, 4096, 1, 40, ctypes.byref(n)) == 1
    assert b.lib().dgq_groups_info(None, *([None] * 10)) == 1
    assert b.lib().dgq_quantize_act(None, 0, 0, 0, None, ctypes.c_int64(1), ctypes.c_int64(8), None, None, None, None) == 1
