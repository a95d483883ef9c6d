"""The C-ABI library builds for sm_100a, loads without a GPU, and exports every
function that include/excp.h declares; its pure size arithmetic agrees with the
oracle's layout."""
import ctypes
import os
import re

import pytest

from oracle import excp_oracle as orc
from paper_2406_11257_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "excp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(excp_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_function():
    lib = binding.load_library()
    names = declared_functions()
    assert len(names) >= 10
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(binding.EXPORTS) == names


def test_record_size_arithmetic_matches_the_layout():
    for numel, nnz_w, nnz_o in [(0, 0, 0), (1, 1, 1), (33, 20, 3), (4096, 4096, 0), (1000003, 530001, 58001)]:
        assert binding.record_bytes(numel, nnz_w, nnz_o, 4) == orc.record_bytes(numel, nnz_w, nnz_o, 4)
    assert binding.compress_bound(1000, 4) == orc.record_bytes(1000, 1000, 1000, 4)
    assert binding.record_bytes(10, 1, 1, 3) == 0


def test_status_strings_and_null_handle():
    lib = binding.load_library()
    assert lib.excp_status_string(0) == b"ok"
    assert b"corrupt" in lib.excp_status_string(-5)
    assert lib.excp_destroy(None) == 0
    e = ctypes.c_int(7)
    assert lib.excp_last_cuda_error(None, ctypes.byref(e)) == -1


def test_struct_sizes_match_the_header():
    # float, float, int, int, u64, int, unsigned -> 32 bytes; 4 x u64 + 4 x float + 3 x double -> 72 bytes
    assert ctypes.sizeof(binding.CParams) == 32
    assert ctypes.sizeof(binding.CStats) == 72
