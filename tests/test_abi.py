"""The C-ABI library loads, exports every symbol include/mwu.h declares, and rejects bad
arguments before launching anything (runs without a GPU)."""
import ctypes
import os
import re

import pytest

from paper_2106_08301_b200 import binding as B
from paper_2106_08301_b200 import build as build_mod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    build_mod.build()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "mwu.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mwu_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    L = ctypes.CDLL(B.LIB_PATH)
    names = declared_symbols()
    assert "mwu_project" in names and "mwu_gemm" in names and "mwu_conv_implicit" in names
    for name in names:
        assert hasattr(L, name), name
    assert sorted(n for n in B.EXPORTS) == sorted(n for n in names if n in B.EXPORTS)
    assert set(B.EXPORTS) <= set(names)


def test_count_from_permille_and_strings():
    assert B.mwu_count_from_permille(36864, 600) == 22118
    assert B.mwu_count_from_permille(4194304, 800) == 3355443
    assert B.mwu_count_from_permille(3, 500) == 2
    assert B.status_string(0) == "ok"
    assert "shape" in B.status_string(2)


def test_descriptor_validation_without_a_device():
    ok = B.make_desc(256, 256, 4, 8192, 4096)
    assert B.mwu_project_workspace_bytes(ok) > 4 * 16384
    assert B.mwu_packed_bytes(ok) > 0
    for bad in [B.make_desc(256, 256, 3, 1, 0),         # block width
                B.make_desc(256, 250, 4, 1, 0),         # cols % block
                B.make_desc(256, 256, 4, 10, 11),       # k_prune > k_unify
                B.make_desc(256, 256, 4, 16385, 0),     # k_unify > Mb
                B.make_desc(0, 256, 4, 0, 0)]:
        assert B.mwu_project_workspace_bytes(bad) == 0
    assert B.mwu_packed_bytes(B.make_desc(256, 96, 4, 0, 0)) == 0    # cols % 64 != 0
    L = B.lib()
    null = ctypes.c_void_p(0)
    one = ctypes.c_void_p(256)
    # null descriptor / null pointers / bad shapes are refused before any CUDA call
    assert L.mwu_project(None, *([one] * 11), 0, null) == 1
    d = B.make_desc(256, 250, 4, 1, 0)
    assert L.mwu_project(ctypes.byref(d), *([one] * 11), 1 << 30, null) == 2
    assert L.mwu_project(ctypes.byref(ok), null, *([one] * 10), 1 << 30, null) == 1
    misaligned = ctypes.c_void_p(260)
    assert L.mwu_project(ctypes.byref(ok), misaligned, *([one] * 10), 1 << 30, null) == 3
    assert L.mwu_project(ctypes.byref(ok), *([one] * 11), 16, null) == 4
    assert L.mwu_pack(ctypes.byref(ok), *([one] * 7), 16, one, null) == 4
    assert L.mwu_pack(ctypes.byref(d), *([one] * 7), 1 << 30, one, null) == 2


def test_packed_bytes_matches_the_format_arithmetic():
    import packed_format as F
    for rows, cols, b, ku, kp in [(256, 256, 4, 8192, 4096), (130, 192, 8, 1000, 10),
                                  (16384, 4096, 16, 3355443, 2516582), (100, 128, 2, 6400, 0)]:
        d = B.make_desc(rows, cols, b, ku, kp)
        mb = rows * cols // b
        assert B.mwu_packed_bytes(d) == F.packed_layout(rows, cols, b, ku - kp, mb - ku, kp)["total"]
