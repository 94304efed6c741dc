"""The C-ABI library: loads, exports what include/attnw.h declares, and rejects bad arguments
on the host (these calls return before anything touches a GPU)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "attnw.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2407_13885_b200 import build
    build.build_library()
    from paper_2407_13885_b200 import binding
    return binding.lib


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return re.findall(r"^\s*(?:const\s+)?(?:int|long long|char\s*\*|const char\s*\*)\s*\*?\s*(\w+)\s*\(", text, flags=re.M)


def test_header_declares_the_entry_points():
    names = declared_functions()
    for must in ("attnw_fused", "attnw_fused_f32", "softmax_rows", "softmax_rows_f32", "attnw_query_status",
                 "attnw_fused_host", "softmax_rows_host", "attnw_strerror", "attnw_version"):
        assert must in names


def test_library_exports_every_declared_symbol(lib):
    from paper_2407_13885_b200 import binding
    raw = ctypes.CDLL(binding.library_path())
    names = declared_functions()
    assert len(names) >= 9
    for name in names:
        assert hasattr(raw, name), f"libattnw.so lacks {name}"
        assert name in binding.SIGNATURES, f"binding lacks {name}"
    assert set(binding.SIGNATURES) == set(names)


def test_version_and_strerror(lib):
    assert lib.attnw_version() >= 100
    seen = set()
    for code in range(0, 8):
        msg = lib.attnw_strerror(code).decode()
        assert msg and msg not in seen
        seen.add(msg)
    assert "unknown" in lib.attnw_strerror(12345).decode()


A = 0x10000  # a 16-byte aligned, non-null fake address: validation never dereferences pointers


def test_fused_argument_errors_are_host_side(lib):
    f = lib.attnw_fused
    assert f(None, A, A, 1, 1, 128, 64, 0.125, None) == 1
    assert f(A, None, A, 1, 1, 128, 64, 0.125, None) == 1
    assert f(A, A, None, 1, 1, 128, 64, 0.125, None) == 1
    assert f(A, A, 0x900000, 0, 1, 128, 64, 0.125, None) == 2
    assert f(A, A, 0x900000, 1, 1, 0, 64, 0.125, None) == 2
    assert f(A, A, 0x900000, 1, 1, 128, 64, -1.0, None) == 2
    assert f(A, A, 0x900000, 1, 1, 128, 64, float("nan"), None) == 2
    assert f(A, A, 0x900000, 1, 1, 128, 64, float("inf"), None) == 2
    assert f(A, A, 0x900000, 1, 1, 128, 32, 0.125, None) == 4
    assert f(A, A, 0x900000, 1, 1, 128, 256, 0.125, None) == 4
    assert f(A + 2, A, 0x900000, 1, 1, 128, 64, 0.125, None) == 3
    assert f(A, A, 0x900000 + 8, 1, 1, 128, 64, 0.125, None) == 3
    assert f(A, A, 0x900000, 1, 1, 132, 64, 0.125, None) == 3          # 132 * 2 bytes not a multiple of 16
    assert lib.attnw_fused_f32(A, A, 0x900000, 1, 1, 130, 64, 0.125, None) == 3
    assert f(A, 0x200000, A + 4096, 1, 1, 128, 64, 0.125, None) == 7   # P inside Q
    assert f(0x200000, A, A + 4096, 1, 1, 128, 64, 0.125, None) == 7   # P inside K
    assert f(A, A, 0x900000, 65536, 65536, 128, 64, 0.125, None) == 2  # B*H overflows


def test_projection_argument_errors_are_host_side(lib):
    f = lib.attnw_project_qk
    X, WQ, WK, Q, K = 0x100000, 0x2000000, 0x3000000, 0x4000000, 0x5000000
    for i in range(5):
        ptrs = [X, WQ, WK, Q, K]
        ptrs[i] = None
        assert f(*ptrs, 1, 128, 64, 1, 64, None) == 1
    assert f(X, WQ, WK, Q, K, 0, 128, 64, 1, 64, None) == 2
    assert f(X, WQ, WK, Q, K, 1, 0, 64, 1, 64, None) == 2
    assert f(X, WQ, WK, Q, K, 1, 128, 0, 1, 64, None) == 2
    assert f(X, WQ, WK, Q, K, 1, 128, 64, 0, 64, None) == 2
    assert f(X, WQ, WK, Q, K, 1, 128, (1 << 20) + 8, 1, 64, None) == 2
    assert f(X, WQ, WK, Q, K, 1, 128, 64, 1, 32, None) == 4            # d must be 64 or 128
    assert f(X, WQ, WK, Q, K, 1, 128, 68, 1, 64, None) == 3            # rows of X would not start on 16 bytes
    assert f(X + 2, WQ, WK, Q, K, 1, 128, 64, 1, 64, None) == 3
    assert f(X, WQ, WK, Q, K + 8, 1, 128, 64, 1, 64, None) == 3
    assert f(X, WQ, WK, Q, Q, 1, 128, 64, 1, 64, None) == 7            # Q and K may not share memory
    assert f(X, WQ, WK, X, K, 1, 128, 64, 1, 64, None) == 7            # an output over an input
    assert f(X, WQ, WK, Q, WK + 16, 1, 128, 64, 1, 64, None) == 7


def test_rows_argument_errors_are_host_side(lib):
    f = lib.softmax_rows
    assert f(None, A, 4, 8, None) == 1
    assert f(A, None, 4, 8, None) == 1
    assert f(A, 0x900000, 0, 8, None) == 2
    assert f(A, 0x900000, 4, 0, None) == 2
    assert f(A, 0x900000, 4, 6, None) == 3
    assert f(A + 4, 0x900000, 4, 8, None) == 3
    assert f(A, A, 4, 8, None) == 7                       # bf16 output may not alias the input
    assert f(A, A + 16, 4, 8, None) == 7
    assert lib.softmax_rows_f32(A, A + 16, 4, 8, None) == 7  # partial overlap
    assert f(A, 0x900000, 1 << 41, 8, None) == 2


def test_fused_variant_knob(lib):
    assert lib.attnw_set_fused_variant(5) == 2
    assert lib.attnw_set_fused_variant(-1) == 2
    for v in (1, 2, 3, 4, 0):
        assert lib.attnw_set_fused_variant(v) == 0


def test_rows_variant_knob(lib):
    assert lib.attnw_set_rows_variant(4) == 2
    assert lib.attnw_set_rows_variant(-1) == 2
    for v in (1, 2, 3, 0):
        assert lib.attnw_set_rows_variant(v) == 0


def test_attention_variant_knob(lib):
    assert lib.attnw_set_attn_variant(3) == 2
    assert lib.attnw_set_attn_variant(-1) == 2
    for v in (1, 2, 0):
        assert lib.attnw_set_attn_variant(v) == 0


def test_query_status_rejects_null(lib):
    assert lib.attnw_query_status(None, None) == 1
