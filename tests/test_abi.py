"""The C-ABI library loads, exports every function the header declares, and rejects bad
arguments on the host before touching a device.  CPU only: no compute call is made."""
import ctypes
import os
import re

import pytest

import __graft_entry__ as entry

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    entry.build()
    from paper_2603_12617_b200 import binding
    return binding._lib


def declared_functions():
    text = open(os.path.join(ROOT, "include", "sd_verify.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sd_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_expected_entry_points():
    names = declared_functions()
    for must in ["sd_verify_feedback", "sd_verify_feedback_bf16", "sd_verify_feedback_ex",
                 "sd_verify_feedback_host", "sd_verify_feedback_static", "sd_verify_greedy",
                 "sd_greedy_workspace_bytes", "sd_verify_error_feedback", "sd_ensemble_feedback",
                 "sd_workspace_bytes", "sd_strerror", "sd_version"]:
        assert must in names


def test_library_exports_every_declared_symbol(lib):
    for name in declared_functions():
        assert hasattr(lib, name), f"{name} is declared in sd_verify.h but not exported"


def test_version_and_strerror(lib):
    assert lib.sd_version() == 100
    for code in range(0, -9, -1):
        assert lib.sd_strerror(code)
    assert b"unknown" in lib.sd_strerror(-99)


def test_workspace_bytes(lib):
    assert lib.sd_workspace_bytes(1, 1, 1, 0) > 0
    assert lib.sd_workspace_bytes(256, 6, 128256, 0) % 256 == 0
    assert lib.sd_workspace_bytes(0, 1, 1, 0) == 0
    assert lib.sd_workspace_bytes(1, 65, 1, 0) == 0
    assert lib.sd_workspace_bytes(1, 1, 1, 7) == 0
    # grows with every dimension
    assert lib.sd_workspace_bytes(64, 4, 151936, 1) > lib.sd_workspace_bytes(32, 4, 151936, 1)


def test_host_side_argument_errors(lib):
    buf = (ctypes.c_float * 64)()
    p = ctypes.cast(buf, ctypes.c_void_p)
    odd = ctypes.c_void_p(p.value + 2)
    f = lib.sd_verify_feedback
    assert f(None, p, p, p, 1.0, 1, 1, 4, p, p, p, p, None) == -1          # SD_ERR_NULL
    assert f(p, p, p, p, 1.0, 0, 1, 4, p, p, p, p, None) == -2            # SD_ERR_SHAPE
    assert f(p, p, p, p, 1.0, 1, 65, 4, p, p, p, p, None) == -2
    assert f(p, p, p, p, 0.0, 1, 1, 4, p, p, p, p, None) == -3            # SD_ERR_TEMPERATURE
    assert f(p, p, p, p, float("nan"), 1, 1, 4, p, p, p, p, None) == -3
    assert f(p, p, p, p, float("inf"), 1, 1, 4, p, p, p, p, None) == -3
    assert f(odd, p, p, p, 1.0, 1, 1, 4, p, p, p, p, None) == -8          # SD_ERR_ALIGN
    ex = lib.sd_verify_feedback_ex
    assert ex(p, p, p, p, 1.0, 1, 1, 4, 9, p, p, p, p, None, None, p, 1 << 20, None) == -5   # SD_ERR_DTYPE
    assert ex(p, p, p, p, 1.0, 1, 1, 4, 0, p, p, p, p, None, None, None, 0, None) == -4      # SD_ERR_WORKSPACE
    assert ex(p, p, p, p, 1.0, 1, 1, 4, 0, p, p, p, p, None, None, p, 16, None) == -4
    host = lib.sd_verify_feedback_host
    assert host(p, None, p, p, 1.0, 1, 1, 4, 0, p, p, p, p, None, None) == -1


def test_host_side_argument_errors_of_the_variants(lib):
    buf = (ctypes.c_float * 64)()
    p = ctypes.cast(buf, ctypes.c_void_p)
    odd = ctypes.c_void_p(p.value + 2)
    # greedy verification
    g = lib.sd_verify_greedy
    assert g(None, p, 1, 1, 4, 0, p, p, p, None, 0, None) == -1           # SD_ERR_NULL
    assert g(p, p, 1, 1, 4, 5, p, p, p, None, 0, None) == -5              # SD_ERR_DTYPE
    assert g(p, p, 0, 1, 4, 0, p, p, p, None, 0, None) == -2              # SD_ERR_SHAPE
    assert g(p, p, 1, 65, 4, 0, p, p, p, None, 0, None) == -2
    assert g(odd, p, 1, 1, 4, 0, p, p, p, None, 0, None) == -8            # SD_ERR_ALIGN
    assert g(p, p, 1, 1, 4, 0, p, p, None, p, 16, None) == -4             # SD_ERR_WORKSPACE (too small)
    assert lib.sd_greedy_workspace_bytes(1, 1) >= 256 + 16
    assert lib.sd_greedy_workspace_bytes(256, 6) % 256 == 0
    assert lib.sd_greedy_workspace_bytes(0, 1) == 0 and lib.sd_greedy_workspace_bytes(1, 65) == 0
    # error-position feedback
    e = lib.sd_verify_error_feedback
    assert e(p, None, p, p, 1.0, 1, 1, 4, 0, p, p, p, p, None, None, 0, None) == -1
    assert e(p, p, p, p, -1.0, 1, 1, 4, 0, p, p, p, p, None, None, 0, None) == -3
    assert e(p, p, p, p, 1.0, 1, 1, 5, 0, p, p, p, p, None, None, 0, None) == -8      # rows of 20 bytes
    assert e(p, p, p, p, 1.0, 1, 1, 4, 0, p, p, p, p, None, p, 16, None) == -4
    # ensemble feedback: host arrays of device pointers
    arr = (ctypes.c_void_p * 2)(p.value, p.value)
    bad = (ctypes.c_void_p * 2)(p.value, None)
    f = lib.sd_ensemble_feedback
    ok_tail = (None, p, None, p, p, p, None, None, 0, None)
    assert f(None, arr, 2, 1.0, 10.0, 1, 1, 4, 0, *ok_tail) == -1
    assert f(p, bad, 2, 1.0, 10.0, 1, 1, 4, 0, *ok_tail) == -1
    assert f(p, arr, 0, 1.0, 10.0, 1, 1, 4, 0, *ok_tail) == -2
    assert f(p, arr, 9, 1.0, 10.0, 1, 1, 4, 0, *ok_tail) == -2
    assert f(p, arr, 2, 0.0, 10.0, 1, 1, 4, 0, *ok_tail) == -3
    assert f(p, arr, 2, 1.0, -1.0, 1, 1, 4, 0, *ok_tail) == -3
    assert f(p, arr, 2, 1.0, 10.0, 1, 1, 5, 0, *ok_tail) == -8
    assert f(p, arr, 2, 1.0, 10.0, 1, 1, 4, 3, *ok_tail) == -5
