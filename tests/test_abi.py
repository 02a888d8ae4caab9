"""The C-ABI library loads and exports every symbol that include/gsd.h declares (no compute)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "gsd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(gsd_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


@pytest.fixture(scope="module")
def library():
    from paper_2407_16207_b200 import build
    return ctypes.CDLL(build.build())


def test_header_declares_the_expected_calls():
    names = declared_functions()
    for must in ("gsd_verify_attn", "gsd_accept", "gsd_verify_step_host",
                 "gsd_verify_attn_workspace_bytes", "gsd_accept_workspace_bytes"):
        assert must in names


def test_every_declared_symbol_is_exported(library):
    for name in declared_functions():
        assert hasattr(library, name), name


def test_binding_lists_the_same_symbols():
    from paper_2407_16207_b200 import binding
    assert sorted(binding.EXPORTS) == declared_functions()


def test_version_and_status_strings(library):
    library.gsd_status_string.restype = ctypes.c_char_p
    assert library.gsd_version() == 101
    assert library.gsd_status_string(0) == b"ok"
    for code in range(-6, 0):
        assert library.gsd_status_string(code) not in (b"ok", b"unknown status")
    assert library.gsd_status_string(-99) == b"unknown status"


def test_host_side_validation_needs_no_gpu(library):
    from paper_2407_16207_b200.binding import AcceptParams, AttnParams
    library.gsd_accept_workspace_bytes.restype = ctypes.c_size_t
    assert library.gsd_accept_workspace_bytes(ctypes.byref(AcceptParams(2, 16, 100, 32, 16))) >= 2 * 16 * 8 + 8
    assert library.gsd_accept_workspace_bytes(ctypes.byref(AcceptParams(2, 513, 100, 32, 16))) == 0
    # null pointers and bad shapes are rejected before anything touches a device
    p = AttnParams(1, 16, 4, 4, 64, 128, 0.0, 0, 0)
    assert library.gsd_verify_attn(None, None, None, None, None, None, None, None,
                                   ctypes.byref(p), None, 0, None, None) == -1
    bad = AttnParams(1, 16, 4, 3, 64, 128, 0.0, 0, 0)
    one = ctypes.c_void_p(16)
    assert library.gsd_verify_attn(one, one, one, one, one, one, one, one,
                                   ctypes.byref(bad), None, 0, None, None) == -2
    bad = AttnParams(1, 16, 4, 4, 96, 128, 0.0, 0, 0)
    assert library.gsd_verify_attn(one, one, one, one, one, one, one, one,
                                   ctypes.byref(bad), None, 0, None, None) == -2
    odd = ctypes.c_void_p(8)
    assert library.gsd_verify_attn(odd, one, one, one, one, one, one, one,
                                   ctypes.byref(p), None, 0, None, None) == -3
    ap = AcceptParams(1, 0, 10, 1, 1)
    assert library.gsd_accept(one, one, one, one, one, one, None, ctypes.byref(ap), one, 64,
                              None, None) == -2
    ap = AcceptParams(1, 4, 10, 4, 4)
    assert library.gsd_accept(one, one, one, one, one, one, None, ctypes.byref(ap), None, 0,
                              None, None) == -4
    # the host-buffer step refuses what its acceptance half would refuse before a byte is copied
    # (V = 0 here): no device is needed to see that nothing was enqueued
    good = AttnParams(1, 16, 4, 4, 64, 128, 0.0, 0, 0)
    cp = AcceptParams(1, 16, 0, 8, 16)
    args = [one] * 8 + [ctypes.byref(good)] + [one] * 6 + [None, ctypes.byref(cp), ctypes.c_void_p(256),
                                                            ctypes.c_size_t(1 << 30), None, None]
    library.gsd_verify_step_host.restype = ctypes.c_int
    assert library.gsd_verify_step_host(*args) == -2
