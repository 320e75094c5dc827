"""The shared library builds, loads without a GPU and exports every entry point that
include/qasg.h declares.  No compute call is made here."""
import ctypes
import os
import re

import pytest

from paper_2208_05631_b200 import build, libqasg

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return libqasg.load()


def _declared():
    text = open(os.path.join(ROOT, "include", "qasg.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(qasg_[a-z_0-9]+)\s*\(", text)))


def test_header_and_binding_agree(lib):
    names = _declared()
    assert sorted(libqasg.EXPORTS) == names
    for name in names:
        assert getattr(lib, name) is not None


def test_host_only_calls(lib):
    assert libqasg.code_words(1) == 1 and libqasg.code_words(16) == 1 and libqasg.code_words(17) == 2
    assert libqasg.code_words(1 << 28) == 1 << 24
    assert libqasg.status_string(libqasg.OK) == "ok"
    assert "non-finite" in libqasg.status_string(libqasg.ERR_NONFINITE)
    assert ctypes.sizeof(libqasg.Params) == 32


def test_argument_errors_are_synchronous(lib):
    h = ctypes.c_void_p()
    assert lib.qasg_create(ctypes.byref(h), 0, 0, 4, 0) == libqasg.ERR_INVALID_ARG       # d_max = 0
    assert lib.qasg_create(ctypes.byref(h), 0, 1 << 35, 4, 0) == libqasg.ERR_INVALID_ARG  # d_max too large
    assert lib.qasg_create(ctypes.byref(h), 0, 1024, 65, 0) == libqasg.ERR_INVALID_ARG    # M_max > 64
    assert lib.qasg_create(None, 0, 1024, 4, 0) == libqasg.ERR_INVALID_ARG
    assert not h.value
    assert lib.qasg_destroy(None) == libqasg.ERR_INVALID_ARG
    p = libqasg.make_params()
    assert lib.qasg_step(None, 0, None, 16, 16, 1, 1, ctypes.byref(p), None, None, None, None, None,
                         None) == libqasg.ERR_INVALID_ARG
