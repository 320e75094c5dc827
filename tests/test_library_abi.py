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


def test_header_constants_and_binding_agree(lib):
    """Enumerators and macros of the header against the binding's copies; every kernel id has a name."""
    text = open(os.path.join(ROOT, "include", "qasg.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    header = {k: int(v, 0) for k, v in re.findall(r"\b(QASG_[A-Z_0-9]+)\s*=\s*(\d+|0x[0-9a-fA-F]+)", text)}
    header.update({k: int(v.rstrip("u"), 0) for k, v in re.findall(r"#define\s+(QASG_[A-Z_0-9]+)\s+(\d+u?)\b", text)})
    pairs = {"QASG_OK": libqasg.OK, "QASG_ERR_NONFINITE": libqasg.ERR_NONFINITE, "QASG_ERR_TIMEOUT": libqasg.ERR_TIMEOUT,
             "QASG_ERR_BAD_INDEX": libqasg.ERR_BAD_INDEX, "QASG_ERR_INVALID_ARG": libqasg.ERR_INVALID_ARG,
             "QASG_Q_THRESHOLD": libqasg.Q_THRESHOLD, "QASG_Q_TERNARY_STOCH": libqasg.Q_TERNARY_STOCH,
             "QASG_Q_NONE": libqasg.Q_NONE, "QASG_RULE_CMD": libqasg.RULE_CMD, "QASG_RULE_RDA": libqasg.RULE_RDA,
             "QASG_OPT_STREAM_ROW_BYTES": libqasg.OPT_STREAM_ROW_BYTES, "QASG_OPT_STREAM_LAG": libqasg.OPT_STREAM_LAG,
             "QASG_OPT_WAIT_POLLS": libqasg.OPT_WAIT_POLLS,
             "QASG_OPT_ONE_LAUNCH_STEP_BYTES": libqasg.OPT_ONE_LAUNCH_STEP_BYTES,
             "QASG_CREATE_SERIAL_LAUNCHES": libqasg.CREATE_SERIAL_LAUNCHES,
             "QASG_CREATE_NO_CODE_SCRATCH": libqasg.CREATE_NO_CODE_SCRATCH, "QASG_KERNEL_COUNT": libqasg.KERNEL_COUNT}
    for name, value in pairs.items():
        assert header[name] == value, name
    lib.qasg_kernel_name.restype = ctypes.c_char_p
    names = [lib.qasg_kernel_name(k).decode() for k in range(libqasg.KERNEL_COUNT)]
    assert all(names) and len(set(names)) == len(names)
    assert lib.qasg_kernel_name(libqasg.KERNEL_COUNT).decode() == ""


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
