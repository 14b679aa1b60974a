"""CPU-side checks of the C ABI: the library builds, loads and exports every function the header
declares; the binding names them all.  No kernel is launched here."""
import ctypes as C
import os
import re

import pytest

from paper_2511_02017_b200 import binding as tp
from paper_2511_02017_b200 import build as tpbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "tapout.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tapout_[a-z0-9_]+)\s*\(", text)))


@pytest.fixture(scope="module")
def lib():
    tpbuild.build()
    return tp.load()


def test_header_functions_are_exported(lib):
    names = _declared()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(tp.EXPORTS) == names


def test_error_strings(lib):
    assert lib.tapout_strerror(0) == b"ok"
    for code in range(-6, 0):
        assert lib.tapout_strerror(code) not in (b"ok", b"unknown error")
    assert lib.tapout_strerror(-99) == b"unknown error"


def test_param_keys_match_header():
    text = open(os.path.join(ROOT, "include", "tapout.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    keys = re.findall(r"TAPOUT_P_([A-Z0-9_]+)\s*=\s*(\d+)", text)
    table = {k.lower(): int(v) for k, v in keys if not k.startswith("_")}
    assert table == tp.PARAM


def test_null_handle_is_rejected_without_touching_a_device(lib):
    assert lib.tapout_update(None) == tp.E_INVALID_ARG
    assert lib.tapout_destroy(None) == tp.E_INVALID_ARG
    assert lib.tapout_draft_step(None, None, None, None) == tp.E_INVALID_ARG
    assert lib.tapout_create(None, 1, 8, 1, 1, 0, 0) == tp.E_INVALID_ARG
    h = C.c_void_p()
    assert lib.tapout_create(C.byref(h), 0, 8, 1, 1, 0, 0) == tp.E_INVALID_ARG
