"""The C-ABI library builds, loads and exports every symbol include/twn.h declares.
No kernel is launched here; only argument checks that return before any CUDA call."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_1605_04711_b200 import build
    return C.CDLL(build.build())


def declared_functions():
    text = open(os.path.join(ROOT, "include", "twn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(twn_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_north_star_entry_points_once_built():
    names = declared_functions()
    assert "twn_ternarize" in names and "twn_pack" in names


def test_every_declared_symbol_is_exported(lib):
    for name in declared_functions():
        assert hasattr(lib, name), f"{name} declared in twn.h but not exported"


def test_strerror_and_workspace_size(lib):
    lib.twn_strerror.restype = C.c_char_p
    assert lib.twn_strerror(0) == b"ok"
    assert b"align" in lib.twn_strerror(-2)
    lib.twn_ternarize_workspace_bytes.restype = C.c_size_t
    assert 0 < lib.twn_ternarize_workspace_bytes() <= 1 << 20


def test_host_side_argument_checks_need_no_device(lib):
    # ld_codes not a multiple of 64 / smaller than cols / NULL stats: rejected before any CUDA call
    bad = lib.twn_ternarize(None, C.c_int64(1), C.c_int64(100), C.c_double(0.7), None, None,
                            C.c_int64(100), None, None, C.c_size_t(0), None)
    assert bad == -1
    bad = lib.twn_pack(None, C.c_int64(2), C.c_int64(100), None, C.c_int64(64), None, None)
    assert bad == -1
    bad = lib.twn_unpack(None, C.c_int64(-1), C.c_int64(1), C.c_int64(64), None, None, None)
    assert bad == -1


def test_binding_names_match_the_header():
    from paper_1605_04711_b200 import twn
    for name in declared_functions():
        short = name[len("twn_"):]
        assert hasattr(twn, short), f"binding lacks {short}"
