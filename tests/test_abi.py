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


REQUIRED = [
    # the five entry points the contract names
    "twn_ternarize", "twn_pack", "twn_gemm", "twn_conv2d_fwd", "twn_conv2d_bwd_data",
    # their companions: inverse of pack, code re-layout for the backward pass, weight gradient
    "twn_unpack", "twn_transpose_codes", "twn_conv2d_bwd_weight",
    # library helpers: error text, device status, scratch sizes
    "twn_strerror", "twn_read_status", "twn_ternarize_workspace_bytes",
    "twn_ternarize_batch_workspace_bytes", "twn_conv2d_bwd_weight_workspace_bytes",
]


def test_header_declares_every_contract_entry_point_by_name():
    names = declared_functions()
    for name in REQUIRED:
        assert name in names, f"{name} is missing from include/twn.h"


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


class _Desc(C.Structure):
    _fields_ = [("B", C.c_int64), ("H", C.c_int64), ("W", C.c_int64), ("Cin", C.c_int64),
                ("Cout", C.c_int64), ("kh", C.c_int32), ("kw", C.c_int32),
                ("stride_h", C.c_int32), ("stride_w", C.c_int32),
                ("pad_h", C.c_int32), ("pad_w", C.c_int32)]


def test_contractions_refuse_bad_arguments_on_the_host(lib):
    """twn_gemm, twn_conv2d_fwd and twn_conv2d_bwd_data through raw ctypes with arguments the host can
    see are wrong: each returns its error code before any CUDA call, so no device is needed."""
    i64, null = C.c_int64, None
    # negative extent / NULL operands with work to do / row pitch smaller than K / pitch not a multiple of 64
    assert lib.twn_gemm(null, i64(64), null, i64(64), null, i64(-1), i64(8), i64(64), null, null, i64(8), null, null) == -1
    assert lib.twn_gemm(null, i64(64), null, i64(64), null, i64(4), i64(8), i64(64), null, null, i64(8), null, null) == -1
    fake = C.c_void_p(4096)          # never dereferenced: every call below fails a host check first
    assert lib.twn_gemm(fake, i64(32), fake, i64(64), null, i64(4), i64(8), i64(64), null, fake, i64(8), null, null) == -1
    assert lib.twn_gemm(fake, i64(64), fake, i64(100), null, i64(4), i64(8), i64(64), null, fake, i64(8), null, null) == -1
    # an empty product is fine and launches nothing
    assert lib.twn_gemm(null, i64(64), null, i64(64), null, i64(0), i64(8), i64(64), null, null, i64(8), null, null) == 0
    # operand pitch not a multiple of 8 elements, misaligned pointer
    assert lib.twn_gemm(fake, i64(68), fake, i64(64), null, i64(4), i64(8), i64(64), null, fake, i64(8), null, null) == -2
    assert lib.twn_gemm(C.c_void_p(4098), i64(64), fake, i64(64), null, i64(4), i64(8), i64(64), null, fake, i64(8), null, null) == -2
    for fn in (lib.twn_conv2d_fwd, lib.twn_conv2d_bwd_data):
        assert fn(null, fake, fake, i64(64), null, null, fake, null, null) == -1            # no descriptor
        d = _Desc(2, 8, 8, 16, 16, 3, 3, 1, 1, 1, 1)
        assert fn(C.byref(d), null, fake, i64(192), null, null, fake, null, null) == -1     # NULL input
        assert fn(C.byref(d), fake, fake, i64(64), null, null, fake, null, null) == -1      # pitch < kh*kw*C
        bad = _Desc(2, 8, 8, 16, 16, 3, 3, 0, 1, 1, 1)
        assert fn(C.byref(bad), fake, fake, i64(192), null, null, fake, null, null) == -1   # stride 0
        bad = _Desc(2, 2, 2, 16, 16, 7, 7, 1, 1, 0, 0)
        assert fn(C.byref(bad), fake, fake, i64(1024), null, null, fake, null, null) == -1  # window larger than the image
    # channel counts the tensor copies cannot address: the reduction runs over Cin in the forward pass
    # and over Cout in the backward pass, and needs runs of 16 codes (8 for a 1x1 filter)
    d = _Desc(2, 8, 8, 24, 40, 3, 3, 1, 1, 1, 1)
    assert lib.twn_conv2d_fwd(C.byref(d), fake, fake, i64(256), null, null, fake, null, null) == -2
    assert lib.twn_conv2d_bwd_data(C.byref(d), fake, fake, i64(384), null, null, fake, null, null) == -2
    d = _Desc(2, 8, 8, 32, 130, 1, 1, 1, 1, 0, 0)
    assert lib.twn_conv2d_bwd_data(C.byref(d), fake, fake, i64(192), null, null, fake, null, null) == -2


def test_binding_names_match_the_header():
    from paper_1605_04711_b200 import twn
    for name in declared_functions():
        short = name[len("twn_"):]
        assert hasattr(twn, short), f"binding lacks {short}"
