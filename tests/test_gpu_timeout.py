"""The bounded wait of the tensor-core kernels, run to its limit on purpose.

Every mbarrier wait in the contraction and weight-gradient kernels gives up after a time limit, writes
TWN_ERR_TIMEOUT to the status word the call was given and lets the kernel return normally.  A correct run never
gets there, so a test-support entry point (not in the public header) launches one block whose three roles wait,
with a limit of one millisecond, on a barrier nobody arrives on.  Nothing faults and nothing waits without
bound; the context stays usable, which the GEMM after it shows."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
from paper_1605_04711_b200 import datagen as dg
from paper_1605_04711_b200 import twn
from _gpu_util import dev_bf16
from test_gpu_contract import ternarized, assert_within

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_reports_timeout_and_the_device_stays_usable():
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.full((4,), -1, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream()
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    rc = twn.lib().twn_selftest_wait_timeout(C.c_void_p(status.data_ptr()), C.c_void_p(out.data_ptr()),
                                             C.c_ulonglong(1_000_000), C.c_void_p(stream.cuda_stream))
    t1.record()
    assert rc == 0
    torch.cuda.synchronize()                       # the kernel returned by itself
    assert t0.elapsed_time(t1) < 500.0             # milliseconds: far below the one-second default limit
    assert twn.read_status(status) == -5
    assert "wait" in twn.strerror(-5)
    assert out.cpu().tolist() == [0, 0, 0, 1]      # no wait reported success; the abort flag was raised
    # the context is intact: a GEMM on the same device right after
    M, N, K = 300, 200, 256
    alpha, codes, packed, ld, stats = ternarized(50, "after-timeout", N, K)
    X = dg.draw_bf16(50, "after-timeout-x", M * K, "normal").reshape(M, K)
    Y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    status2 = torch.zeros(1, dtype=torch.int32, device="cuda")
    twn.gemm(dev_bf16(X), K, packed, ld, stats, M, N, K, None, Y, N, status2)
    Yr, A = oracle.gemm(X, codes, alpha)
    assert twn.read_status(status2) == 0
    assert_within(Y.cpu().numpy(), Yr, A, alpha)


def test_the_self_test_entry_point_is_not_part_of_the_public_header():
    import os
    hdr = open(os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include", "twn.h")).read()
    assert "selftest" not in hdr
