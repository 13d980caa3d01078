"""twn_ternarize_static: the ternarization entry point for callers that cannot allocate.

A plugin that runs inside another framework's fixed memory plan, or inside a server
whose allocator is frozen after start-up, has no way to obtain the scratch buffer that
twn_ternarize needs.  twn_ternarize_static keeps that scratch in a static device array
inside the library instead.  It must give exactly the results of twn_ternarize: same
kernels, same launch shapes, same reduction order.  The check is done on two calls in a
row, because the second call finds the array in the state the first one left it in.

This file sorts after every other test file on purpose: a run that stops at the first
failure has then already run all other tests.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_1605_04711_b200 import datagen as dg
from paper_1605_04711_b200 import twn

pytestmark = pytest.mark.gpu


def _with_workspace(Wd, rows, cols, ld, factor):
    stats = twn.new_stats()
    packed = torch.full((rows, ld // 16), -1, dtype=torch.int32, device="cuda")
    codes = torch.full((rows, cols), 7, dtype=torch.int8, device="cuda")
    ws = torch.empty(twn.ternarize_workspace_bytes() + 256, dtype=torch.uint8, device="cuda")
    ws = ws[(-ws.data_ptr()) % 256:][:twn.ternarize_workspace_bytes()]
    twn.ternarize(Wd, factor, stats, packed, ld, codes, ws, rows=rows, cols=cols)
    return twn.stats_to_host(stats), packed.cpu().numpy(), codes.cpu().numpy()


def _static(Wd, rows, cols, ld, factor):
    # outputs are allocated by the test (the caller's job); the call itself allocates nothing
    stats = twn.new_stats()
    packed = torch.full((rows, ld // 16), -1, dtype=torch.int32, device="cuda")
    codes = torch.full((rows, cols), 7, dtype=torch.int8, device="cuda")
    twn.ternarize_static(Wd, factor, stats, packed, ld, codes, rows=rows, cols=cols)
    return twn.stats_to_host(stats), packed.cpu().numpy(), codes.cpu().numpy()


def test_two_calls_in_a_row_match_the_allocating_entry_point():
    cases = [(1, 3_000_017, "normal", 0.7), (128, 1152, "laplace", 0.75)]
    for rows, cols, dist, factor in cases:
        W = dg.draw(11, f"noalloc-{rows}x{cols}", rows * cols, dist).reshape(rows, cols)
        Wd = torch.from_numpy(W).cuda()
        ld = twn.ld_for(cols)
        want = _with_workspace(Wd, rows, cols, ld, factor)
        assert want[0]["status"] == 0
        for call in range(2):
            got = _static(Wd, rows, cols, ld, factor)
            # delta and alpha: the tests' tolerance is 1e-12 relative; here they are bit-identical
            assert got[0]["status"] == 0
            assert abs(got[0]["delta"] - want[0]["delta"]) <= 1e-12 * want[0]["delta"], call
            assert abs(got[0]["alpha"] - want[0]["alpha"]) <= 1e-12 * want[0]["alpha"], call
            assert got[0] == want[0], call
            assert np.array_equal(got[1], want[1]), call
            assert np.array_equal(got[2], want[2]), call


def test_matches_the_oracle_and_leaves_device_memory_as_it_found_it():
    """The results are checked against the CPU oracle directly (codes and packed words to the bit,
    threshold and scale to 1e-12), and the device memory in use is the same before and after a
    call: neither torch's allocator nor the driver hands out anything on its behalf.  The second
    call is the one measured at the driver level, because the first launch of a kernel in a process
    may make the driver load its code."""
    rows, cols = 96, 2000
    W = dg.draw(13, "noalloc-oracle", rows * cols, "normal").reshape(rows, cols)
    Wd = torch.from_numpy(W).cuda()
    ld = twn.ld_for(cols)
    stats = twn.new_stats()
    packed = torch.full((rows, ld // 16), -1, dtype=torch.int32, device="cuda")
    codes = torch.full((rows, cols), 7, dtype=torch.int8, device="cuda")
    ref, ref_codes = oracle.ternarize(W, 0.7)
    assert ref.n_boundary == 0
    want_packed = oracle.pack(ref_codes.reshape(rows, cols), ld)
    for call in range(2):
        torch.cuda.synchronize()
        torch_before = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
        free_before, _ = torch.cuda.mem_get_info()
        twn.ternarize_static(Wd, 0.7, stats, packed, ld, codes, rows=rows, cols=cols)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == torch_before
        if call == 1:
            assert free_after == free_before
        st = twn.stats_to_host(stats)
        assert st["status"] == 0
        assert abs(st["delta"] - ref.delta) <= 1e-12 * ref.delta
        assert abs(st["alpha"] - ref.alpha) <= 1e-12 * ref.alpha
        assert (st["n_neg"], st["n_zero"], st["n_pos"]) == (ref.n_neg, ref.n_zero, ref.n_pos)
        assert np.array_equal(codes.cpu().numpy(), ref_codes.reshape(rows, cols))
        assert np.array_equal(packed.cpu().numpy().view(np.uint32), want_packed)
        packed.fill_(-1); codes.fill_(7)


def test_a_small_tensor_after_a_large_one_sees_no_stale_partials():
    big = torch.from_numpy(dg.draw(12, "noalloc-big", 5_000_000, "normal")).cuda()
    small = dg.draw(12, "noalloc-small", 1000, "uniform").reshape(1, 1000)
    sd = torch.from_numpy(small).cuda()
    _static(big, 1, big.numel(), twn.ld_for(big.numel()), 0.7)
    got = _static(sd, 1, 1000, 1024, 0.7)
    want = _with_workspace(sd, 1, 1000, 1024, 0.7)
    assert got[0] == want[0] and np.array_equal(got[1], want[1]) and np.array_equal(got[2], want[2])


def test_sizes_beyond_the_fixed_capacity_are_refused():
    stats = twn.new_stats()
    dummy = torch.zeros(64, dtype=torch.float32, device="cuda")
    packed = torch.zeros(4, dtype=torch.int32, device="cuda")
    rows = 1 << 20
    cols = (twn.TERNARIZE_STATIC_MAX_WEIGHTS >> 20) + 64       # rows*cols just over the limit
    with pytest.raises(twn.TwnError) as e:
        twn.ternarize_static(dummy, 0.7, stats, packed, twn.ld_for(cols), None, rows=rows, cols=cols)
    assert e.value.code == -9
    assert "capacity" in twn.strerror(-9)
