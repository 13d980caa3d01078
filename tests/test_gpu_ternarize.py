"""GPU parity: twn_ternarize / twn_pack / twn_unpack / twn_transpose_codes against the oracle.

Bar: packed codes and counts bit-exact (elements within 1e-12*delta of the
threshold are counted and must be absent), delta and alpha within 1e-12 relative.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_1605_04711_b200 import datagen as dg
from paper_1605_04711_b200 import twn
from _gpu_util import dev_f32, dev_u32, host_u32, workspace

pytestmark = pytest.mark.gpu

REL = 1e-12


def run_ternarize(W2d, factor=0.7, ld=None, want_i8=True):
    rows, cols = W2d.shape
    ld = twn.ld_for(cols) if ld is None else ld
    Wd = dev_f32(W2d)
    stats = twn.new_stats()
    packed = torch.full((rows, ld // 16), -1, dtype=torch.int32, device="cuda")
    codes = torch.full((rows, cols), 7, dtype=torch.int8, device="cuda") if want_i8 else None
    ws = workspace(twn.ternarize_workspace_bytes())
    twn.ternarize(Wd, factor, stats, packed, ld, codes, ws, rows=rows, cols=cols)
    torch.cuda.synchronize()
    return twn.stats_to_host(stats), host_u32(packed), (codes.cpu().numpy() if want_i8 else None)


def check_against_oracle(W2d, factor=0.7, ld=None, want_i8=True):
    rows, cols = W2d.shape
    ld = twn.ld_for(cols) if ld is None else ld
    st, packed, codes = run_ternarize(W2d, factor, ld, want_i8)
    ref, ref_codes = oracle.ternarize(W2d, factor)
    assert st["status"] == 0
    assert ref.n_boundary == 0, "an element sits within 1e-12*delta of the threshold"
    if ref.delta == 0.0:
        assert st["delta"] == 0.0
    else:
        assert abs(st["delta"] - ref.delta) <= REL * ref.delta
    if ref.alpha == 0.0:
        assert st["alpha"] == 0.0
    else:
        assert abs(st["alpha"] - ref.alpha) <= REL * ref.alpha
        assert abs(st["sum_abs_kept"] - ref.sum_abs_kept) <= REL * ref.sum_abs_kept
    assert (st["n_neg"], st["n_zero"], st["n_pos"]) == (ref.n_neg, ref.n_zero, ref.n_pos)
    want = oracle.pack(ref_codes.reshape(rows, cols), ld)
    assert np.array_equal(packed, want)
    if want_i8:
        assert np.array_equal(codes, ref_codes.reshape(rows, cols))
    return st


@pytest.mark.parametrize("n", [1, 3, 15, 16, 17, 63, 64, 65, 511, 512, 513, 1000, 4099, 10000, 65536 + 7])
def test_flat_sizes_including_ragged_tails(n):
    check_against_oracle(dg.draw(0, f"flat{n}", n, "normal").reshape(1, n))


@pytest.mark.parametrize("rows,cols", [(32, 25), (128, 27), (64, 147), (64, 800), (10, 512), (5, 64),
                                       (128, 1152), (512, 4608), (1000, 512), (3, 1)])
def test_filter_shaped_tensors(rows, cols):
    W = dg.he_normal(0, f"w{rows}x{cols}", rows, cols)
    check_against_oracle(W)


def test_wider_row_pitch_is_padded_with_zero_codes():
    W = dg.he_normal(1, "pitch", 7, 100)
    st, packed, _ = run_ternarize(W, ld=256)
    full = oracle.unpack(packed, 7, 256, 256)
    assert not full[:, 100:].any()
    check_against_oracle(W, ld=256)


@pytest.mark.parametrize("factor", [0.75, 2.0 / 3.0, 0.0, 0.05])
def test_other_threshold_factors(factor):
    check_against_oracle(dg.draw(2, "fac", 70001, "laplace").reshape(1, -1), factor)


def test_paper_factor_0p75_hand_worked():
    W = np.array([[0.1, -0.2, 0.3, -2.0, 4.0]], dtype=np.float32)
    st, packed, codes = run_ternarize(W, 0.75)
    assert codes.tolist() == [[0, 0, 0, -1, 1]]
    assert st["alpha"] == pytest.approx(3.0, rel=1e-12)


def test_elements_exactly_on_the_threshold_become_zero():
    W = np.array([[1.0, -1.0, 3.0, -3.0]], dtype=np.float32)
    st, packed, codes = run_ternarize(W, 0.5)
    assert st["delta"] == 1.0 and st["alpha"] == 3.0
    assert codes.tolist() == [[0, 0, 1, -1]]
    assert (st["n_neg"], st["n_zero"], st["n_pos"]) == (1, 2, 1)


def test_degenerate_inputs():
    st, packed, codes = run_ternarize(np.zeros((1, 700), dtype=np.float32))
    assert st["delta"] == 0.0 and st["alpha"] == 0.0 and st["n_zero"] == 700 and not packed.any()
    tiny = np.float32(1e-42)
    W = np.array([[-0.0, tiny, -tiny, 0.0]], dtype=np.float32)
    st, packed, codes = run_ternarize(W)
    assert codes.tolist() == [[0, 1, -1, 0]]
    assert st["alpha"] == pytest.approx(float(tiny), rel=1e-12)


def test_empty_tensor():
    stats = twn.new_stats()
    ws = workspace(twn.ternarize_workspace_bytes())
    W = torch.empty(0, dtype=torch.float32, device="cuda")
    packed = torch.empty(0, dtype=torch.int32, device="cuda")
    twn.ternarize(W, 0.7, stats, packed, 0, None, ws, rows=0, cols=0)
    st = twn.stats_to_host(stats)
    assert st["status"] == 0 and st["delta"] == 0.0 and st["alpha"] == 0.0 and st["n_zero"] == 0


def test_nonfinite_weights_set_the_device_status():
    W = dg.draw(0, "nf", 5000, "normal").reshape(1, -1).copy()
    W[0, 1234] = np.inf
    st, _, _ = run_ternarize(W)
    assert st["status"] == -4
    W[0, 1234] = np.nan
    st, _, _ = run_ternarize(W)
    assert st["status"] == -4


def test_host_detected_errors():
    ws = workspace(twn.ternarize_workspace_bytes())
    W = torch.zeros(128, device="cuda")
    packed = torch.zeros(8, dtype=torch.int32, device="cuda")
    stats = twn.new_stats()
    with pytest.raises(twn.TwnError) as e:
        twn.ternarize(W, 0.7, stats, packed, 100, None, ws, rows=1, cols=100)
    assert e.value.code == -1
    with pytest.raises(twn.TwnError) as e:
        twn.ternarize(W[1:], 0.7, stats, packed, 128, None, ws, rows=1, cols=100)
    assert e.value.code == -2
    with pytest.raises(twn.TwnError) as e:
        twn.ternarize(W, 0.7, stats, packed, 128, None, ws[:1024], rows=1, cols=100)
    assert e.value.code == -3


def test_bitwise_determinism_and_workspace_reuse():
    W = dg.draw(0, "det", 3_000_001, "normal").reshape(1, -1)
    a = run_ternarize(W, want_i8=False)
    b = run_ternarize(W, want_i8=False)
    assert a[0] == b[0] and np.array_equal(a[1], b[1])
    # the same workspace serves back-to-back calls on one stream
    Wd = dev_f32(W)
    ws = workspace(twn.ternarize_workspace_bytes())
    outs = []
    for _ in range(3):
        stats = twn.new_stats()
        packed = torch.empty((1, twn.ld_for(W.size) // 16), dtype=torch.int32, device="cuda")
        twn.ternarize(Wd, 0.7, stats, packed, twn.ld_for(W.size), None, ws, rows=1, cols=W.size)
        outs.append((stats, packed))
    torch.cuda.synchronize()
    for s, p in outs:
        assert twn.stats_to_host(s) == a[0] and np.array_equal(host_u32(p), a[1])


@pytest.mark.parametrize("dist", ["normal", "laplace", "uniform"])
@pytest.mark.parametrize("seed", [0, 1, 2])
@pytest.mark.parametrize("n", [10_000, 1_000_000, 10_000_000])
def test_sweep_small_and_medium(dist, seed, n):
    check_against_oracle(dg.draw(seed, f"sweep-{dist}", n, dist).reshape(1, n), want_i8=False)


@pytest.mark.parametrize("dist", ["normal", "laplace", "uniform"])
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_sweep_full_size_1e8(dist, seed):
    n = 100_000_000
    st = check_against_oracle(dg.draw(seed, f"sweep-{dist}", n, dist).reshape(1, n), want_i8=False)
    assert st["n_neg"] + st["n_zero"] + st["n_pos"] == n


# ------------------------------------------------------------------ pack
@pytest.mark.parametrize("rows,cols", [(1, 1), (1, 16), (3, 17), (7, 100), (64, 1152), (2, 1025), (1, 1_000_003)])
def test_pack_unpack_round_trip(rows, cols):
    u = dg.draw(5, "pk", rows * cols, "uniform")
    codes = (np.where(u > 0.3, 1, 0) - np.where(u < -0.3, 1, 0)).astype(np.int8).reshape(rows, cols)
    ld = twn.ld_for(cols)
    cd = torch.from_numpy(codes).cuda()
    packed = torch.full((rows, ld // 16), -1, dtype=torch.int32, device="cuda")
    counts = twn.new_stats()
    twn.pack(cd, rows, cols, packed, ld, counts)
    assert np.array_equal(host_u32(packed), oracle.pack(codes, ld))
    c = twn.stats_to_host(counts)
    assert (c["n_neg"], c["n_zero"], c["n_pos"], c["status"]) == (
        int((codes == -1).sum()), int((codes == 0).sum()), int((codes == 1).sum()), 0)
    back = torch.full((rows, cols), 9, dtype=torch.int8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    twn.unpack(packed, rows, cols, ld, back, status)
    assert np.array_equal(back.cpu().numpy(), codes)
    assert twn.read_status(status) == 0


def test_pack_flags_codes_outside_the_ternary_set():
    codes = torch.tensor([[1, 0, -1, 2, 1, -2, 0, 1]], dtype=torch.int8, device="cuda")
    packed = torch.zeros((1, 4), dtype=torch.int32, device="cuda")
    counts = twn.new_stats()
    twn.pack(codes, 1, 8, packed, 64, counts)
    assert twn.stats_to_host(counts)["status"] == -8
    want = oracle.pack(np.array([[1, 0, -1, 0, 1, 0, 0, 1]], dtype=np.int8), 64)
    assert np.array_equal(host_u32(packed), want)


def test_unpack_flags_the_unused_field():
    # element 0 (bits 15:14) = +1, element 1 (bits 31:30) = the unused field 10
    packed = dev_u32(np.array([[(0b01 << 14) | (0b10 << 30), 0, 0, 0]], dtype=np.uint32))
    out = torch.zeros((1, 2), dtype=torch.int8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    twn.unpack(packed, 1, 2, 64, out, status)
    assert twn.read_status(status) == -8
    assert out.cpu().tolist() == [[1, 0]]


@pytest.mark.parametrize("Cout,Cin,k", [(64, 64, 3), (128, 64, 1), (10, 512, 1), (32, 8, 5), (6, 3, 3), (512, 256, 3), (192, 96, 3)])
def test_transpose_codes(Cout, Cin, k):
    u = dg.draw(6, "tr", Cout * k * k * Cin, "uniform")
    codes = (np.where(u > 0.3, 1, 0) - np.where(u < -0.3, 1, 0)).astype(np.int8).reshape(Cout, k, k, Cin)
    ld_f, ld_b = twn.ld_for(k * k * Cin), twn.ld_for(k * k * Cout)
    pf = dev_u32(oracle.pack(codes.reshape(Cout, -1), ld_f))
    pb = torch.full((Cin, ld_b // 16), -1, dtype=torch.int32, device="cuda")
    twn.transpose_codes(pf, ld_f, twn.conv_desc(1, 8, 8, Cin, Cout, k), pb, ld_b)
    want = oracle.pack(np.ascontiguousarray(codes.transpose(3, 1, 2, 0)).reshape(Cin, -1), ld_b)
    assert np.array_equal(host_u32(pb), want)


def test_transpose_codes_with_a_wider_row_pitch_zeroes_the_rest_of_the_row():
    Cout, Cin, k = 128, 48, 3
    u = dg.draw(7, "trp", Cout * k * k * Cin, "uniform")
    codes = (np.where(u > 0.3, 1, 0) - np.where(u < -0.3, 1, 0)).astype(np.int8).reshape(Cout, k, k, Cin)
    ld_f, ld_b = twn.ld_for(k * k * Cin) + 64, twn.ld_for(k * k * Cout) + 128
    pf = dev_u32(oracle.pack(codes.reshape(Cout, -1), ld_f))
    pb = torch.full((Cin, ld_b // 16), -1, dtype=torch.int32, device="cuda")
    twn.transpose_codes(pf, ld_f, twn.conv_desc(1, 8, 8, Cin, Cout, k), pb, ld_b)
    want = oracle.pack(np.ascontiguousarray(codes.transpose(3, 1, 2, 0)).reshape(Cin, -1), ld_b)
    assert np.array_equal(host_u32(pb), want)


def test_batched_call_equals_one_call_per_tensor():
    """twn_ternarize_batch (the first loop of Algorithm 1 for a whole network in one launch per
    sweep) gives every tensor the bits of a twn_ternarize call of its own, and those match the oracle."""
    shapes = [(64, 147), (64, 576), (128, 1152), (256, 2304), (1000, 512), (10, 1024), (32, 25), (3, 5),
              (1, 1), (512, 4608), (1, 70000), (7, 0)]
    Ws = [dg.he_normal(31, f"batch{i}", r, max(c, 1))[:, :c] * np.float32(0.3 + i) for i, (r, c) in enumerate(shapes)]
    Ws = [np.ascontiguousarray(w) for w in Ws]
    dev, items, outs = [], [], []
    for w in Ws:
        rows, cols = w.shape
        ld = twn.ld_for(max(cols, 1))
        Wd = dev_f32(w) if w.size else torch.zeros(4, dtype=torch.float32, device="cuda")
        stats = twn.new_stats()
        packed = torch.full((rows, ld // 16), -1, dtype=torch.int32, device="cuda")
        codes = torch.full((rows, max(cols, 1)), 7, dtype=torch.int8, device="cuda")[:, :cols].contiguous() if cols else None
        dev.append(Wd)
        items.append((Wd, rows, cols, stats, packed, ld, codes))
        outs.append((stats, packed, codes))
    ws = workspace(twn.ternarize_batch_workspace_bytes(len(items)))
    twn.ternarize_batch(items, 0.7, ws)
    torch.cuda.synchronize()
    for w, (stats, packed, codes) in zip(Ws, outs):
        rows, cols = w.shape
        ld = twn.ld_for(max(cols, 1))
        st1, packed1, codes1 = run_ternarize(w, 0.7, ld) if w.size else (None, None, None)
        st = twn.stats_to_host(stats)
        if w.size == 0:
            assert st["status"] == 0 and st["delta"] == 0.0 and st["alpha"] == 0.0
            assert not host_u32(packed).any()
            continue
        assert st == st1                                   # same reduction order: same bits
        assert np.array_equal(host_u32(packed), packed1)
        assert np.array_equal(codes.cpu().numpy(), codes1)
        ref, ref_codes = oracle.ternarize(w, 0.7)
        assert abs(st["delta"] - ref.delta) <= REL * ref.delta and abs(st["alpha"] - ref.alpha) <= REL * ref.alpha
        assert np.array_equal(host_u32(packed), oracle.pack(ref_codes.reshape(rows, cols), ld))


def test_batched_call_argument_checks():
    ws = workspace(twn.ternarize_batch_workspace_bytes(2))
    W = torch.zeros((1, 64), dtype=torch.float32, device="cuda")
    item = (W, 1, 64, twn.new_stats(), torch.zeros((1, 4), dtype=torch.int32, device="cuda"), 64, None)
    twn.ternarize_batch([], 0.7, ws)
    with pytest.raises(twn.TwnError):
        twn.ternarize_batch([item] * 33, 0.7, ws)               # more than 32 tensors
    with pytest.raises(twn.TwnError):
        twn.ternarize_batch([item] * 3, 0.7, ws)                # workspace sized for two
    bad = (W, 1, 64, twn.new_stats(), torch.zeros((1, 4), dtype=torch.int32, device="cuda"), 32, None)
    with pytest.raises(twn.TwnError):
        twn.ternarize_batch([bad], 0.7, ws)                     # pitch shorter than the row


def test_batched_transpose_equals_one_call_per_filter_bank():
    cases = [(64, 64, 3), (64, 128, 3), (128, 256, 1), (512, 1000, 1), (16, 24, 5)]
    items, want = [], []
    for i, (cin, cout, k) in enumerate(cases):
        K = k * k * cin
        codes = np.sign(dg.draw(41, f"tb{i}", cout * K, "normal")).astype(np.int8).reshape(cout, K)
        codes[np.abs(dg.draw(42, f"tbz{i}", cout * K, "normal").reshape(cout, K)) < 0.5] = 0
        ld, ld_b = twn.ld_for(K), twn.ld_for(k * k * cout)
        pf = dev_u32(oracle.pack(codes, ld))
        d = twn.conv_desc(1, 8, 8, cin, cout, k, 1, k // 2)
        one = torch.full((cin, ld_b // 16), -1, dtype=torch.int32, device="cuda")
        twn.transpose_codes(pf, ld, d, one, ld_b)
        out = torch.full((cin, ld_b // 16), -1, dtype=torch.int32, device="cuda")
        items.append((pf, ld, d, out, ld_b))
        # [Cout][taps][Cin] -> [Cin][taps][Cout]
        t = codes.reshape(cout, k * k, cin).transpose(2, 1, 0).reshape(cin, k * k * cout)
        want.append((one, oracle.pack(np.ascontiguousarray(t), ld_b)))
    twn.transpose_codes_batch(items)
    torch.cuda.synchronize()
    for (pf, ld, d, out, ld_b), (one, ref) in zip(items, want):
        assert torch.equal(out, one)
        assert np.array_equal(host_u32(out), ref)
