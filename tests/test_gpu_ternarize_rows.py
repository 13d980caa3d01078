"""GPU parity: twn_ternarize_rows / twn_rows_scale (Algorithm 1 as printed, one threshold and
one scale per filter) against the oracle, and the ternary contractions driven by per-filter scales.

Bar: packed codes and counts bit-exact per filter (elements within 1e-12*delta_r of a threshold
are counted and must be absent), delta_r and alpha_r within 1e-12 relative; contraction outputs
within 1e-4 * alpha_n * sum_k |x_k t_k| + 1e-6.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_1605_04711_b200 import datagen as dg
from paper_1605_04711_b200 import twn
from _gpu_util import dev_bf16, dev_f32, host_u32

pytestmark = pytest.mark.gpu

REL = 1e-12


def run_rows(W2d, factor=0.7, ld=None, want_i8=True, Wd=None):
    rows, cols = W2d.shape
    ld = twn.ld_for(cols) if ld is None else ld
    Wd = dev_f32(W2d) if Wd is None else Wd
    stats = twn.new_stats_rows(rows)
    packed = torch.full((rows, ld // 16), -1, dtype=torch.int32, device="cuda")
    codes = torch.full((rows, cols), 7, dtype=torch.int8, device="cuda") if want_i8 else None
    twn.ternarize_rows(Wd, factor, stats, packed, ld, codes)
    torch.cuda.synchronize()
    return stats, twn.stats_rows_to_host(stats), host_u32(packed), (codes.cpu().numpy() if want_i8 else None)


def check_rows(W2d, factor=0.7, ld=None, want_i8=True, Wd=None):
    rows, cols = W2d.shape
    ld = twn.ld_for(cols) if ld is None else ld
    stats, st, packed, codes = run_rows(W2d, factor, ld, want_i8, Wd)
    ref, ref_codes = oracle.ternarize_rows(W2d, factor)
    for r in range(rows):
        assert st[r]["status"] == 0
        assert ref[r].n_boundary == 0, "an element sits within 1e-12*delta of its filter's threshold"
        assert abs(st[r]["delta"] - ref[r].delta) <= REL * ref[r].delta
        assert abs(st[r]["alpha"] - ref[r].alpha) <= REL * ref[r].alpha
        assert abs(st[r]["sum_abs"] - ref[r].sum_abs) <= REL * ref[r].sum_abs
        assert (st[r]["n_neg"], st[r]["n_zero"], st[r]["n_pos"]) == (ref[r].n_neg, ref[r].n_zero, ref[r].n_pos)
    assert np.array_equal(packed, oracle.pack(ref_codes, ld))
    if want_i8:
        assert np.array_equal(codes, ref_codes)
    return stats, ref, ref_codes


# filter shapes of the LeNet-5 / VGG-7 / ResNet-18 layers, ragged ones, one longer than the
# on-chip limit (16384) and one that is not a multiple of four
@pytest.mark.parametrize("rows,cols", [(32, 25), (64, 147), (64, 576), (128, 1152), (256, 2304), (512, 4608),
                                       (1024, 8192), (10, 1024), (1000, 512), (3, 5), (1, 1), (5, 16), (7, 17),
                                       (4, 8196), (2, 40000), (3, 12289), (2, 16384), (2, 16388), (1500, 64)])
def test_filters_match_the_oracle(rows, cols):
    W = dg.he_normal(21, f"rows{rows}x{cols}", rows, cols)
    W *= np.linspace(0.05, 7.0, rows, dtype=np.float32)[:, None]
    check_rows(W)


@pytest.mark.parametrize("dist", ["normal", "laplace", "uniform"])
def test_distributions_and_paper_factor(dist):
    W = dg.draw(22, f"rows-{dist}", 96 * 1152, dist).reshape(96, 1152)
    check_rows(W, factor=0.75)
    check_rows(W, factor=0.7, want_i8=False)


def test_wider_row_pitch_is_zero_padded():
    W = dg.he_normal(23, "rows-ld", 9, 100)
    check_rows(W, ld=256)


def test_unaligned_matrix_takes_the_general_path():
    # a view that starts 4 bytes into an allocation: rows are no longer 16-byte aligned
    W = dg.he_normal(24, "rows-unaligned", 6, 64)
    flat = torch.zeros(6 * 64 + 1, dtype=torch.float32, device="cuda")
    flat[1:].copy_(torch.from_numpy(W.reshape(-1)))
    check_rows(W, Wd=flat[1:].view(6, 64), want_i8=False)


def test_zero_filter_nonfinite_filter_and_status_merge():
    W = dg.he_normal(25, "rows-edge", 5, 576)
    W[1] = 0.0
    W[3, 77] = np.nan
    stats, st, packed, codes = run_rows(W)
    assert st[1]["delta"] == 0.0 and st[1]["alpha"] == 0.0 and not codes[1].any() and st[1]["n_zero"] == 576
    assert st[3]["status"] == -4
    ref, ref_codes = oracle.ternarize_rows(W, 0.7)
    for r in (0, 2, 4):
        assert st[r]["status"] == 0 and np.array_equal(codes[r], ref_codes[r])
        assert abs(st[r]["alpha"] - ref[r].alpha) <= REL * ref[r].alpha
    scale = torch.empty(5, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    twn.rows_scale(stats, 5, None, scale, status)
    assert twn.read_status(status) == -4
    got = scale.cpu().numpy()
    for r in (0, 1, 2, 4):
        assert got[r] == np.float32(st[r]["alpha"])


def test_results_are_deterministic():
    W = dg.he_normal(26, "rows-det", 300, 2304)
    a = run_rows(W)
    b = run_rows(W)
    assert torch.equal(a[0], b[0]) and np.array_equal(a[2], b[2])


def test_empty_and_argument_checks():
    stats = twn.new_stats_rows(1)
    packed = torch.zeros((1, 4), dtype=torch.int32, device="cuda")
    twn.ternarize_rows(torch.zeros((0, 64), dtype=torch.float32, device="cuda"), 0.7, stats, packed, 64)
    W = torch.zeros((1, 64), dtype=torch.float32, device="cuda")
    with pytest.raises(twn.TwnError):
        twn.ternarize_rows(W, 0.7, stats, packed, 32)          # pitch shorter than the filter
    with pytest.raises(twn.TwnError):
        twn.ternarize_rows(W, -1.0, stats, packed, 64)


@pytest.mark.parametrize("case", [dict(B=2, H=12, W=12, Cin=64, Cout=96, k=3, s=1, p=1),
                                  dict(B=3, H=9, W=9, Cin=128, Cout=208, k=3, s=2, p=1),
                                  dict(B=4, H=1, W=1, Cin=512, Cout=40, k=1, s=1, p=0)])
def test_convolution_forward_and_backward_with_per_filter_scales(case):
    """Eq. 2 with the scales of Algorithm 1: forward Y = relu(bn_scale_n * alpha_n * (X * T_n) + shift_n)
    through twn_rows_scale; backward dX = sum_n alpha_n dz_n T_n with the alphas folded into the
    gradient by twn_act_bwd."""
    B, H, Wd_, Cin, Cout, k, s, p = (case[x] for x in ("B", "H", "W", "Cin", "Cout", "k", "s", "p"))
    K = k * k * Cin
    Wm = dg.he_normal(27, f"rows-conv{Cout}", Cout, K)
    Wm *= np.linspace(0.3, 3.0, Cout, dtype=np.float32)[:, None]
    ld = twn.ld_for(K)
    stats, ref, ref_codes = check_rows(Wm, want_i8=False)
    packed = torch.empty((Cout, ld // 16), dtype=torch.int32, device="cuda")
    twn.ternarize_rows(dev_f32(Wm), 0.7, stats, packed, ld)
    bn = dg.draw(27, "rows-bn", Cout, "normal", 1.0, 0.3)
    shift = dg.draw(27, "rows-shift", Cout, "normal", 0.0, 0.3)
    scale_d = torch.empty(Cout, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    twn.rows_scale(stats, Cout, dev_f32(bn), scale_d, status)
    alphas = np.array([r.alpha for r in ref])
    want_scale = (alphas.astype(np.float32) * bn).astype(np.float32)
    assert np.array_equal(scale_d.cpu().numpy(), want_scale)

    d = twn.conv_desc(B, H, Wd_, Cin, Cout, k, s, p)
    od = oracle.conv_desc(B, H, Wd_, Cin, Cout, k, s, p)
    codes4 = ref_codes.reshape(Cout, k, k, Cin)
    X = dg.draw_bf16(27, "rows-x", B * H * Wd_ * Cin, "normal").reshape(B, H, Wd_, Cin)
    Y = torch.empty((B, d.Ho, d.Wo, Cout), dtype=torch.float32, device="cuda")
    shift_d = dev_f32(shift)      # the epilogue struct keeps no reference: the tensors must outlive the call
    epi = twn.epilogue(scale_d, shift_d, None, relu=True, out_dtype=twn.F32)
    twn.conv2d_fwd(d, dev_bf16(X), packed, ld, None, epi, Y, status)
    Yr, A = oracle.conv2d_fwd(od, X, codes4, 1.0, scale=want_scale, shift=shift, relu=True)
    tol = 1e-4 * np.abs(want_scale.astype(np.float64)) * A + 1e-6
    assert np.all(np.abs(Y.cpu().numpy() - Yr) <= tol)

    # backward for data: dz_n = g_n * alpha_n (rounded to bf16 by twn_act_bwd), then the
    # transposed ternary convolution without a scalar alpha
    g = dg.draw_bf16(27, "rows-g", B * d.Ho * d.Wo * Cout, "normal", 0.0, 0.1).reshape(B, d.Ho, d.Wo, Cout)
    alpha_d = torch.empty(Cout, dtype=torch.float32, device="cuda")
    twn.rows_scale(stats, Cout, None, alpha_d, status)
    dz = torch.empty((B, d.Ho, d.Wo, Cout), dtype=torch.bfloat16, device="cuda")
    twn.act_bwd(dev_bf16(g), None, alpha_d, g.size, Cout, dz, None)
    dz_bits = dz.view(torch.int16).cpu().numpy().view(np.uint16)
    want_dz = dg.f32_to_bf16_bits((dg.bf16_bits_to_f64(g).astype(np.float32) * alphas.astype(np.float32)).astype(np.float32))
    assert np.array_equal(dg.bf16_bits_to_f64(dz_bits), dg.bf16_bits_to_f64(want_dz))
    ld_b = twn.ld_for(k * k * Cout)
    packed_b = torch.empty((Cin, ld_b // 16), dtype=torch.int32, device="cuda")
    twn.transpose_codes(packed, ld, d, packed_b, ld_b)
    dX = torch.empty((B, H, Wd_, Cin), dtype=torch.float32, device="cuda")
    twn.conv2d_bwd_data(d, dz, packed_b, ld_b, None, None, dX, status)
    dXr, Ab = oracle.conv2d_bwd_data(od, dz_bits, codes4, 1.0)
    assert np.all(np.abs(dX.cpu().numpy() - dXr) <= 1e-4 * Ab + 1e-6)
    assert twn.read_status(status) == 0
