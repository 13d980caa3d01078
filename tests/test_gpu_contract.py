"""GPU parity: twn_gemm / twn_conv2d_fwd / twn_conv2d_bwd_data against the oracle.

Bar (per output element): |y - y_ref| <= 1e-4 * alpha * |scale_n| * A + 1e-6 with
A = sum_k |x_k t_k| from the oracle; bf16 outputs must equal the correctly rounded
fp32 result up to one more bf16 rounding of a value inside that tolerance.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_1605_04711_b200 import datagen as dg
from paper_1605_04711_b200 import twn
from _gpu_util import dev_bf16, dev_f32, dev_u32, host_bf16_bits, workspace

pytestmark = pytest.mark.gpu


def ternarized(seed, name, rows, cols, factor=0.7):
    """Master weights -> (alpha, int8 codes [rows, cols], device packed, ld, device stats) via the oracle
    for the reference side and via twn_ternarize for the device side (both must agree)."""
    W = dg.he_normal(seed, name, rows, cols)
    ref, codes = oracle.ternarize(W, factor)
    ld = twn.ld_for(cols)
    stats = twn.new_stats()
    packed = torch.empty((rows, ld // 16), dtype=torch.int32, device="cuda")
    twn.ternarize(dev_f32(W), factor, stats, packed, ld, None,
                  workspace(twn.ternarize_workspace_bytes()), rows=rows, cols=cols)
    assert np.array_equal(packed.cpu().numpy().view(np.uint32), oracle.pack(codes.reshape(rows, cols), ld))
    return ref.alpha, codes.reshape(rows, cols), packed, ld, stats


def assert_within(y, y_ref, A, alpha, scale=None):
    tol = 1e-4 * alpha * A
    if scale is not None:
        tol = tol * np.abs(scale.astype(np.float64))
    tol = tol + 1e-6
    err = np.abs(y.astype(np.float64) - y_ref)
    bad = ~(err <= tol)
    assert not bad.any(), f"{int(bad.sum())} outputs out of tolerance, worst err/tol = {np.nanmax(err / tol):.3g}"


GEMM_SHAPES = [
    (128, 128, 64), (1, 1, 8), (7, 3, 16), (100, 10, 512), (129, 257, 200), (300, 200, 136),
    (128, 512, 1024), (1000, 130, 72), (64, 1000, 512), (128, 1024, 8192), (515, 64, 576),
    # enough tiles for the 256-pixel kernel, with ragged edges in both dimensions
    (8192, 640, 512), (40000, 130, 200), (20001, 257, 1152),
]


@pytest.mark.parametrize("M,N,K", GEMM_SHAPES)
def test_gemm_matches_oracle(M, N, K):
    alpha, codes, packed, ld, stats = ternarized(0, f"g{N}x{K}", N, K)
    X = dg.draw_bf16(1, f"gx{M}x{K}", M * K, "normal").reshape(M, K)
    Y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    twn.gemm(dev_bf16(X), K, packed, ld, stats, M, N, K, None, Y, N, status)
    Yr, A = oracle.gemm(X, codes, alpha)
    assert twn.read_status(status) == 0
    assert_within(Y.cpu().numpy(), Yr, A, alpha)


def test_gemm_leading_dimensions_and_untouched_padding():
    M, N, K, ldx, ldy = 70, 50, 100, 104, 64
    alpha, codes, packed, ld, stats = ternarized(2, "ldw", N, K)
    X = dg.draw_bf16(2, "ldx", M * ldx, "normal").reshape(M, ldx)
    Y = torch.full((M, ldy), -7.0, dtype=torch.float32, device="cuda")
    twn.gemm(dev_bf16(X), ldx, packed, ld, stats, M, N, K, None, Y, ldy)
    Yr, A = oracle.gemm(np.ascontiguousarray(X[:, :K]), codes, alpha)
    Yh = Y.cpu().numpy()
    assert_within(Yh[:, :N], Yr, A, alpha)
    assert np.all(Yh[:, N:] == -7.0)


@pytest.mark.parametrize("out_bf16", [False, True])
def test_gemm_epilogue(out_bf16):
    M, N, K = 200, 150, 256
    alpha, codes, packed, ld, stats = ternarized(3, "ew", N, K)
    X = dg.draw_bf16(3, "ex", M * K, "normal").reshape(M, K)
    scale = dg.draw(3, "es", N, "normal", 1.0, np.sqrt(0.1)); shift = dg.draw(3, "eb", N, "normal", 0.0, np.sqrt(0.1))
    res_bits = dg.draw_bf16(3, "er", M * N, "normal").reshape(M, N)
    res = dev_bf16(res_bits)
    sd, bd = dev_f32(scale), dev_f32(shift)
    epi = twn.epilogue(sd, bd, res, relu=True, out_dtype=twn.BF16 if out_bf16 else twn.F32)
    Y = torch.zeros((M, N), dtype=torch.bfloat16 if out_bf16 else torch.float32, device="cuda")
    twn.gemm(dev_bf16(X), K, packed, ld, stats, M, N, K, epi, Y, N)
    Yr, A = oracle.gemm(X, codes, alpha, scale, shift, dg.bf16_bits_to_f64(res_bits), relu=True)
    if out_bf16:
        got = dg.bf16_bits_to_f64(host_bf16_bits(Y))
        tol = 1e-4 * alpha * A * np.abs(scale.astype(np.float64)) + 1e-6
        # a correctly rounded bf16 of any value within tol of the reference
        lo = dg.bf16_bits_to_f64(dg.f32_to_bf16_bits((Yr - tol).astype(np.float32)))
        hi = dg.bf16_bits_to_f64(dg.f32_to_bf16_bits((Yr + tol).astype(np.float32)))
        assert np.all((got >= np.minimum(lo, hi) - 1e-6) & (got <= np.maximum(lo, hi) + 1e-6))
    else:
        assert_within(Y.cpu().numpy(), Yr, A, alpha, scale)


def test_gemm_alpha_null_means_one_and_zero_alpha():
    M, N, K = 64, 32, 64
    alpha, codes, packed, ld, stats = ternarized(4, "aw", N, K)
    X = dg.draw_bf16(4, "ax", M * K, "normal").reshape(M, K)
    Y = torch.zeros((M, N), dtype=torch.float32, device="cuda")
    twn.gemm(dev_bf16(X), K, packed, ld, None, M, N, K, None, Y, N)
    Yr, A = oracle.gemm(X, codes, 1.0)
    assert_within(Y.cpu().numpy(), Yr, A, 1.0)


def test_gemm_host_errors():
    X = torch.zeros((8, 64), dtype=torch.bfloat16, device="cuda")
    T = torch.zeros((8, 4), dtype=torch.int32, device="cuda")
    Y = torch.zeros((8, 8), dtype=torch.float32, device="cuda")
    with pytest.raises(twn.TwnError) as e:
        twn.gemm(X, 60, T, 64, None, 8, 8, 64, None, Y, 8)
    assert e.value.code == -1
    with pytest.raises(twn.TwnError) as e:
        twn.gemm(X, 68, T, 64, None, 8, 8, 64, None, Y, 8)
    assert e.value.code == -2
    with pytest.raises(twn.TwnError) as e:
        twn.gemm(X, 64, T, 32, None, 8, 8, 64, None, Y, 8)
    assert e.value.code == -1


CONV_CASES = [
    # B, H, W, Cin, Cout, k, stride, pad
    (2, 8, 8, 64, 128, 3, 1, 1),
    (3, 7, 7, 64, 64, 3, 1, 1),
    (2, 12, 12, 32, 64, 5, 1, 0),
    (1, 14, 14, 128, 256, 3, 2, 1),
    (2, 9, 11, 16, 40, 3, 2, 1),
    (2, 16, 16, 64, 128, 1, 2, 0),
    (5, 6, 6, 8, 24, 1, 1, 0),
    (1, 33, 20, 80, 130, 3, 1, 1),
    (2, 10, 10, 48, 16, 3, 1, 0),
    (1, 15, 15, 16, 32, 7, 2, 3),
    # enough pixels for the 256-pixel kernel
    (8, 64, 64, 64, 256, 3, 1, 1),
    (37, 28, 28, 128, 256, 3, 2, 1),
    # shapes for which the tile cost model picks the 192-pixel kernel (8 x 8 x 3 pixel tiles): ragged
    # in width, height (60 of 64) and batch (5 of 6); 64 and 96 channels (half-empty channel tile)
    (5, 60, 60, 64, 64, 3, 1, 1),
    (5, 62, 59, 64, 96, 3, 1, 1),
    (64, 14, 14, 64, 384, 3, 1, 1),
]


@pytest.mark.parametrize("case", CONV_CASES)
def test_conv_fwd_matches_oracle(case):
    B, H, W, Cin, Cout, k, s, p = case
    alpha, codes, packed, ld, stats = ternarized(5, f"c{case}", Cout, k * k * Cin)
    d = twn.conv_desc(B, H, W, Cin, Cout, k, s, p)
    X = dg.draw_bf16(5, f"cx{case}", B * H * W * Cin, "normal").reshape(B, H, W, Cin)
    Y = torch.full((B, d.Ho, d.Wo, Cout), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    twn.conv2d_fwd(d, dev_bf16(X), packed, ld, stats, None, Y, status)
    Yr, A = oracle.conv2d_fwd(oracle.conv_desc(B, H, W, Cin, Cout, k, s, p), X, codes, alpha)
    assert twn.read_status(status) == 0
    assert_within(Y.cpu().numpy(), Yr, A, alpha)


def test_conv_fwd_epilogue_affine_relu_residual_bf16_out():
    B, H, W, Cin, Cout, k, s, p = 2, 8, 8, 64, 64, 3, 1, 1
    alpha, codes, packed, ld, stats = ternarized(6, "cew", Cout, k * k * Cin)
    d = twn.conv_desc(B, H, W, Cin, Cout, k, s, p)
    X = dg.draw_bf16(6, "cex", B * H * W * Cin, "normal").reshape(B, H, W, Cin)
    scale = dg.draw(6, "ces", Cout, "normal", 1.0, np.sqrt(0.1)); shift = dg.draw(6, "ceb", Cout, "normal", 0.0, np.sqrt(0.1))
    res = dg.draw(6, "cer", B * H * W * Cout, "normal").reshape(B, H, W, Cout)
    sd, bd, rd = dev_f32(scale), dev_f32(shift), dev_f32(res)
    Y = torch.zeros((B, H, W, Cout), dtype=torch.float32, device="cuda")
    twn.conv2d_fwd(d, dev_bf16(X), packed, ld, stats, twn.epilogue(sd, bd, rd, relu=True), Y)
    Yr, A = oracle.conv2d_fwd(oracle.conv_desc(B, H, W, Cin, Cout, k, s, p), X, codes, alpha, scale, shift,
                              res.astype(np.float64), relu=True)
    assert_within(Y.cpu().numpy(), Yr, A, alpha, scale)


@pytest.mark.parametrize("case", CONV_CASES)
def test_conv_bwd_data_matches_oracle(case):
    B, H, W, Cin, Cout, k, s, p = case
    if Cout % 16 != 0 and k > 1 or Cout % 8 != 0:
        # The backward pass reduces over Cout: its tensor copies need channel runs of 16 codes (8 for
        # a 1x1 filter), as the forward pass needs them of Cin.  Such a layer is refused on the host.
        d = twn.conv_desc(B, H, W, Cin, Cout, k, s, p)
        ld_b = twn.ld_for(k * k * Cout)
        buf = torch.zeros((max(Cin, 1), ld_b // 16), dtype=torch.int32, device="cuda")
        dZ = torch.zeros((B, d.Ho, d.Wo, Cout), dtype=torch.bfloat16, device="cuda")
        dX = torch.zeros((B, H, W, Cin), dtype=torch.float32, device="cuda")
        with pytest.raises(twn.TwnError) as e:
            twn.conv2d_bwd_data(d, dZ, buf, ld_b, None, None, dX)
        assert e.value.code == -2
        return
    alpha, codes, packed, ld, stats = ternarized(7, f"b{case}", Cout, k * k * Cin)
    d = twn.conv_desc(B, H, W, Cin, Cout, k, s, p)
    ld_b = twn.ld_for(k * k * Cout)
    packed_b = torch.empty((Cin, ld_b // 16), dtype=torch.int32, device="cuda")
    twn.transpose_codes(packed, ld, d, packed_b, ld_b)
    dZ = dg.draw_bf16(7, f"bz{case}", B * d.Ho * d.Wo * Cout, "normal").reshape(B, d.Ho, d.Wo, Cout)
    dX = torch.full((B, H, W, Cin), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    twn.conv2d_bwd_data(d, dev_bf16(dZ), packed_b, ld_b, stats, None, dX, status)
    dXr, A = oracle.conv2d_bwd_data(oracle.conv_desc(B, H, W, Cin, Cout, k, s, p), dZ,
                                    codes.reshape(Cout, k, k, Cin), alpha)
    assert twn.read_status(status) == 0
    assert_within(dX.cpu().numpy(), dXr, A, alpha)


def test_bwd_data_adds_a_second_gradient_branch_through_the_residual():
    B, H, W, Cin, Cout, k, s, p = 2, 8, 8, 64, 128, 1, 2, 0
    alpha, codes, packed, ld, stats = ternarized(8, "rw", Cout, Cin)
    d = twn.conv_desc(B, H, W, Cin, Cout, k, s, p)
    ld_b = twn.ld_for(Cout)
    packed_b = torch.empty((Cin, ld_b // 16), dtype=torch.int32, device="cuda")
    twn.transpose_codes(packed, ld, d, packed_b, ld_b)
    dZ = dg.draw_bf16(8, "rz", B * d.Ho * d.Wo * Cout, "normal").reshape(B, d.Ho, d.Wo, Cout)
    other = dg.draw(8, "ro", B * H * W * Cin, "normal").reshape(B, H, W, Cin)
    od = dev_f32(other)
    dX = torch.full((B, H, W, Cin), float("nan"), dtype=torch.float32, device="cuda")
    twn.conv2d_bwd_data(d, dev_bf16(dZ), packed_b, ld_b, stats, twn.epilogue(residual=od), dX)
    dXr, A = oracle.conv2d_bwd_data(oracle.conv_desc(B, H, W, Cin, Cout, k, s, p), dZ,
                                    codes.reshape(Cout, k, k, Cin), alpha)
    assert_within(dX.cpu().numpy(), dXr + other.astype(np.float64), A, alpha)


@pytest.mark.parametrize("gate_dtype,out_dtype", [("bf16", "bf16"), ("f32", "f32"), ("bf16", "f32")])
@pytest.mark.parametrize("stride", [1, 2])
def test_bwd_data_gated_by_the_lower_layers_output(gate_dtype, out_dtype, stride):
    """TWN_RESIDUAL_GATE: the backward-for-data pass writes the lower layer's dZ, i.e. the gradient
    times that layer's scale where its (ReLU) output is positive and 0 elsewhere."""
    B, H, W, Cin, Cout, k, p = 3, 10, 10, 96, 64, 3, 1
    alpha, codes, packed, ld, stats = ternarized(9, f"gw{stride}", Cout, k * k * Cin)
    d = twn.conv_desc(B, H, W, Cin, Cout, k, stride, p)
    ld_b = twn.ld_for(k * k * Cout)
    packed_b = torch.empty((Cin, ld_b // 16), dtype=torch.int32, device="cuda")
    twn.transpose_codes(packed, ld, d, packed_b, ld_b)
    dZ = dg.draw_bf16(9, f"gz{stride}", B * d.Ho * d.Wo * Cout, "normal").reshape(B, d.Ho, d.Wo, Cout)
    ybits = dg.draw_bf16(9, "gy", B * H * W * Cin, "normal").reshape(B, H, W, Cin)
    y = np.maximum(dg.bf16_bits_to_f64(ybits), 0.0)                  # a ReLU output: about half zeros
    scale = dg.draw(9, "gs", Cin, "normal", 1.0, 0.3)
    yd = dev_bf16(dg.f32_to_bf16_bits(y.astype(np.float32))) if gate_dtype == "bf16" else dev_f32(y)
    sd = dev_f32(scale)
    tdt = torch.bfloat16 if out_dtype == "bf16" else torch.float32
    dX = torch.full((B, H, W, Cin), float("nan"), dtype=tdt, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    epi = twn.epilogue(scale=sd, residual=yd, out_dtype=twn.BF16 if out_dtype == "bf16" else twn.F32,
                       residual_op=twn.RESIDUAL_GATE)
    twn.conv2d_bwd_data(d, dev_bf16(dZ), packed_b, ld_b, stats, epi, dX, status)
    dXr, A = oracle.conv2d_bwd_data(oracle.conv_desc(B, H, W, Cin, Cout, k, stride, p), dZ,
                                    codes.reshape(Cout, k, k, Cin), alpha)
    want = np.where(y > 0, dXr * scale.astype(np.float64), 0.0)
    tol = 1e-4 * alpha * np.abs(scale.astype(np.float64)) * A + 1e-6
    assert twn.read_status(status) == 0
    got = dX.float().cpu().numpy().astype(np.float64)
    if out_dtype == "bf16":
        tol = tol + 2.0 ** -8 * (np.abs(want) + tol)
    assert np.all(np.abs(got - want) <= tol)
    assert np.all(got[y <= 0] == 0.0)


def test_epilogue_rejects_an_unknown_residual_op():
    alpha, codes, packed, ld, stats = ternarized(9, "gbad", 64, 64)
    X = torch.zeros((8, 64), dtype=torch.bfloat16, device="cuda")
    Y = torch.zeros((8, 64), dtype=torch.float32, device="cuda")
    epi = twn.epilogue(residual=Y, residual_op=7)
    with pytest.raises(twn.TwnError):
        twn.gemm(X, 64, packed, ld, stats, 8, 64, 64, epi, Y, 64)


SWEEP = [(K, N, M) for (K, N) in [(512, 512), (1152, 128), (2304, 256), (4608, 512), (4096, 4096)]
         for M in (128, 1024, 4096, 16384)]


@pytest.mark.parametrize("K,N,M", SWEEP)
def test_gemm_sweep_full_sizes_on_sampled_rows(K, N, M):
    """The GEMM sweep at its full sizes: the oracle evaluates 64 seeded rows plus every row next
    to a 128/256-row tile boundary of the first and last tiles."""
    alpha, codes, packed, ld, stats = ternarized(0, f"sweep{N}x{K}", N, K)
    X = dg.draw_bf16(1, f"sweepx{M}x{K}", M * K, "normal").reshape(M, K)
    Y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    twn.gemm(dev_bf16(X), K, packed, ld, stats, M, N, K, None, Y, N, status)
    rng = np.random.default_rng(M + K)
    rows = np.concatenate([rng.integers(0, M, 64), [0, 127, 128, 255, 256, M - 257, M - 256, M - 129, M - 128, M - 1]])
    rows = np.unique(rows[(rows >= 0) & (rows < M)])
    Yr, A = oracle.gemm(np.ascontiguousarray(X[rows]), codes, alpha)
    assert twn.read_status(status) == 0
    Yh = Y.cpu().numpy()
    assert not np.isnan(Yh).any()
    assert_within(Yh[rows], Yr, A, alpha)
