"""GPU parity for binary precision weights (Sec. 3, the BPWN baseline): twn_binarize against the oracle
(sign codes and 1-bit words to the bit, scale to 1e-12) and the contractions on 1-bit codes
(twn_gemm_b1, twn_conv2d_fwd_b1, twn_conv2d_bwd_data_b1) against the oracle's fp64 contractions on the
same +-1 codes: |y - y_ref| <= 1e-4 * alpha * |scale_n| * A + 1e-6 with A = sum_k |x_k b_k|."""
import numpy as np
import pytest
import torch

import oracle
from paper_1605_04711_b200 import datagen as dg
from paper_1605_04711_b200 import twn
from _gpu_util import dev_bf16, dev_f32, host_u32, host_bf16_bits, workspace
from test_gpu_narrow import check

pytestmark = pytest.mark.gpu


def binarized(seed, name, rows, cols, dist="he"):
    W = dg.he_normal(seed, name, rows, cols) if dist == "he" else dg.draw(seed, name, rows * cols, dist).reshape(rows, cols)
    ref, codes = oracle.binarize(W)
    ld = twn.ld_for_b1(cols)
    stats = twn.new_stats()
    packed = torch.full((rows, ld // 32), -1, dtype=torch.int32, device="cuda")
    twn.binarize(dev_f32(W), stats, packed, ld, workspace(twn.binarize_workspace_bytes()), rows=rows, cols=cols)
    st = twn.stats_to_host(stats)
    assert st["status"] == 0
    assert np.array_equal(host_u32(packed), oracle.pack1(codes.reshape(rows, cols), ld))
    assert abs(st["alpha"] - ref.alpha) <= 1e-12 * ref.alpha
    assert abs(st["sum_abs"] - ref.sum_abs) <= 1e-12 * ref.sum_abs
    assert (st["n_neg"], st["n_zero"], st["n_pos"]) == (ref.n_neg, 0, ref.n_pos) and st["delta"] == 0.0
    return ref.alpha, codes.reshape(rows, cols), packed, ld, stats


@pytest.mark.parametrize("rows,cols,dist", [(1, 1, "normal"), (1, 31, "uniform"), (3, 100, "laplace"), (64, 1152, "he"),
                                            (1, 128 * 4001, "normal"), (7, 1000, "normal"), (512, 4608, "he"),
                                            (1, 10_000_000, "normal")])
def test_binarize_matches_oracle(rows, cols, dist):
    binarized(30, f"b{rows}x{cols}", rows, cols, dist)


def test_binarize_zeros_negative_zero_nonfinite_and_determinism():
    W = np.array([[0.0, -0.0, 1.0, -1.0, 1e-45, -1e-45, 3.5, -2.25]], dtype=np.float32)
    ref, codes = oracle.binarize(W)
    assert codes.tolist() == [[1, 1, 1, -1, 1, -1, 1, -1]]
    ws = workspace(twn.binarize_workspace_bytes())
    stats = twn.new_stats()
    packed = torch.zeros((1, 4), dtype=torch.int32, device="cuda")
    twn.binarize(dev_f32(W), stats, packed, 128, ws, rows=1, cols=8)
    assert np.array_equal(host_u32(packed), oracle.pack1(codes, 128))
    back = torch.zeros((1, 8), dtype=torch.int8, device="cuda")
    twn.unpack_b1(packed, 1, 8, 128, back)
    assert np.array_equal(back.cpu().numpy(), codes)
    Wn = W.copy(); Wn[0, 2] = np.inf
    twn.binarize(dev_f32(Wn), stats, packed, 128, ws, rows=1, cols=8)
    assert twn.stats_to_host(stats)["status"] == -4
    # same bits on a second run, same workspace
    big = dg.draw(31, "bdet", 3_000_064, "normal").reshape(1, -1)
    outs = []
    for _ in range(2):
        st = twn.new_stats()
        p = torch.empty((1, big.size // 32), dtype=torch.int32, device="cuda")
        twn.binarize(dev_f32(big), st, p, big.size, ws, rows=1, cols=big.size)
        outs.append((twn.stats_to_host(st), host_u32(p)))
    assert outs[0][0] == outs[1][0] and np.array_equal(outs[0][1], outs[1][1])


def test_binarize_host_errors():
    W = torch.zeros(256, dtype=torch.float32, device="cuda")
    stats = twn.new_stats()
    packed = torch.zeros(8, dtype=torch.int32, device="cuda")
    ws = workspace(twn.binarize_workspace_bytes())
    with pytest.raises(twn.TwnError) as e:
        twn.binarize(W, stats, packed, 64, ws, rows=1, cols=64)          # pitch not a multiple of 128
    assert e.value.code == -1
    with pytest.raises(twn.TwnError) as e:
        twn.binarize(W, stats, packed, 256, ws[:64], rows=1, cols=256)   # scratch too small
    assert e.value.code == -3


SWEEP = [(K, N, M) for (K, N) in [(512, 512), (1152, 128), (2304, 256), (4608, 512), (4096, 4096)]
         for M in (128, 1024, 4096, 16384)]


@pytest.mark.parametrize("K,N,M", SWEEP + [(200, 130, 515), (576, 64, 3000), (64, 16, 129)])
def test_binary_gemm_sweep_on_sampled_rows(K, N, M):
    alpha, codes, packed, ld, stats = binarized(32, f"bg{N}x{K}", N, K)
    X = dg.draw_bf16(33, f"bgx{M}x{K}", M * K, "normal").reshape(M, K)
    Y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    twn.gemm_b1(dev_bf16(X), K, packed, ld, stats, M, N, K, None, Y, N, status)
    rng = np.random.default_rng(M + K)
    rows = np.unique(np.concatenate([rng.integers(0, M, 48), [0, 127, 128, 255, 256, M - 257, M - 256, M - 129, M - 128, M - 1]]))
    rows = rows[(rows >= 0) & (rows < M)]
    Yr, A = oracle.gemm(np.ascontiguousarray(X[rows]), codes, alpha)
    assert twn.read_status(status) == 0
    Yh = Y.cpu().numpy()
    assert not np.isnan(Yh).any()
    check(Y[torch.from_numpy(rows).cuda()], Yr, 1e-4 * alpha * A + 1e-6, False)


# B, H, W, Cin, Cout, k, stride, pad: the 3x3 layers of the VGG-7 shape (batch reduced to keep the oracle
# within seconds), ragged and narrow cases
CONV = [(8, 32, 32, 128, 128, 3, 1, 1), (8, 16, 16, 256, 256, 3, 1, 1), (16, 8, 8, 512, 512, 3, 1, 1),
        (3, 13, 9, 64, 64, 3, 1, 1), (2, 9, 11, 32, 40, 3, 2, 1), (2, 16, 16, 64, 128, 1, 2, 0), (5, 20, 18, 96, 48, 3, 1, 1)]


@pytest.mark.parametrize("case", CONV)
def test_binary_conv_fwd_with_epilogue(case):
    B, H, W, Cin, Cout, k, s, p = case
    alpha, codes, packed, ld, stats = binarized(34, f"bc{case}", Cout, k * k * Cin)
    d = twn.conv_desc(B, H, W, Cin, Cout, k, s, p)
    od = oracle.conv_desc(B, H, W, Cin, Cout, k, s, p)
    X = dg.draw_bf16(34, f"bcx{case}", B * H * W * Cin, "normal").reshape(B, H, W, Cin)
    scale = dg.draw(34, "bcs", Cout, "normal", 1.0, 0.3); shift = dg.draw(34, "bcb", Cout, "normal", 0.0, 0.3)
    sd, bd = dev_f32(scale), dev_f32(shift)
    Y = torch.full((B, d.Ho, d.Wo, Cout), float("nan"), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    twn.conv2d_fwd_b1(d, dev_bf16(X), packed, ld, stats, twn.epilogue(sd, bd, None, relu=True, out_dtype=twn.BF16), Y, status)
    want, A = oracle.conv2d_fwd(od, X, codes.reshape(Cout, k, k, Cin), alpha, scale, shift, None, relu=True)
    assert twn.read_status(status) == 0
    check(Y, want, 1e-4 * alpha * A * np.abs(scale.astype(np.float64)) + 1e-6, True)


@pytest.mark.parametrize("case", [(4, 16, 16, 128, 128, 3, 1, 1), (3, 14, 14, 64, 128, 3, 2, 1), (2, 16, 16, 64, 128, 1, 2, 0),
                                  (3, 12, 12, 64, 64, 3, 1, 1)])
def test_binary_conv_bwd_data(case):
    B, H, W, Cin, Cout, k, s, p = case
    alpha, codes, packed, ld, stats = binarized(35, f"bb{case}", Cout, k * k * Cin)
    d = twn.conv_desc(B, H, W, Cin, Cout, k, s, p)
    ld_b = twn.ld_for_b1(k * k * Cout)
    packed_b = torch.full((Cin, ld_b // 32), -1, dtype=torch.int32, device="cuda")
    twn.transpose_codes_b1(packed, ld, d, packed_b, ld_b)
    # the re-layout against the oracle's packing of the transposed code tensor
    tr = codes.reshape(Cout, k * k, Cin).transpose(2, 1, 0).reshape(Cin, k * k * Cout)
    assert np.array_equal(host_u32(packed_b), oracle.pack1(tr, ld_b))
    dZ = dg.draw_bf16(35, f"bbz{case}", B * d.Ho * d.Wo * Cout, "normal").reshape(B, d.Ho, d.Wo, Cout)
    dX = torch.full((B, H, W, Cin), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    twn.conv2d_bwd_data_b1(d, dev_bf16(dZ), packed_b, ld_b, stats, None, dX, status)
    dXr, A = oracle.conv2d_bwd_data(oracle.conv_desc(B, H, W, Cin, Cout, k, s, p), dZ, codes.reshape(Cout, k, k, Cin), alpha)
    assert twn.read_status(status) == 0
    check(dX, dXr, 1e-4 * alpha * A + 1e-6, False)


def test_binary_contractions_refuse_what_the_format_cannot_address():
    d = twn.conv_desc(2, 8, 8, 48, 64, 3, 1, 1)          # 3x3 with Cin % 32 != 0
    X = torch.zeros((2, 8, 8, 48), dtype=torch.bfloat16, device="cuda")
    T = torch.zeros((64, 512 // 32), dtype=torch.int32, device="cuda")
    Y = torch.zeros((2, 8, 8, 64), dtype=torch.float32, device="cuda")
    with pytest.raises(twn.TwnError) as e:
        twn.conv2d_fwd_b1(d, X, T, 512, None, None, Y)
    assert e.value.code == -2
    with pytest.raises(twn.TwnError) as e:
        twn.gemm_b1(X.view(128, 48), 48, T, 64, None, 128, 64, 48, None, Y.view(128, 64), 64)    # pitch not a multiple of 128
    assert e.value.code == -1
