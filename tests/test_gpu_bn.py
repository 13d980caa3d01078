"""GPU parity: batch statistics out of the convolution epilogue (twn_conv2d_fwd_bn) and the affine
derived from them (twn_bn_finalize), against the fp64 oracle.

Tolerance of a sum over the n outputs of a channel: every output z may be off by its own bound
t = 1e-4 * alpha * |scale| * A + 1e-6, and the kernel adds at most a tile's pixels (256) per thread in fp32
before it goes to fp64: |S - S_ref| <= sum t + 2^-15 * sum |z|, and for the squares
|Q - Q_ref| <= sum (2 |z| t + t^2) + 2^-15 * sum z^2."""
import numpy as np
import pytest
import torch

import oracle
from paper_1605_04711_b200 import datagen as dg
from paper_1605_04711_b200 import twn
from _gpu_util import dev_bf16, dev_f32, workspace
from test_gpu_contract import ternarized

pytestmark = pytest.mark.gpu

CASES = [  # B, H, W, Cin, Cout, k, stride, pad, affine
    (2, 8, 8, 64, 128, 3, 1, 1, False),
    (3, 7, 9, 64, 64, 3, 1, 1, True),        # a narrow layer: statistics come from the general kernel
    (5, 20, 18, 32, 40, 3, 1, 1, True),      # ragged in every dimension, channels not a multiple of 32
    (2, 16, 16, 128, 256, 3, 2, 1, False),
    (16, 28, 28, 128, 128, 3, 1, 1, True),   # several tiles per block
    (4, 14, 14, 256, 384, 1, 1, 0, False),   # three channel tiles
]


@pytest.mark.parametrize("case", CASES)
def test_conv_fwd_bn_statistics(case):
    B, H, W, Cin, Cout, k, s, p, affine = case
    alpha, codes, packed, ld, stats = ternarized(41, f"bn{case}", Cout, k * k * Cin)
    d = twn.conv_desc(B, H, W, Cin, Cout, k, s, p)
    od = oracle.conv_desc(B, H, W, Cin, Cout, k, s, p)
    X = dg.draw_bf16(41, f"bnx{case}", B * H * W * Cin, "normal").reshape(B, H, W, Cin)
    scale = dg.draw(41, "bns", Cout, "normal", 1.0, 0.3) if affine else None
    shift = dg.draw(41, "bnb", Cout, "normal", 0.5, 0.3) if affine else None
    sd = dev_f32(scale) if affine else None
    bd = dev_f32(shift) if affine else None
    epi = twn.epilogue(sd, bd, None, relu=True, out_dtype=twn.BF16)
    Y = torch.full((B, d.Ho, d.Wo, Cout), float("nan"), dtype=torch.bfloat16, device="cuda")
    bsum = torch.full((Cout,), float("nan"), dtype=torch.float64, device="cuda")
    bsq = torch.full((Cout,), float("nan"), dtype=torch.float64, device="cuda")
    ws = workspace(twn.conv2d_fwd_bn_workspace_bytes(d))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    outs = []
    for _ in range(2):
        twn.conv2d_fwd_bn(d, dev_bf16(X), packed, ld, stats, epi, Y, bsum, bsq, ws, status)
        outs.append((bsum.cpu().numpy().copy(), bsq.cpu().numpy().copy()))
    assert twn.read_status(status) == 0
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])      # deterministic
    # z: before the ReLU; the stored output: after it
    Z, A = oracle.conv2d_fwd(od, X, codes.reshape(Cout, k, k, Cin), alpha, scale, shift, None, relu=False)
    t = 1e-4 * alpha * A * (np.abs(scale.astype(np.float64)) if affine else 1.0) + 1e-6
    S, Q = oracle.bn_stats(Z)
    tol_s = t.reshape(-1, Cout).sum(0) + 2.0 ** -15 * np.abs(Z).reshape(-1, Cout).sum(0)
    tol_q = (2 * np.abs(Z) * t + t * t).reshape(-1, Cout).sum(0) + 2.0 ** -15 * (Z * Z).reshape(-1, Cout).sum(0)
    assert np.all(np.abs(outs[0][0] - S) <= tol_s), np.max(np.abs(outs[0][0] - S) / tol_s)
    assert np.all(np.abs(outs[0][1] - Q) <= tol_q), np.max(np.abs(outs[0][1] - Q) / tol_q)
    # the convolution output itself is unchanged by the statistics
    Y2 = torch.empty_like(Y)
    twn.conv2d_fwd(d, dev_bf16(X), packed, ld, stats, epi, Y2, status)
    assert torch.equal(Y.view(torch.int16), Y2.view(torch.int16))
    # the affine of the normalisation
    n = B * d.Ho * d.Wo
    gamma = dg.draw(42, "bngam", Cout, "normal", 1.0, 0.2); beta = dg.draw(42, "bnbet", Cout, "normal", 0.0, 0.2)
    gd, btd = dev_f32(gamma), dev_f32(beta)
    sc_o = torch.empty(Cout, dtype=torch.float32, device="cuda"); sh_o = torch.empty_like(sc_o)
    mean_o = torch.empty(Cout, dtype=torch.float64, device="cuda"); var_o = torch.empty_like(mean_o)
    twn.bn_finalize(bsum, bsq, n, Cout, gd, btd, 1e-5, sc_o, sh_o, mean_o, var_o)
    mean, var, sc, sh = oracle.bn_affine(outs[0][0], outs[0][1], n, gamma, beta, 1e-5)
    np.testing.assert_allclose(mean_o.cpu().numpy(), mean, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(var_o.cpu().numpy(), var, rtol=1e-9, atol=1e-14)
    np.testing.assert_allclose(sc_o.cpu().numpy(), sc, rtol=2e-7)
    np.testing.assert_allclose(sh_o.cpu().numpy(), sh, rtol=2e-7, atol=1e-7)


def test_conv_fwd_bn_refuses_a_small_workspace():
    d = twn.conv_desc(2, 8, 8, 64, 128, 3, 1, 1)
    X = torch.zeros((2, 8, 8, 64), dtype=torch.bfloat16, device="cuda")
    T = torch.zeros((128, 576 // 16), dtype=torch.int32, device="cuda")
    Y = torch.zeros((2, 8, 8, 128), dtype=torch.float32, device="cuda")
    s1 = torch.zeros(128, dtype=torch.float64, device="cuda")
    with pytest.raises(twn.TwnError) as e:
        twn.conv2d_fwd_bn(d, X, T, 576, None, None, Y, s1, s1.clone(), torch.zeros(16, dtype=torch.uint8, device="cuda"))
    assert e.value.code == -3
