"""Pins for the oracle's contractions (CPU only): inner product, convolution,
backward for data, straight-through weight gradient and the pooling glue.

The oracle's loops are checked against library routines that share no code
with them (numpy matmul, torch conv2d / autograd in fp64), against special
cases with known answers, and against adjoint identities.
"""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from paper_1605_04711_b200 import datagen as dg


def _rand_codes(seed, shape):
    u = dg.draw(seed, "codes", int(np.prod(shape)), "uniform")
    return (np.where(u > 0.3, 1, 0) - np.where(u < -0.3, 1, 0)).astype(np.int8).reshape(shape)


def _x(seed, name, shape):
    return dg.draw_bf16(seed, name, int(np.prod(shape)), "normal").reshape(shape)


# ------------------------------------------------------------------- GEMM
@pytest.mark.parametrize("M,N,K", [(1, 1, 1), (5, 3, 17), (33, 20, 130)])
def test_gemm_equals_numpy_matmul(M, N, K):
    X = _x(0, "x", (M, K)); T = _rand_codes(1, (N, K))
    alpha = 0.37
    Y, A = oracle.gemm(X, T, alpha)
    xd = dg.bf16_bits_to_f64(X)
    np.testing.assert_allclose(Y, alpha * (xd @ T.T.astype(np.float64)), rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(A, np.abs(xd) @ np.abs(T.T).astype(np.float64), rtol=1e-13)


def test_gemm_special_cases():
    M, N, K = 6, 4, 31
    X = _x(2, "x", (M, K)); xd = dg.bf16_bits_to_f64(X)
    Y, _ = oracle.gemm(X, np.ones((N, K), dtype=np.int8), 1.0)
    np.testing.assert_allclose(Y, np.repeat(xd.sum(1, keepdims=True), N, 1), rtol=1e-13, atol=1e-13)
    T = np.zeros((N, K), dtype=np.int8)
    for n in range(N):
        T[n, 3 * n + 1] = -1 if n % 2 else 1
    Y, _ = oracle.gemm(X, T, 2.0)
    for n in range(N):
        np.testing.assert_array_equal(Y[:, n], 2.0 * (-1 if n % 2 else 1) * xd[:, 3 * n + 1])


def test_forward_is_linear_in_alpha_and_epilogue_order():
    M, N, K = 9, 7, 40
    X = _x(3, "x", (M, K)); T = _rand_codes(4, (N, K))
    Y1, _ = oracle.gemm(X, T, 1.0)
    Y2, _ = oracle.gemm(X, T, 0.625)
    np.testing.assert_allclose(Y2, 0.625 * Y1, rtol=1e-14)
    scale = dg.draw(5, "s", N, "normal", 1.0, 0.3); shift = dg.draw(5, "b", N, "normal")
    res = dg.draw(6, "r", M * N, "normal").astype(np.float64).reshape(M, N)
    Y3, _ = oracle.gemm(X, T, 0.625, scale, shift, res, relu=True)
    want = np.maximum(Y2 * scale.astype(np.float64) + shift.astype(np.float64) + res, 0.0)
    np.testing.assert_allclose(Y3, want, rtol=1e-14, atol=1e-14)


def test_gemm_on_packed_equals_gemm_on_codes():
    N, K = 11, 150
    T = _rand_codes(7, (N, K))
    ld = oracle.ld_for(K)
    back = oracle.unpack(oracle.pack(T, ld), N, K, ld)
    X = _x(8, "x", (4, K))
    Ya, _ = oracle.gemm(X, T, 1.3)
    Yb, _ = oracle.gemm(X, back, 1.3)
    np.testing.assert_array_equal(Ya, Yb)


# ------------------------------------------------------------------- conv
CONV_CASES = [
    # B, H, W, Cin, Cout, k, stride, pad
    (2, 6, 7, 3, 4, 3, 1, 1),
    (1, 9, 9, 5, 2, 5, 1, 0),
    (2, 11, 10, 4, 6, 3, 2, 1),
    (1, 12, 12, 2, 3, 7, 2, 3),
    (3, 5, 5, 8, 8, 1, 2, 0),
    (2, 4, 4, 6, 5, 1, 1, 0),
]


def _torch_conv(d, X, T, alpha):
    xd = torch.from_numpy(dg.bf16_bits_to_f64(X).reshape(d.B, d.H, d.W, d.Cin)).permute(0, 3, 1, 2)
    wd = torch.from_numpy(T.reshape(d.Cout, d.kh, d.kw, d.Cin).astype(np.float64)).permute(0, 3, 1, 2)
    return xd, wd


@pytest.mark.parametrize("case", CONV_CASES)
def test_conv_fwd_equals_torch_conv2d(case):
    B, H, W, Cin, Cout, k, s, p = case
    d = oracle.conv_desc(B, H, W, Cin, Cout, k, s, p)
    X = _x(0, "cx", (B, H, W, Cin)); T = _rand_codes(1, (Cout, k, k, Cin))
    Y, A = oracle.conv2d_fwd(d, X, T, 0.8)
    xd, wd = _torch_conv(d, X, T, 0.8)
    ref = 0.8 * F.conv2d(xd, wd, stride=s, padding=p).permute(0, 2, 3, 1).numpy()
    assert Y.shape == ref.shape
    np.testing.assert_allclose(Y, ref, rtol=1e-12, atol=1e-12)
    refA = F.conv2d(xd.abs(), wd.abs(), stride=s, padding=p).permute(0, 2, 3, 1).numpy()
    np.testing.assert_allclose(A, refA, rtol=1e-12, atol=1e-12)
    # the pixel-list variant returns the same rows
    pix = np.array([0, Y.shape[1] * Y.shape[2] * B - 1, (Y.shape[1] * Y.shape[2] * B) // 2])
    Yp, Ap = oracle.conv2d_fwd(d, X, T, 0.8, pixels=pix)
    np.testing.assert_array_equal(Yp, Y.reshape(-1, Cout)[pix])
    np.testing.assert_array_equal(Ap, A.reshape(-1, Cout)[pix])


@pytest.mark.parametrize("case", CONV_CASES)
def test_conv_fwd_epilogue_equals_torch_conv2d_then_the_same_epilogue(case):
    """Per-channel scale and shift, an fp64 residual of the output's shape and ReLU, applied by the
    oracle inside both convolution entry points (full tensor and pixel list), against torch's fp64
    conv2d followed by the same four steps written out with numpy.  The scale and shift differ per
    channel and the residual per element, so a wrong channel or a wrong residual index shows."""
    B, H, W, Cin, Cout, k, s, p = case
    d = oracle.conv_desc(B, H, W, Cin, Cout, k, s, p)
    X = _x(20, "cx", (B, H, W, Cin)); T = _rand_codes(21, (Cout, k, k, Cin))
    alpha = 0.55
    scale = dg.draw(22, "s", Cout, "normal", 1.0, 0.4)
    shift = dg.draw(22, "b", Cout, "normal", 0.0, 0.5)
    res = dg.draw(23, "r", B * d.Ho * d.Wo * Cout, "normal").astype(np.float64).reshape(B, d.Ho, d.Wo, Cout)
    xd, wd = _torch_conv(d, X, T, alpha)
    z = alpha * F.conv2d(xd, wd, stride=s, padding=p).permute(0, 2, 3, 1).numpy()
    pre = z * scale.astype(np.float64)[None, None, None, :] + shift.astype(np.float64)[None, None, None, :] + res
    want = np.maximum(pre, 0.0)
    assert (pre < 0).any() and (pre > 0).any()          # the ReLU must matter
    Y, _ = oracle.conv2d_fwd(d, X, T, alpha, scale, shift, res, relu=True)
    np.testing.assert_allclose(Y, want, rtol=1e-12, atol=1e-12)
    # without ReLU, and each step alone
    Y, _ = oracle.conv2d_fwd(d, X, T, alpha, scale, shift, res, relu=False)
    np.testing.assert_allclose(Y, pre, rtol=1e-12, atol=1e-12)
    Y, _ = oracle.conv2d_fwd(d, X, T, alpha, residual=res)
    np.testing.assert_allclose(Y, z + res, rtol=1e-12, atol=1e-12)
    Y, _ = oracle.conv2d_fwd(d, X, T, alpha, shift=shift)
    np.testing.assert_allclose(Y, z + shift.astype(np.float64), rtol=1e-12, atol=1e-12)
    # the pixel-list form, in an order that is not the tensor's: the residual is still indexed by
    # the flat position in the full output
    npix = B * d.Ho * d.Wo
    pix = np.array(sorted(set([0, npix - 1, npix // 2, npix // 3, 1, max(npix - 2, 0)])))[::-1].copy()
    Yp, Ap = oracle.conv2d_fwd(d, X, T, alpha, scale, shift, res, relu=True, pixels=pix)
    np.testing.assert_allclose(Yp, want.reshape(-1, Cout)[pix], rtol=1e-12, atol=1e-12)
    Yf, Af = oracle.conv2d_fwd(d, X, T, alpha, scale, shift, res, relu=True)
    np.testing.assert_array_equal(Yp, Yf.reshape(-1, Cout)[pix])
    np.testing.assert_array_equal(Ap, Af.reshape(-1, Cout)[pix])


def test_conv_1x1_is_the_gemm():
    d = oracle.conv_desc(2, 3, 5, 16, 9, 1, 1, 0)
    X = _x(2, "cx", (2, 3, 5, 16)); T = _rand_codes(3, (9, 1, 1, 16))
    Yc, Ac = oracle.conv2d_fwd(d, X, T, 1.1)
    Yg, Ag = oracle.gemm(X.reshape(30, 16), T.reshape(9, 16), 1.1)
    np.testing.assert_array_equal(Yc.reshape(30, 9), Yg)
    np.testing.assert_array_equal(Ac.reshape(30, 9), Ag)


@pytest.mark.parametrize("case", CONV_CASES)
def test_bwd_data_is_the_adjoint_and_matches_autograd(case):
    B, H, W, Cin, Cout, k, s, p = case
    d = oracle.conv_desc(B, H, W, Cin, Cout, k, s, p)
    X = _x(4, "cx", (B, H, W, Cin)); T = _rand_codes(5, (Cout, k, k, Cin))
    dZ = _x(6, "dz", (B, d.Ho, d.Wo, Cout))
    alpha = 0.45
    dX, A = oracle.conv2d_bwd_data(d, dZ, T, alpha)
    Y, _ = oracle.conv2d_fwd(d, X, T, alpha)
    lhs = float((Y * dg.bf16_bits_to_f64(dZ).reshape(Y.shape)).sum())
    rhs = float((dg.bf16_bits_to_f64(X).reshape(dX.shape) * dX).sum())
    assert lhs == pytest.approx(rhs, rel=1e-11, abs=1e-11)
    xd, wd = _torch_conv(d, X, T, alpha)
    xd = xd.clone().requires_grad_(True)
    out = alpha * F.conv2d(xd, wd, stride=s, padding=p)
    out.backward(torch.from_numpy(dg.bf16_bits_to_f64(dZ).reshape(B, d.Ho, d.Wo, Cout)).permute(0, 3, 1, 2))
    np.testing.assert_allclose(dX, xd.grad.permute(0, 2, 3, 1).numpy(), rtol=1e-12, atol=1e-12)
    # gather form == scatter form
    pix = np.arange(B * H * W)
    dXg, Ag = oracle.conv2d_bwd_data(d, dZ, T, alpha, pixels=pix)
    np.testing.assert_allclose(dXg, dX.reshape(-1, Cin), rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(Ag, A.reshape(-1, Cin), rtol=1e-13, atol=1e-13)


@pytest.mark.parametrize("case", CONV_CASES)
def test_bwd_weight_matches_autograd_and_has_no_alpha(case):
    B, H, W, Cin, Cout, k, s, p = case
    d = oracle.conv_desc(B, H, W, Cin, Cout, k, s, p)
    X = _x(7, "cx", (B, H, W, Cin)); dZ = _x(8, "dz", (B, d.Ho, d.Wo, Cout))
    dW, A = oracle.conv2d_bwd_weight(d, X, dZ)
    xd = torch.from_numpy(dg.bf16_bits_to_f64(X).reshape(B, H, W, Cin)).permute(0, 3, 1, 2)
    w = torch.zeros(Cout, Cin, k, k, dtype=torch.float64, requires_grad=True)
    F.conv2d(xd, w, stride=s, padding=p).backward(
        torch.from_numpy(dg.bf16_bits_to_f64(dZ).reshape(B, d.Ho, d.Wo, Cout)).permute(0, 3, 1, 2))
    np.testing.assert_allclose(dW, w.grad.permute(0, 2, 3, 1).numpy(), rtol=1e-12, atol=1e-12)
    idx = np.array([0, dW.size - 1, dW.size // 3])
    dWe, Ae = oracle.conv2d_bwd_weight(d, X, dZ, entries=idx)
    np.testing.assert_array_equal(dWe, dW.reshape(-1)[idx])
    np.testing.assert_array_equal(Ae, A.reshape(-1)[idx])
    assert np.all(A.reshape(-1) >= np.abs(dW.reshape(-1)) - 1e-12)


# ------------------------------------------------------------------- glue
@pytest.mark.parametrize("k,s,p,H,W", [(2, 2, 0, 8, 6), (3, 2, 1, 9, 12), (3, 2, 1, 7, 7)])
def test_maxpool_matches_torch(k, s, p, H, W):
    x = dg.draw(0, "mp", 2 * H * W * 5, "normal").astype(np.float64).reshape(2, H, W, 5)
    y, arg = oracle.maxpool(x, k, s, p)
    xt = torch.from_numpy(x).permute(0, 3, 1, 2).clone().requires_grad_(True)
    yt = F.max_pool2d(xt, k, s, p)
    np.testing.assert_array_equal(y, yt.detach().permute(0, 2, 3, 1).numpy())
    dy = dg.draw(1, "dmp", y.size, "normal").astype(np.float64).reshape(y.shape)
    yt.backward(torch.from_numpy(dy).permute(0, 3, 1, 2))
    dx = oracle.maxpool_bwd(dy, arg, H, W)
    np.testing.assert_allclose(dx, xt.grad.permute(0, 2, 3, 1).numpy(), rtol=1e-14, atol=1e-14)


def test_avgpool():
    x = dg.draw(0, "ap", 3 * 7 * 7 * 4, "normal").astype(np.float64).reshape(3, 7, 7, 4)
    y = oracle.global_avgpool(x)
    np.testing.assert_allclose(y, x.reshape(3, 49, 4).sum(1) / 49, rtol=1e-14)
    dx = oracle.global_avgpool_bwd(y, 7, 7)
    assert dx.shape == x.shape and np.allclose(dx[:, 3, 2, :], y / 49)


# ------------------------------------------------------------------- batch statistics
def test_bn_statistics_and_affine_match_torch_batch_norm_in_training_mode():
    """The two per-channel sums and the affine derived from them against torch's batch_norm in training mode
    (batch statistics, biased variance), on the output of an oracle convolution."""
    B, H, W, Cin, Cout, k, s, p = 3, 9, 8, 4, 6, 3, 1, 1
    d = oracle.conv_desc(B, H, W, Cin, Cout, k, s, p)
    X = _x(30, "bnx", (B, H, W, Cin)); T = _rand_codes(31, (Cout, k, k, Cin))
    Z, _ = oracle.conv2d_fwd(d, X, T, 0.7)
    ssum, ssq = oracle.bn_stats(Z)
    n = B * d.Ho * d.Wo
    zt = torch.from_numpy(Z).permute(0, 3, 1, 2)
    var_t, mean_t = torch.var_mean(zt, dim=(0, 2, 3), unbiased=False)
    gamma = dg.draw(32, "bng", Cout, "normal", 1.0, 0.2).astype(np.float64)
    beta = dg.draw(32, "bnb", Cout, "normal", 0.0, 0.3).astype(np.float64)
    mean, var, scale, shift = oracle.bn_affine(ssum, ssq, n, gamma, beta, eps=1e-5)
    np.testing.assert_allclose(mean, mean_t.numpy(), rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(var, var_t.numpy(), rtol=1e-10)
    want = F.batch_norm(zt, None, None, torch.from_numpy(gamma), torch.from_numpy(beta), training=True, eps=1e-5)
    got = Z * scale[None, None, None, :] + shift[None, None, None, :]
    np.testing.assert_allclose(got, want.permute(0, 2, 3, 1).numpy(), rtol=1e-9, atol=1e-10)
    # a constant channel has zero variance; sums are plain sums
    C2 = np.zeros((2, 3, 3, 2)); C2[..., 0] = 1.5; C2[..., 1] = np.arange(18).reshape(2, 3, 3)
    s2, q2 = oracle.bn_stats(C2)
    assert s2.tolist() == [27.0, 153.0] and q2.tolist() == [40.5, float(sum(i * i for i in range(18)))]
