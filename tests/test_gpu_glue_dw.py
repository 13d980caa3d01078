"""GPU parity: straight-through weight gradient and the layer glue against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_1605_04711_b200 import datagen as dg
from paper_1605_04711_b200 import twn
from _gpu_util import dev_bf16, dev_f32, host_bf16_bits

pytestmark = pytest.mark.gpu

DW_CASES = [
    # B, H, W, Cin, Cout, k, stride, pad
    (2, 8, 8, 64, 128, 3, 1, 1),
    (3, 7, 7, 64, 64, 3, 1, 1),
    (4, 14, 14, 128, 256, 3, 2, 1),
    (2, 16, 16, 64, 128, 1, 2, 0),
    (64, 1, 1, 512, 1000, 1, 1, 0),
    (2, 12, 12, 32, 64, 5, 1, 0),
    (1, 20, 20, 320, 72, 3, 1, 1),
    (5, 9, 11, 16, 40, 3, 2, 1),
    (16, 28, 28, 128, 128, 3, 1, 1),
    # filters of one column (k = (kh, kw)): the tile carries its extra rows and serves all taps
    (3, 20, 17, 64, 64, (4, 1), 1, 0),
    (2, 9, 30, 128, 192, (3, 1), 1, 1),
    (5, 33, 8, 64, 48, (2, 1), 1, 0),
    (40, 6, 6, 64, 64, (4, 1), 1, 1),
]


@pytest.mark.parametrize("case", DW_CASES)
def test_bwd_weight_matches_oracle(case):
    B, H, W, Cin, Cout, k, s, p = case
    d = twn.conv_desc(B, H, W, Cin, Cout, k, s, p)
    X = dg.draw_bf16(0, f"dwx{case}", B * H * W * Cin, "normal").reshape(B, H, W, Cin)
    dZ = dg.draw_bf16(0, f"dwz{case}", B * d.Ho * d.Wo * Cout, "normal", 0.0, 0.1).reshape(B, d.Ho, d.Wo, Cout)
    kh, kw = (k, k) if isinstance(k, int) else k
    dW = torch.full((Cout, kh, kw, Cin), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(twn.conv2d_bwd_weight_workspace_bytes(d) + 16, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    twn.conv2d_bwd_weight(d, dev_bf16(X), dev_bf16(dZ), dW, ws, status)
    assert twn.read_status(status) == 0
    od = oracle.conv_desc(B, H, W, Cin, Cout, k, s, p)
    got = dW.cpu().numpy().astype(np.float64)
    if got.size <= 400_000:
        ref, A = oracle.conv2d_bwd_weight(od, X, dZ)
    else:
        idx = np.unique(np.concatenate([np.arange(0, got.size, 997), np.arange(2000), np.arange(got.size - 2000, got.size)]))
        ref, A = oracle.conv2d_bwd_weight(od, X, dZ, entries=idx)
        got = got.reshape(-1)[idx]
    tol = 1e-4 * A + 1e-6
    err = np.abs(got.reshape(ref.shape) - ref)
    assert not np.isnan(got).any()
    assert np.all(err <= tol), f"worst err/tol {np.max(err / tol):.3g}"


def test_bwd_weight_is_deterministic():
    d = twn.conv_desc(8, 14, 14, 64, 64, 3, 1, 1)
    X = dev_bf16(dg.draw_bf16(1, "detx", 8 * 14 * 14 * 64, "normal"))
    dZ = dev_bf16(dg.draw_bf16(1, "detz", 8 * 14 * 14 * 64, "normal"))
    ws = torch.empty(twn.conv2d_bwd_weight_workspace_bytes(d), dtype=torch.uint8, device="cuda")
    outs = []
    for _ in range(2):
        dW = torch.empty((64, 3, 3, 64), dtype=torch.float32, device="cuda")
        twn.conv2d_bwd_weight(d, X, dZ, dW, ws)
        outs.append(dW.cpu().numpy())
    assert np.array_equal(outs[0], outs[1])


@pytest.mark.parametrize("case", [(2, 28, 28, 1, 5, 1, 0), (3, 32, 32, 3, 3, 1, 1), (2, 30, 30, 3, 7, 2, 3)])
def test_im2col_then_gemm_is_the_small_channel_conv(case):
    B, H, W, Cin, k, s, p = case
    Cout = 32
    d = twn.conv_desc(B, H, W, Cin, Cout, k, s, p)
    K = k * k * Cin
    ldk = (K + 7) // 8 * 8
    Wm = dg.he_normal(2, f"i2c{case}", Cout, K)
    ref, codes = oracle.ternarize(Wm, 0.7)
    ld = twn.ld_for(K)
    stats = twn.new_stats()
    packed = torch.empty((Cout, ld // 16), dtype=torch.int32, device="cuda")
    wsb = torch.empty(twn.ternarize_workspace_bytes(), dtype=torch.uint8, device="cuda")
    twn.ternarize(dev_f32(Wm), 0.7, stats, packed, ld, None, wsb, rows=Cout, cols=K)
    X = dg.draw_bf16(2, f"i2cx{case}", B * H * W * Cin, "uniform01").reshape(B, H, W, Cin)
    M = B * d.Ho * d.Wo
    Xcol = torch.full((M, ldk), 7.0, dtype=torch.bfloat16, device="cuda")
    twn.im2col(d, dev_bf16(X), Xcol, ldk)
    Y = torch.empty((M, Cout), dtype=torch.float32, device="cuda")
    twn.gemm(Xcol, ldk, packed, ld, stats, M, Cout, K, None, Y, Cout)
    Yr, A = oracle.conv2d_fwd(oracle.conv_desc(B, H, W, Cin, Cout, k, s, p), X, codes.reshape(Cout, k, k, Cin), ref.alpha)
    err = np.abs(Y.cpu().numpy().astype(np.float64).reshape(Yr.shape) - Yr)
    assert np.all(err <= 1e-4 * ref.alpha * A + 1e-6)
    assert np.all(host_bf16_bits(Xcol)[:, K:] == 0)


FOLD_CASES = [
    # B, H, W, Cin, Cout, k, pad  (stride 2)
    (2, 30, 30, 3, 32, 7, 3),      # the ResNet stem shape in small
    (3, 17, 23, 3, 64, 7, 3),      # odd extents: ragged last window
    (2, 20, 20, 1, 16, 5, 2),      # one channel, 5x5
    (1, 9, 9, 4, 8, 8, 4),         # largest filter and channel count the fold takes
    (2, 12, 10, 2, 24, 2, 0),      # one folded row, no padding
    (4, 64, 64, 3, 64, 7, 3),      # several tiles
]


@pytest.mark.parametrize("case", FOLD_CASES)
def test_folded_layer_is_the_strided_small_channel_conv(case):
    """twn_fold_input + twn_fold_codes + twn_conv2d_fwd_folded / twn_conv2d_bwd_weight_folded against the
    oracle's plain convolution and weight gradient of the unfolded layer."""
    B, H, W, Cin, Cout, k, p = case
    d = twn.conv_desc(B, H, W, Cin, Cout, k, 2, p)
    od = oracle.conv_desc(B, H, W, Cin, Cout, k, 2, p)
    K = k * k * Cin
    Hf, Wf, ldf = twn.fold_dims(d)
    assert (Hf, Wf, ldf) == (d.Ho + (k + 1) // 2 - 1, d.Wo + 3, 64 * ((k + 1) // 2))
    Wm = dg.he_normal(3, f"fold{case}", Cout, K)
    ref, codes = oracle.ternarize(Wm, 0.7)
    ld = twn.ld_for(K)
    stats = twn.new_stats()
    packed = torch.empty((Cout, ld // 16), dtype=torch.int32, device="cuda")
    wsb = torch.empty(twn.ternarize_workspace_bytes(), dtype=torch.uint8, device="cuda")
    twn.ternarize(dev_f32(Wm), 0.7, stats, packed, ld, None, wsb, rows=Cout, cols=K)
    X = dg.draw_bf16(3, f"foldx{case}", B * H * W * Cin, "normal").reshape(B, H, W, Cin)
    Xf = torch.full((B, Hf, Wf, 16), 7.0, dtype=torch.bfloat16, device="cuda")
    twn.fold_input(d, dev_bf16(X), Xf)
    # the folded tensor, element by element (bit-exact: it only moves values)
    xf = host_bf16_bits(Xf).reshape(B, Hf, Wf, 16)
    want = np.zeros_like(xf)
    for dy in range(2):
        for dx in range(2):
            hs = 2 * np.arange(Hf) + dy - p
            ws_ = 2 * np.arange(Wf) + dx - p
            hv, wv = (hs >= 0) & (hs < H), (ws_ >= 0) & (ws_ < W)
            blk = np.zeros((B, Hf, Wf, Cin), dtype=xf.dtype)
            blk[np.ix_(np.arange(B), np.nonzero(hv)[0], np.nonzero(wv)[0])] = X[np.ix_(np.arange(B), hs[hv], ws_[wv])]
            want[..., (dy * 2 + dx) * Cin:(dy * 2 + dx + 1) * Cin] = blk
    assert np.array_equal(xf, want)
    Tf = torch.full((Cout, ldf // 16), -1, dtype=torch.int32, device="cuda")
    twn.fold_codes(d, packed, ld, Tf, ldf)
    cf = oracle.unpack(Tf.cpu().numpy().view(np.uint32), Cout, ldf, ldf).reshape(Cout, ldf // 64, 4, 16)
    c4 = codes.reshape(Cout, k, k, Cin)
    for rf in range(ldf // 64):
        for sf in range(4):
            for dy in range(2):
                for dx in range(2):
                    r, sx = 2 * rf + dy, 2 * sf + dx
                    got = cf[:, rf, sf, (dy * 2 + dx) * Cin:(dy * 2 + dx + 1) * Cin]
                    assert np.array_equal(got, c4[:, r, sx, :] if r < k and sx < k else np.zeros_like(got))
            assert not cf[:, rf, sf, 4 * Cin:].any()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Y = torch.full((B, d.Ho, d.Wo, Cout), float("nan"), dtype=torch.float32, device="cuda")
    twn.conv2d_fwd_folded(d, Xf, Tf, ldf, stats, None, Y, status)
    assert twn.read_status(status) == 0
    Yr, A = oracle.conv2d_fwd(od, X, c4, ref.alpha)
    err = np.abs(Y.cpu().numpy().astype(np.float64) - Yr)
    assert np.all(err <= 1e-4 * ref.alpha * A + 1e-6)
    # straight-through weight gradient of the same layer
    dZ = dg.draw_bf16(3, f"foldz{case}", B * d.Ho * d.Wo * Cout, "normal", 0.0, 0.1).reshape(B, d.Ho, d.Wo, Cout)
    kh, kw = (k, k) if isinstance(k, int) else k
    dW = torch.full((Cout, kh, kw, Cin), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(twn.conv2d_bwd_weight_folded_workspace_bytes(d), dtype=torch.uint8, device="cuda")
    twn.conv2d_bwd_weight_folded(d, Xf, dev_bf16(dZ), dW, ws, status)
    assert twn.read_status(status) == 0
    dref, Aw = oracle.conv2d_bwd_weight(od, X, dZ)
    errw = np.abs(dW.cpu().numpy().astype(np.float64).reshape(dref.shape) - dref)
    assert np.all(errw <= 1e-4 * Aw + 1e-6), f"worst err/tol {np.max(errw / (1e-4 * Aw + 1e-6)):.3g}"


def test_fold_rejects_layers_it_cannot_take():
    assert twn.fold_dims(twn.conv_desc(1, 8, 8, 3, 8, 3, 1, 1)) is None      # stride 1
    assert twn.fold_dims(twn.conv_desc(1, 8, 8, 8, 8, 3, 2, 1)) is None      # 4*Cin > 16
    assert twn.fold_dims(twn.conv_desc(1, 32, 32, 3, 8, 9, 2, 4)) is None    # more than 8 taps per side


@pytest.mark.parametrize("k,s,p,H,W,C", [(2, 2, 0, 24, 24, 32), (3, 2, 1, 112, 112, 8), (3, 2, 1, 7, 9, 5), (2, 2, 0, 8, 8, 512),
                                          (3, 2, 1, 7, 9, 16), (3, 2, 1, 10, 13, 64), (3, 2, 1, 1, 1, 8), (3, 1, 1, 9, 6, 16), (3, 2, 1, 112, 112, 64)])
def test_maxpool_forward_and_backward(k, s, p, H, W, C):
    B = 2
    xb = dg.draw_bf16(3, f"mp{H}{C}", B * H * W * C, "normal").reshape(B, H, W, C)
    Ho, Wo = (H + 2 * p - k) // s + 1, (W + 2 * p - k) // s + 1
    Y = torch.empty((B, Ho, Wo, C), dtype=torch.bfloat16, device="cuda")
    arg = torch.empty((B, Ho, Wo, C), dtype=torch.uint8, device="cuda")
    twn.maxpool2d_fwd(dev_bf16(xb), B, H, W, C, k, s, p, Y, arg)
    yr, argr = oracle.maxpool(dg.bf16_bits_to_f64(xb), k, s, p)
    assert np.array_equal(dg.bf16_bits_to_f64(host_bf16_bits(Y)), yr)
    dyb = dg.draw_bf16(3, f"mpd{H}{C}", B * Ho * Wo * C, "normal").reshape(B, Ho, Wo, C)
    dX = torch.empty((B, H, W, C), dtype=torch.bfloat16, device="cuda")
    twn.maxpool2d_bwd(dev_bf16(dyb), arg, B, H, W, C, k, s, p, dX)
    dxr = oracle.maxpool_bwd(dg.bf16_bits_to_f64(dyb), argr, H, W)
    got = dg.bf16_bits_to_f64(host_bf16_bits(dX))
    # up to four window gradients are added in fp32 and rounded once to bf16
    assert np.all(np.abs(got - dxr) <= 2.0 ** -8 * np.abs(dxr) + 1e-30)
    # fused with the backward through y = relu(z * scale + shift) of the layer below the pool:
    # windows whose pooled value is not positive pass nothing, the sum is scaled per channel
    scale = dg.draw(3, f"mps{H}{C}", C, "normal", 1.0, 0.3)
    dZ = torch.full((B, H, W, C), float("nan"), dtype=torch.bfloat16, device="cuda")
    sd = dev_f32(scale)
    twn.maxpool2d_bwd_act(dev_bf16(dyb), arg, Y, sd, B, H, W, C, k, s, p, dZ)
    gated = np.where(yr > 0, dg.bf16_bits_to_f64(dyb), 0.0)
    dzr = oracle.maxpool_bwd(gated, argr, H, W) * scale.astype(np.float64)
    gotz = dg.bf16_bits_to_f64(host_bf16_bits(dZ))
    assert np.all(np.abs(gotz - dzr) <= 2.0 ** -8 * np.abs(dzr) + 1e-30)


@pytest.mark.parametrize("B,H,W,C", [(4, 7, 7, 512), (3, 5, 4, 320), (2, 3, 3, 20)])
def test_avgpool_and_activation_backward(B, H, W, C):
    xb = dg.draw_bf16(4, "ap", B * H * W * C, "normal").reshape(B, H, W, C)
    Y = torch.empty((B, C), dtype=torch.bfloat16, device="cuda")
    twn.avgpool_fwd(dev_bf16(xb), B, H * W, C, Y)
    yr = oracle.global_avgpool(dg.bf16_bits_to_f64(xb))
    got = dg.bf16_bits_to_f64(host_bf16_bits(Y))
    assert np.all(np.abs(got - yr) <= 2.0 ** -8 * np.abs(yr) + 1e-6)
    dyb = dg.draw_bf16(4, "apd", B * C, "normal").reshape(B, C)
    dX = torch.empty((B, H, W, C), dtype=torch.bfloat16, device="cuda")
    twn.avgpool_bwd(dev_bf16(dyb), B, H * W, C, dX)
    dxr = oracle.global_avgpool_bwd(dg.bf16_bits_to_f64(dyb), H, W)
    assert np.all(np.abs(dg.bf16_bits_to_f64(host_bf16_bits(dX)) - dxr) <= 2.0 ** -8 * np.abs(dxr) + 1e-30)
    # dPre = dY [Y > 0], dZ = dPre * scale
    yb = dg.draw_bf16(5, "act-y", B * H * W * C, "normal").reshape(-1)
    yb = np.where(dg.bf16_bits_to_f64(yb) > 0, yb, np.uint16(0)).astype(np.uint16)
    gb = dg.draw_bf16(5, "act-g", B * H * W * C, "normal").reshape(-1)
    scale = dg.draw(5, "act-s", C, "normal", 1.0, 0.3)
    dZ = torch.empty(yb.size, dtype=torch.bfloat16, device="cuda")
    dPre = torch.empty(yb.size, dtype=torch.bfloat16, device="cuda")
    sd = dev_f32(scale)
    twn.act_bwd(dev_bf16(gb), dev_bf16(yb), sd, yb.size, C, dZ, dPre)
    g = dg.bf16_bits_to_f64(gb) * (dg.bf16_bits_to_f64(yb) > 0)
    assert np.array_equal(dg.bf16_bits_to_f64(host_bf16_bits(dPre)), g)
    want = (g.astype(np.float32) * np.tile(scale, yb.size // C)).astype(np.float32)
    # compare values (a masked negative gradient is -0 in numpy, +0 from the kernel)
    assert np.array_equal(dg.bf16_bits_to_f64(host_bf16_bits(dZ)), dg.bf16_bits_to_f64(dg.f32_to_bf16_bits(want)))
