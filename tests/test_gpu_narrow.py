"""GPU parity for layers of at most 64 output channels, which run in the kernel that keeps the
layer's decoded weights resident in shared memory and serves all taps of a filter from one
activation tile with a halo (convolution forward, backward for data, inner product).

Same bar as the other contraction tests: |y - y_ref| <= 1e-4 * alpha * |scale_n| * A + 1e-6 against
the fp64 oracle, A = sum_k |x_k t_k|; a bf16 output may differ by one more rounding.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_1605_04711_b200 import datagen as dg
from paper_1605_04711_b200 import twn
from _gpu_util import dev_bf16, dev_f32, host_bf16_bits
from test_gpu_contract import ternarized

pytestmark = pytest.mark.gpu


def check(got_t, want, tol, out_bf16):
    if out_bf16:
        got = dg.bf16_bits_to_f64(host_bf16_bits(got_t))
        tol = tol + 2.0 ** -8 * (np.abs(want) + tol)
    else:
        got = got_t.cpu().numpy().astype(np.float64)
    assert not np.isnan(got).any()
    err = np.abs(got - want)
    bad = ~(err <= tol)
    assert not bad.any(), f"{int(bad.sum())} of {bad.size} outputs out of tolerance, worst err/tol {np.nanmax(err / tol):.3g}"


# B, H, W, Cin, Cout, k, pad, residual ("add", "gate", None), relu, affine, out_bf16
FWD_CASES = [
    (2, 8, 8, 64, 64, 3, 1, None, False, False, False),
    (3, 7, 7, 64, 64, 3, 1, "add", True, True, True),
    (2, 13, 9, 64, 32, 3, 1, "add", True, True, False),
    (5, 20, 18, 32, 16, 3, 1, None, True, True, True),
    (1, 33, 20, 16, 48, 3, 1, "gate", False, True, True),
    (2, 12, 12, 32, 64, 5, 0, None, True, False, True),
    (2, 11, 17, 128, 64, 3, 1, "add", True, True, True),       # two channel blocks per tap
    (2, 10, 10, 96, 40, 3, 1, None, False, True, False),       # ragged channel block, ragged Cout
    (3, 9, 9, 64, 64, 7, 3, None, True, True, True),           # 49 taps: does not fit, general kernel
    (2, 16, 16, 64, 64, 1, 0, "add", True, True, True),        # no halo: free tile shape
    (5, 6, 6, 8, 24, 1, 0, None, False, False, True),
    (9, 56, 56, 64, 64, 3, 1, "add", True, True, True),        # 252 tiles: several per block, all four accumulators
    (7, 30, 28, 64, 64, 3, 1, "gate", False, True, True),
    (4, 57, 50, 48, 64, 3, 1, None, True, True, False),
]


@pytest.mark.parametrize("case", FWD_CASES)
def test_narrow_conv_fwd_matches_oracle(case):
    B, H, W, Cin, Cout, k, p, res_kind, relu, affine, out_bf16 = case
    alpha, codes, packed, ld, stats = ternarized(21, f"n{case}", Cout, k * k * Cin)
    d = twn.conv_desc(B, H, W, Cin, Cout, k, 1, p)
    od = oracle.conv_desc(B, H, W, Cin, Cout, k, 1, p)
    X = dg.draw_bf16(21, f"nx{case}", B * H * W * Cin, "normal").reshape(B, H, W, Cin)
    scale = dg.draw(21, "ns", Cout, "normal", 1.0, 0.3) if affine else None
    shift = dg.draw(21, "nb", Cout, "normal", 0.0, 0.3) if affine else None
    oshape = (B, d.Ho, d.Wo, Cout)
    rbits = dg.draw_bf16(22, f"nr{case}", int(np.prod(oshape)), "normal").reshape(oshape) if res_kind else None
    r64 = dg.bf16_bits_to_f64(rbits) if res_kind else None
    sd = dev_f32(scale) if affine else None
    bd = dev_f32(shift) if affine else None
    rd = dev_bf16(rbits) if res_kind else None
    epi = twn.epilogue(sd, bd, rd, relu=relu,
                       out_dtype=twn.BF16 if out_bf16 else twn.F32,
                       residual_op=twn.RESIDUAL_GATE if res_kind == "gate" else twn.RESIDUAL_ADD)
    Y = torch.full(oshape, float("nan"), dtype=torch.bfloat16 if out_bf16 else torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    twn.conv2d_fwd(d, dev_bf16(X), packed, ld, stats, epi, Y, status)
    codes4 = codes.reshape(Cout, k, k, Cin)
    if res_kind == "gate":
        Z, A = oracle.conv2d_fwd(od, X, codes4, alpha, scale, shift, None, relu=relu)
        want = np.where(r64 > 0, Z, 0.0)
    else:
        want, A = oracle.conv2d_fwd(od, X, codes4, alpha, scale, shift, r64, relu=relu)
    tol = 1e-4 * alpha * A * (np.abs(scale.astype(np.float64)) if affine else 1.0) + 1e-6
    assert twn.read_status(status) == 0
    check(Y, want, tol, out_bf16)


# B, H, W, Cin (<= 64: the outputs of the backward pass), Cout, k, stride, pad, residual kind, out_bf16
BWD_CASES = [
    (2, 8, 8, 64, 64, 3, 1, 1, None, False),
    (3, 14, 14, 64, 128, 3, 2, 1, "add", True),     # the four residue classes of a stride-2 layer
    (2, 16, 16, 64, 128, 1, 2, 0, "add", True),     # 1x1 stride 2: three classes have no tap at all
    (2, 15, 13, 32, 64, 3, 2, 1, "gate", True),
    (5, 28, 28, 64, 64, 3, 1, 1, "gate", True),
    (2, 9, 9, 16, 96, 3, 1, 1, None, False),
    (9, 56, 56, 64, 64, 3, 1, 1, "add", True),
    # two 64-channel blocks per tap and room for only two activation stages: both MMA-issuing threads
    # walk the same small ring, several times per block
    (6, 40, 40, 64, 96, 3, 1, 1, "add", True),
    (16, 44, 40, 64, 128, 3, 1, 1, None, True),
]


@pytest.mark.parametrize("case", BWD_CASES)
def test_narrow_conv_bwd_data_matches_oracle(case):
    B, H, W, Cin, Cout, k, s, p, res_kind, out_bf16 = case
    alpha, codes, packed, ld, stats = ternarized(23, f"nb{case}", Cout, k * k * Cin)
    d = twn.conv_desc(B, H, W, Cin, Cout, k, s, p)
    ld_b = twn.ld_for(k * k * Cout)
    packed_b = torch.empty((Cin, ld_b // 16), dtype=torch.int32, device="cuda")
    twn.transpose_codes(packed, ld, d, packed_b, ld_b)
    dZ = dg.draw_bf16(23, f"nz{case}", B * d.Ho * d.Wo * Cout, "normal").reshape(B, d.Ho, d.Wo, Cout)
    scale = dg.draw(23, "nbs", Cin, "normal", 1.0, 0.3)
    rbits = dg.draw_bf16(24, f"nbr{case}", B * H * W * Cin, "normal").reshape(B, H, W, Cin) if res_kind else None
    r64 = dg.bf16_bits_to_f64(rbits) if res_kind else None
    gate = res_kind == "gate"
    sd, rd = dev_f32(scale) if gate else None, dev_bf16(rbits) if res_kind else None
    epi = twn.epilogue(sd, None, rd,
                       out_dtype=twn.BF16 if out_bf16 else twn.F32,
                       residual_op=twn.RESIDUAL_GATE if gate else twn.RESIDUAL_ADD)
    dX = torch.full((B, H, W, Cin), float("nan"), dtype=torch.bfloat16 if out_bf16 else torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    twn.conv2d_bwd_data(d, dev_bf16(dZ), packed_b, ld_b, stats, epi, dX, status)
    dXr, A = oracle.conv2d_bwd_data(oracle.conv_desc(B, H, W, Cin, Cout, k, s, p), dZ,
                                    codes.reshape(Cout, k, k, Cin), alpha)
    tol = 1e-4 * alpha * A + 1e-6
    if gate:
        want = np.where(r64 > 0, dXr * scale.astype(np.float64), 0.0)
        tol = 1e-4 * alpha * A * np.abs(scale.astype(np.float64)) + 1e-6
    elif res_kind == "add":
        want = dXr + r64
    else:
        want = dXr
    assert twn.read_status(status) == 0
    check(dX, want, tol, out_bf16)


@pytest.mark.parametrize("M,N,K,out_bf16", [(515, 64, 576, False), (1000, 32, 200, True), (70000, 64, 320, True),
                                            (129, 16, 64, False), (4096, 48, 1024, True)])
def test_narrow_gemm_matches_oracle(M, N, K, out_bf16):
    alpha, codes, packed, ld, stats = ternarized(25, f"ng{N}x{K}", N, K)
    X = dg.draw_bf16(25, f"ngx{M}x{K}", M * K, "normal").reshape(M, K)
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16 if out_bf16 else torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    twn.gemm(dev_bf16(X), K, packed, ld, stats, M, N, K, twn.epilogue(out_dtype=twn.BF16 if out_bf16 else twn.F32),
             Y, N, status)
    rows = np.unique(np.concatenate([np.random.default_rng(M).integers(0, M, 256), [0, 127, 128, M - 129, M - 128, M - 1]]))
    rows = rows[(rows >= 0) & (rows < M)]
    Yr, A = oracle.gemm(np.ascontiguousarray(X[rows]), codes, alpha)
    assert twn.read_status(status) == 0
    sub = Y[torch.from_numpy(rows).cuda()]
    check(sub, Yr, 1e-4 * alpha * A + 1e-6, out_bf16)
    assert not torch.isnan(Y.float()).any()
