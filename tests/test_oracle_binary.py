"""Pins for the oracle's binary-precision-weight functions (CPU only): the sign/scale rule of the
paper's BPWN baseline (Sec. 3) and the 1-bit storage of its codes.

Checked against what the mathematics fixes: a hand-worked tensor, the closed-form minimiser of the
1-D quadratic in alpha, full enumeration of all 2^n sign vectors, the relation to the ternary
optimum of Eq. 1, the large-n limit E|W| of a normal sample, and every bit position of a packed word.
"""
import math

import numpy as np
import pytest

import oracle
from paper_1605_04711_b200 import datagen as dg


def test_hand_worked_tensor_including_zeros():
    W = np.array([0.5, -0.25, 0.0, -0.0, 2.0, -1.25], dtype=np.float32)
    st, codes = oracle.binarize(W)
    # sign with the reading sign(0) = sign(-0) = +1
    assert codes.tolist() == [1, -1, 1, 1, 1, -1]
    assert st.alpha == pytest.approx((0.5 + 0.25 + 0.0 + 0.0 + 2.0 + 1.25) / 6, rel=1e-15)
    assert (st.n_pos, st.n_neg, st.n_zero) == (4, 2, 0)
    assert st.delta == 0.0 and st.sum_abs == pytest.approx(4.0, rel=1e-15) and not st.nonfinite


def test_alpha_is_the_minimiser_for_the_sign_codes_and_equals_the_quotient_form():
    W = dg.draw(3, "bin-a", 1000, "normal")
    st, codes = oracle.binarize(W)
    j0 = oracle.objective(W, codes, st.alpha)
    assert oracle.objective(W, codes, st.alpha * (1 + 1e-4)) > j0
    assert oracle.objective(W, codes, st.alpha * (1 - 1e-4)) > j0
    # Algorithm 1 writes the scale as (W . W~) / (W~ . W~); with W~ = sign(W) that is mean |W|
    assert oracle.alpha_alg1(W, codes) == pytest.approx(st.alpha, rel=1e-14)
    assert st.alpha == pytest.approx(math.fsum(abs(float(x)) for x in W) / W.size, rel=1e-15)
    # J = sum W^2 - n alpha^2 for the optimal scale
    assert j0 == pytest.approx(math.fsum(float(x) ** 2 for x in W) - W.size * st.alpha ** 2, rel=1e-12)


@pytest.mark.parametrize("n,seed,dist", [(1, 0, "normal"), (5, 1, "uniform"), (10, 2, "normal"), (12, 3, "laplace"), (12, 4, "normal")])
def test_full_enumeration_of_sign_vectors_gives_the_sign_rule(n, seed, dist):
    W = dg.draw(seed, f"bin-enum-{n}", n, dist)
    st, codes = oracle.binarize(W)
    bc, ba, bj = oracle.bruteforce_enum2(W)
    assert np.array_equal(bc, codes.reshape(-1))
    assert ba == pytest.approx(st.alpha, rel=1e-14)
    assert bj == pytest.approx(oracle.objective(W, codes, st.alpha), rel=1e-12)


def test_a_zero_weight_may_take_either_sign_at_no_cost():
    W = np.array([0.7, 0.0, -0.3], dtype=np.float32)
    st, codes = oracle.binarize(W)
    flipped = codes.copy(); flipped[1] = -1
    assert oracle.objective(W, codes, st.alpha) == pytest.approx(oracle.objective(W, flipped, st.alpha), rel=1e-15)


@pytest.mark.parametrize("dist", ["normal", "uniform", "laplace"])
def test_the_ternary_optimum_is_never_worse_than_the_binary_one(dist):
    # a ternary code with threshold 0 and no zero weights is the binary code: Eq. 1's optimum can only be lower
    W = dg.draw(5, f"bin-vs-tern-{dist}", 2000, dist)
    st, codes = oracle.binarize(W)
    jb = oracle.objective(W, codes, st.alpha)
    _, _, jt, _ = oracle.bruteforce_threshold(W)
    assert jt <= jb * (1 + 1e-12)
    # and the threshold rule at factor 0 reproduces the binary codes and scale (no weight is exactly 0 here)
    t0, tc = oracle.ternarize(W, 0.0)
    assert np.array_equal(tc, codes) and t0.alpha == pytest.approx(st.alpha, rel=1e-15)


def test_large_sample_limits_for_normal_weights():
    n = 400_000
    W = dg.draw(6, "bin-limit", n, "normal")
    st, codes = oracle.binarize(W)
    assert st.alpha == pytest.approx(math.sqrt(2.0 / math.pi), abs=4.0 / math.sqrt(n))       # E|W| of N(0,1)
    assert abs(st.n_pos - n / 2) < 4 * math.sqrt(n) / 2
    # relative error of the approximation: 1 - 2/pi for a normal sample
    W64 = W.astype(np.float64)
    assert oracle.objective(W, codes, st.alpha) / float((W64 ** 2).sum()) == pytest.approx(1 - 2 / math.pi, abs=0.01)


def test_nonfinite_weights_are_flagged():
    st, _ = oracle.binarize(np.array([1.0, float("inf"), -2.0], dtype=np.float32))
    assert st.nonfinite
    st, _ = oracle.binarize(np.array([1.0, float("nan")], dtype=np.float32))
    assert st.nonfinite


def test_one_bit_words_by_hand_and_size():
    # element 0 -> bit 15, element 1 -> bit 31, element 2 -> bit 14, element 31 -> bit 16
    for e, bit in [(0, 15), (1, 31), (2, 14), (3, 30), (30, 0), (31, 16)]:
        codes = np.ones((1, 32), dtype=np.int8); codes[0, e] = -1
        assert oracle.pack1(codes, 32)[0, 0] == np.uint32(1 << bit), (e, bit)
    assert oracle.pack1(np.ones((1, 32), dtype=np.int8), 32)[0, 0] == 0
    assert oracle.pack1(-np.ones((1, 32), dtype=np.int8), 32)[0, 0] == 0xFFFFFFFF
    # one bit per weight: 32x smaller than fp32
    assert oracle.pack1(np.ones((3, 256), dtype=np.int8), 256).nbytes * 32 == 3 * 256 * 4
    # ragged rows are padded with zero bits and unpack to the original
    u = dg.draw(7, "bin-rag", 5 * 77, "uniform")
    codes = np.where(u < 0, -1, 1).astype(np.int8).reshape(5, 77)
    p = oracle.pack1(codes, 128)
    assert p.shape == (5, 4) and np.array_equal(oracle.unpack1(p, 5, 77, 128), codes)
    assert (p[:, 3] == 0).all()                                  # columns 96..127: padding only
    with pytest.raises(ValueError):
        oracle.pack1(np.zeros((1, 32), dtype=np.int8), 32)       # 0 is not a binary code


def test_round_trip_over_every_16_bit_pattern_in_both_halves_of_a_word():
    pats = np.arange(1 << 16, dtype=np.uint32)
    bits = ((pats[:, None] >> np.arange(16, dtype=np.uint32)[None, :]) & 1).astype(np.int8)      # [65536, 16]
    for first in (0, 16):
        codes = np.ones((1 << 16, 32), dtype=np.int8)
        codes[:, first:first + 16] = 1 - 2 * bits
        p = oracle.pack1(codes, 32)
        assert np.array_equal(oracle.unpack1(p, 1 << 16, 32, 32), codes)
        assert len(np.unique(p[:, 0])) == 1 << 16                 # the packing is injective


def test_gemm_on_binary_codes_equals_numpy_matmul():
    M, N, K = 9, 6, 70
    W = dg.draw(8, "bin-gemm-w", N * K, "normal").reshape(N, K)
    st, codes = oracle.binarize(W)
    X = dg.draw_bf16(8, "bin-gemm-x", M * K, "normal").reshape(M, K)
    Y, A = oracle.gemm(X, codes, st.alpha)
    xd = dg.bf16_bits_to_f64(X)
    np.testing.assert_allclose(Y, st.alpha * (xd @ np.sign(W.astype(np.float64)).T), rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(A, np.abs(xd).sum(1, keepdims=True).repeat(N, 1), rtol=1e-13)
