"""Pins of the oracle's per-filter ternarization (Algorithm 1 as printed: the first loop runs
over the filters of a layer, each with its own threshold and scale).  CPU only."""
import math

import numpy as np
import pytest

import oracle
from paper_1605_04711_b200 import datagen as dg


def test_hand_worked_two_filters():
    # Filter 0: |w| sums to 10, mean 2.5, delta = 0.7 * 2.5 = 1.75 -> codes (0,-1,+1,-1),
    # alpha = (2+3+4)/3 = 3.  Filter 1: sum 11.5, mean 2.875, delta = 2.0125 -> only the
    # last weight survives, alpha = 10.  One threshold for the whole layer would give
    # delta = 0.7 * 21.5/8 = 1.88125 and alpha = (2+3+4+10)/4 = 4.75 instead.
    W = np.array([[1.0, -2.0, 3.0, -4.0], [0.5, 0.5, -0.5, 10.0]], dtype=np.float32)
    st, codes = oracle.ternarize_rows(W, 0.7)
    assert codes.tolist() == [[0, -1, 1, -1], [0, 0, 0, 1]]
    assert st[0].delta == pytest.approx(1.75, rel=1e-15) and st[0].alpha == pytest.approx(3.0, rel=1e-15)
    assert st[1].delta == pytest.approx(2.0125, rel=1e-15) and st[1].alpha == pytest.approx(10.0, rel=1e-15)
    assert (st[0].n_neg, st[0].n_zero, st[0].n_pos) == (2, 1, 1)
    assert (st[1].n_neg, st[1].n_zero, st[1].n_pos) == (0, 3, 1)
    layer, _ = oracle.ternarize(W, 0.7)
    assert layer.delta == pytest.approx(1.88125, rel=1e-15) and layer.alpha == pytest.approx(4.75, rel=1e-15)


def test_paper_factor_and_threshold_ties_per_filter():
    # delta_r = 0.75 * mean|W_r| (the constant of Sec. 2.3); an element equal to the threshold
    # is coded 0 (Eq. 3 uses "<=") and stays out of the scale
    W = np.array([[3.0, -3.0, 3.0, 7.0], [4.0, 4.0, 4.0, 4.0]], dtype=np.float32)
    st, codes = oracle.ternarize_rows(W, 0.75)
    assert st[0].delta == 3.0 and codes[0].tolist() == [0, 0, 0, 1] and st[0].alpha == 7.0
    assert st[1].delta == 3.0 and codes[1].tolist() == [1, 1, 1, 1] and st[1].alpha == 4.0
    assert st[0].n_boundary == 3 and st[1].n_boundary == 0


@pytest.mark.parametrize("rows,cols", [(7, 25), (64, 147), (16, 1152)])
def test_filters_are_independent(rows, cols):
    W = dg.he_normal(11, f"rows{rows}x{cols}", rows, cols)
    W *= np.linspace(0.1, 9.0, rows, dtype=np.float32)[:, None]      # filters of very different magnitude
    st, codes = oracle.ternarize_rows(W, 0.7)
    perm = np.random.default_rng(0).permutation(rows)
    st_p, codes_p = oracle.ternarize_rows(W[perm], 0.7)
    assert np.array_equal(codes_p, codes[perm])
    for i, r in enumerate(perm):
        assert st_p[i] == st[r]
    # every filter taken alone as a one-row layer gives the same result, and its statistics
    # are those of numpy's exactly rounded sum over that row only
    for r in range(rows):
        one, c1 = oracle.ternarize(W[r], 0.7)
        assert one == st[r] and np.array_equal(c1, codes[r])
        a = np.abs(W[r].astype(np.float64))
        assert st[r].delta == pytest.approx(0.7 * math.fsum(a) / cols, rel=1e-14)
        kept = a > st[r].delta
        assert st[r].alpha == pytest.approx(math.fsum(a[kept]) / kept.sum(), rel=1e-14)
        assert np.array_equal(codes[r], (np.sign(W[r]) * kept).astype(np.int8))


def test_per_filter_scale_is_algorithm1_quotient_and_minimises_each_filters_error():
    W = dg.he_normal(12, "rows-alg1", 32, 576)
    st, codes = oracle.ternarize_rows(W, 0.7)
    for r in range(32):
        assert st[r].alpha == pytest.approx(oracle.alpha_alg1(W[r], codes[r]), rel=1e-13)
        j0 = oracle.objective(W[r], codes[r], st[r].alpha)
        assert j0 <= oracle.objective(W[r], codes[r], st[r].alpha * (1 + 1e-6))
        assert j0 <= oracle.objective(W[r], codes[r], st[r].alpha * (1 - 1e-6))


def test_best_per_filter_thresholds_never_lose_to_the_best_layer_threshold():
    # Eq. 1 solved per filter has more freedom than Eq. 1 solved with one (delta, alpha) for
    # the layer, so the sum of the per-filter optima cannot exceed the layer optimum
    W = dg.he_normal(13, "rows-bf", 12, 200)
    W *= np.linspace(0.2, 5.0, 12, dtype=np.float32)[:, None]
    j_rows = sum(oracle.bruteforce_threshold(W[r])[2] for r in range(12))
    j_layer = oracle.bruteforce_threshold(W.reshape(-1))[2]
    assert j_rows <= j_layer * (1 + 1e-12)
    # and the rule of thumb applied per filter stays close to those optima for Gaussian filters
    st, codes = oracle.ternarize_rows(W, 0.7)
    j_rule = sum(oracle.objective(W[r], codes[r], st[r].alpha) for r in range(12))
    assert j_rows <= j_rule <= 1.05 * j_rows


def test_gemm_with_per_filter_scales_is_a_dense_product_with_the_ternary_weights():
    # Eq. 2 with a scale per filter: Y[m, n] = sum_k X[m, k] * (alpha_n * code[n, k])
    M, N, K = 9, 20, 130
    W = dg.he_normal(14, "rows-gemm", N, K)
    st, codes = oracle.ternarize_rows(W, 0.7)
    alphas = np.array([s.alpha for s in st])
    xb = dg.draw_bf16(14, "rows-gemm-x", M * K, "normal").reshape(M, K)
    Y, A = oracle.gemm(xb, codes, 1.0, scale=alphas.astype(np.float32))
    X = dg.bf16_bits_to_f64(xb)
    a32 = alphas.astype(np.float32).astype(np.float64)      # the scale vector is handed over in fp32
    assert np.allclose(Y, X @ (a32[:, None] * codes).T, rtol=1e-13, atol=1e-13)


def test_zero_filter_and_nonfinite_filter_stay_local():
    W = dg.he_normal(15, "rows-edge", 4, 64)
    W[1] = 0.0
    W[2, 5] = np.inf
    st, codes = oracle.ternarize_rows(W, 0.7)
    assert st[1].delta == 0.0 and st[1].alpha == 0.0 and not codes[1].any()
    assert st[2].nonfinite and not st[0].nonfinite and not st[3].nonfinite
    ref, c0 = oracle.ternarize(W[0], 0.7)
    assert ref == st[0] and np.array_equal(c0, codes[0])
