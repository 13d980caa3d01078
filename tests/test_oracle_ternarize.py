"""Pins for the oracle's ternarization and packing (CPU only).

Each test checks the oracle against something the paper or the mathematics
fixes independently of the oracle's own code: hand-worked tensors for Eq. 3,
Algorithm 1's quotient for Eq. 5, full enumeration of Eq. 1, the closed forms
of Section 2.3, and exactness properties of the 2-bit storage.
"""
import math

import numpy as np
import pytest

import oracle
from paper_1605_04711_b200 import datagen as dg


# ----------------------------------------------------------- Eq. 3, by hand
def test_eq3_hand_worked_with_elements_on_the_threshold():
    # mean|W| = 2, factor 0.5 -> delta = 1 exactly; +-1 sit on the threshold and
    # must map to 0 ("0 if |W_i| <= delta"); alpha = mean(3, 3) = 3.
    W = np.array([1.0, -1.0, 3.0, -3.0], dtype=np.float32)
    st, codes = oracle.ternarize(W, 0.5)
    assert st.delta == 1.0
    assert codes.tolist() == [0, 0, 1, -1]
    assert st.alpha == 3.0
    assert (st.n_neg, st.n_zero, st.n_pos) == (1, 2, 1)
    assert st.n_boundary == 2


def test_eq3_hand_worked_paper_factor():
    # |W| = 0.1, 0.2, 0.3, 2.0, 4.0 ; mean = 1.32 ; 0.75 * mean = 0.99
    W = np.array([0.1, -0.2, 0.3, -2.0, 4.0], dtype=np.float32)
    st, codes = oracle.ternarize(W, 0.75)
    assert codes.tolist() == [0, 0, 0, -1, 1]
    assert st.delta == pytest.approx(0.99, rel=1e-7)
    assert st.alpha == pytest.approx(3.0, rel=1e-12)
    assert st.sum_abs == pytest.approx(6.6, rel=1e-7)


def test_all_zero_tensor_gives_zero_threshold_and_scale():
    st, codes = oracle.ternarize(np.zeros(37, dtype=np.float32))
    assert st.delta == 0.0 and st.alpha == 0.0
    assert not codes.any() and st.n_zero == 37


def test_negative_zero_and_subnormals():
    tiny = np.float32(1e-42)  # subnormal
    W = np.array([-0.0, tiny, -tiny, 0.0], dtype=np.float32)
    st, codes = oracle.ternarize(W, 0.7)
    # mean|W| = tiny/2, delta = 0.35*tiny < tiny -> the subnormals are kept
    assert codes.tolist() == [0, 1, -1, 0]
    assert st.alpha == pytest.approx(float(tiny), rel=1e-12)


def test_nonfinite_is_flagged():
    W = np.array([1.0, np.inf, -2.0], dtype=np.float32)
    st, _ = oracle.ternarize(W)
    assert st.nonfinite
    W[1] = np.nan
    st, _ = oracle.ternarize(W)
    assert st.nonfinite


# ------------------------------------------------ invariants on random draws
@pytest.mark.parametrize("dist", ["normal", "laplace", "uniform"])
@pytest.mark.parametrize("n", [1, 15, 1000, 65537])
def test_code_invariants(dist, n):
    W = dg.draw(3, f"inv-{dist}", n, dist)
    st, codes = oracle.ternarize(W, 0.7)
    assert set(np.unique(codes)).issubset({-1, 0, 1})
    assert st.n_neg + st.n_zero + st.n_pos == n
    kept = codes != 0
    assert np.all(np.sign(W[kept]) == codes[kept])
    a = np.abs(W.astype(np.float64))
    if kept.any():
        assert a[kept].min() > st.delta
    if (~kept).any():
        assert a[~kept].max() <= st.delta
    assert st.n_pos == int((codes == 1).sum()) and st.n_neg == int((codes == -1).sum())
    # factor < 1: the largest |W| exceeds the mean, so the kept set is never empty
    assert kept.any()


def test_sum_matches_long_double_and_fsum():
    W = dg.draw(1, "sum", 300001, "laplace")
    st, _ = oracle.ternarize(W, 0.7)
    exact = math.fsum(np.abs(W.astype(np.float64)).tolist())
    assert st.sum_abs == pytest.approx(exact, rel=2e-16)
    assert oracle.sum_abs_ld(W) == pytest.approx(exact, rel=1e-15)
    assert st.delta == pytest.approx(0.7 * exact / W.size, rel=4e-16)


# --------------------------------------- Eq. 5 vs Algorithm 1 and Eq. 1 / 4
@pytest.mark.parametrize("dist", ["normal", "uniform"])
def test_eq5_equals_algorithm1_quotient(dist):
    W = dg.draw(0, f"alg1-{dist}", 50000, dist)
    st, codes = oracle.ternarize(W, 0.75)
    assert st.alpha == pytest.approx(oracle.alpha_alg1(W, codes), rel=1e-14)


def test_alpha_minimises_the_objective_for_fixed_codes():
    W = dg.draw(5, "quad", 4096, "normal")
    st, codes = oracle.ternarize(W, 0.7)
    j0 = oracle.objective(W, codes, st.alpha)
    for eps in (1e-3, -1e-3, 1e-2, -1e-2):
        assert oracle.objective(W, codes, st.alpha * (1 + eps)) > j0
    # Eq. 4 with Eq. 5 substituted: J = sum W^2 - (sum_I |W|)^2 / |I|
    w64 = W.astype(np.float64)
    closed = math.fsum((w64 * w64).tolist()) - st.sum_abs_kept ** 2 / (st.n_pos + st.n_neg)
    assert j0 == pytest.approx(closed, rel=1e-12)


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("n", [3, 7, 10])
def test_global_optimum_of_eq1_is_a_threshold_solution(seed, n):
    """Enumerate all 3^n ternary vectors: the minimiser of Eq. 1 has the form of
    Eq. 3 for some threshold, with alpha the mean of the kept magnitudes, and the
    threshold sweep finds the same minimum."""
    W = dg.draw(seed, f"enum-{n}", n, "normal")
    codes, alpha, J = oracle.bruteforce_enum(W)
    d_s, a_s, J_s, _ = oracle.bruteforce_threshold(W)
    assert J == pytest.approx(J_s, rel=1e-12, abs=1e-15)
    assert alpha == pytest.approx(a_s, rel=1e-12)
    kept = codes != 0
    a = np.abs(W.astype(np.float64))
    assert np.all(np.sign(W[kept]) == codes[kept])
    if kept.any() and (~kept).any():
        assert a[kept].min() > a[~kept].max()
    assert alpha == pytest.approx(a[kept].mean(), rel=1e-12)
    # ternarize() with a factor that reproduces the sweep's threshold gives the same point
    factor = d_s / a.mean()
    st, c2 = oracle.ternarize(W, factor)
    assert np.array_equal(c2, codes)
    assert st.alpha == pytest.approx(alpha, rel=1e-12)


# ------------------------------------------- Section 2.3 closed-form pins
def _phi(t):
    return math.exp(-t * t / 2) / math.sqrt(2 * math.pi)


def _Q(t):
    return 0.5 * math.erfc(t / math.sqrt(2))


def test_sweep_recovers_uniform_closed_form():
    # W ~ U[-a, a]: delta* = a/3 = (2/3) E|W|
    W = dg.draw(0, "cf-uniform", 400000, "uniform")
    d, a, J, f = oracle.bruteforce_threshold(W)
    assert f == pytest.approx(2.0 / 3.0, abs=0.02)
    assert d == pytest.approx(1.0 / 3.0, abs=0.01)


def test_sweep_recovers_normal_closed_form():
    # W ~ N(0, sigma^2): the paper rounds the optimum to 0.6 sigma = 0.75 E|W|;
    # the stationarity condition phi(t) = 2 t Q(t) has its root at t = 0.6120 sigma.
    lo, hi = 0.1, 2.0
    for _ in range(100):
        mid = 0.5 * (lo + hi)
        lo, hi = (mid, hi) if _phi(mid) - 2 * mid * _Q(mid) > 0 else (lo, mid)
    assert lo == pytest.approx(0.6, abs=0.02)
    W = dg.draw(0, "cf-normal", 400000, "normal")
    d, a, J, f = oracle.bruteforce_threshold(W)
    assert d == pytest.approx(lo, abs=0.03)
    assert f == pytest.approx(0.75, abs=0.05)


@pytest.mark.parametrize("dist,excess", [("normal", 0.0076), ("uniform", 0.0038)])
def test_rule_of_thumb_lands_near_the_optimum(dist, excess):
    W = dg.draw(2, f"near-{dist}", 200000, dist)
    _, _, J_opt, _ = oracle.bruteforce_threshold(W)
    st, codes = oracle.ternarize(W, 0.7)
    J = oracle.objective(W, codes, st.alpha)
    assert J >= J_opt * (1 - 1e-12)
    assert J / J_opt - 1 == pytest.approx(excess, abs=0.004)
    st75, c75 = oracle.ternarize(W, 0.75)
    assert oracle.objective(W, c75, st75.alpha) / J_opt - 1 < 0.03


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_large_n_limits_at_factor_0p7(seed):
    n = 1000000
    tol = 6 / math.sqrt(n)
    # N(0,1): E|W| = sqrt(2/pi)
    st, _ = oracle.ternarize(dg.draw(seed, "lim-normal", n, "normal"), 0.7, want_codes=False)
    d = 0.7 * math.sqrt(2 / math.pi)
    assert st.delta == pytest.approx(d, abs=tol)
    assert (st.n_pos + st.n_neg) / n == pytest.approx(2 * _Q(d), abs=tol)
    assert st.alpha == pytest.approx(_phi(d) / _Q(d), abs=2 * tol)
    assert abs(st.n_pos - st.n_neg) / n < tol
    # U[-1,1): E|W| = 1/2 ; kept = 1 - delta ; alpha = (1 + delta)/2
    st, _ = oracle.ternarize(dg.draw(seed, "lim-uniform", n, "uniform"), 0.7, want_codes=False)
    assert st.delta == pytest.approx(0.35, abs=tol)
    assert (st.n_pos + st.n_neg) / n == pytest.approx(0.65, abs=tol)
    assert st.alpha == pytest.approx(0.675, abs=tol)
    # Laplace(0,1): |W| ~ Exp(1) ; kept = exp(-delta) ; alpha = delta + 1
    st, _ = oracle.ternarize(dg.draw(seed, "lim-laplace", n, "laplace"), 0.7, want_codes=False)
    assert st.delta == pytest.approx(0.7, abs=2 * tol)
    assert (st.n_pos + st.n_neg) / n == pytest.approx(math.exp(-0.7), abs=tol)
    assert st.alpha == pytest.approx(1.7, abs=3 * tol)


def test_golden_closed_forms_file():
    import os
    vals = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "closed_forms.txt")) as f:
        for line in f:
            line = line.split("#")[0].split()
            if len(line) == 2:
                vals[line[0]] = float(line[1])
    assert vals["templates_ternary_3x3"] == 3 ** 9 and vals["templates_binary_3x3"] == 2 ** 9
    assert vals["compression_vs_fp32"] == 32 / vals["bits_per_weight"]
    assert vals["uniform_delta_over_mean_abs"] == pytest.approx(2 / 3)
    # 0.6 sigma / E|W| with E|W| = sigma sqrt(2/pi)
    assert vals["normal_delta_over_sigma"] / math.sqrt(2 / math.pi) == pytest.approx(
        vals["normal_delta_over_mean_abs"], abs=0.01)


# ----------------------------------------------------------- 2-bit storage
def test_pack_hand_worked_word():
    # element e of a 16-group -> bit 14 - 2*(e//2) + 16*(e%2); 0 -> 00, +1 -> 01, -1 -> 11
    # e0 = +1 -> bits 15:14 = 01 ; e1 = 0 ; e2 = -1 -> bits 13:12 = 11 ; e3 = +1 -> bits 29:28 = 01
    codes = np.array([1, 0, -1, 1], dtype=np.int8)
    p = oracle.pack(codes, 16)
    assert p.shape == (1, 1) and int(p[0, 0]) == (0x4000 | 0x3000 | (0x1000 << 16))
    # e14 (even, pair 7) -> bits 1:0 ; e15 (odd, pair 7) -> bits 17:16 ; e16 = element 0 of the
    # next word -> bits 15:14
    codes = np.zeros(32, dtype=np.int8); codes[15] = -1; codes[16] = 1; codes[14] = 1
    p = oracle.pack(codes, 64)
    assert p.shape == (1, 4)
    assert [int(v) for v in p[0]] == [0x00030001, 0x00004000, 0, 0]


def test_pack_round_trip_all_3_pow_16_words():
    digits12 = np.zeros((3 ** 12, 12), dtype=np.int8)
    v = np.arange(3 ** 12)
    for i in range(12):
        digits12[:, i] = (v % 3) - 1
        v //= 3
    seen_words = 0
    for hi in range(81):
        top = np.array([(hi // 3 ** i) % 3 - 1 for i in range(4)], dtype=np.int8)
        codes = np.concatenate([digits12, np.broadcast_to(top, (3 ** 12, 4))], axis=1)
        p = oracle.pack(codes, 16)
        back = oracle.unpack(p, codes.shape[0], 16, 16)
        assert np.array_equal(back, codes)
        assert np.unique(p).size == codes.shape[0]  # injective
        seen_words += codes.shape[0]
    assert seen_words == 3 ** 16


@pytest.mark.parametrize("rows,cols", [(1, 1), (3, 17), (5, 64), (7, 100), (2, 1025)])
def test_pack_ragged_rows_and_size(rows, cols):
    codes = (np.frombuffer(np.random.default_rng(cols).bytes(rows * cols), dtype=np.uint8) % 3
             ).astype(np.int8).reshape(rows, cols) - 1
    ld = oracle.ld_for(cols)
    p = oracle.pack(codes, ld)
    assert p.nbytes == rows * ld // 4              # 2 bits per (padded) weight
    assert np.array_equal(oracle.unpack(p, rows, cols, ld), codes)
    # padding is code 0
    full = oracle.unpack(p, rows, ld, ld)
    assert not full[:, cols:].any()
    # 16x smaller than fp32 when no padding is needed
    if cols % 64 == 0:
        assert p.nbytes * 16 == rows * cols * 4


def test_unpack_rejects_the_unused_field():
    with pytest.raises(ValueError):
        oracle.unpack(np.array([[0b10 << 14]], dtype=np.uint32), 1, 1, 16)
    with pytest.raises(ValueError):
        oracle.pack(np.array([2], dtype=np.int8), 16)
