"""Pins for the oracle's four-term variant: Eq. recover_eqn with the low-low product (the term
Eq. ll_bound bounds) kept.

Anchors independent of the function under test: inputs on which the result is an exact closed
form, the already pinned three-term function on inputs whose low-low product vanishes, exact
rational brute force with an explicit FP32 rounding step, and the FP64 reference.
"""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2507_23387_b200 import inputs
from test_oracle_gemm import _f16_frac, _rn32, _to_frac_matrix


def test_low_low_term_present_with_scale_2_pow_minus_2s():
    # x = p + q 2^-13 (hi = p, residual q 2^-13 exact).  K = 2 with the second column of B negated
    # and equal p-parts, so the hi*hi stream cancels to zero exactly and what is left,
    #   cross 2^-13 + (q q' - q q'') 2^-26,
    # fits FP32 exactly: the result shows the low-low term, its sign and its 2^-2s scale.
    for s in (9, 11, 12):
        A = np.array([[3 + 3 * 2.0 ** -13, 3 - 2 * 2.0 ** -13]], dtype=np.float32)
        B = np.array([[2 + 1 * 2.0 ** -13], [-(2 - 3 * 2.0 ** -13)]], dtype=np.float32)
        hh = 3 * 2 - 3 * 2
        cross = (3 * 1 + 3 * 2) - (3 * -3 + -2 * 2)
        ll = 3 * 1 - (-2 * -3)
        want = hh + cross * 2.0 ** -13 + ll * 2.0 ** -26
        C4 = oracle.sgemm_cube_four_term(A, B, s=s, kb=64)
        assert float(C4[0, 0]) == want
        assert float(C4[0, 0]) == float(A[0].astype(np.float64) @ B[:, 0].astype(np.float64))
        C3 = oracle.sgemm_cube(A, B, s=s, order=oracle.TERMWISE, kb=64)
        assert float(C3[0, 0]) == cross * 2.0 ** -13 and ll != 0


@pytest.mark.parametrize("kb", [1, 5, 64])
def test_equals_three_term_when_one_operand_has_no_residual(kb):
    # B integer-valued: lo_B = 0, so lo_A lo_B = 0 and the four-term sum is the three-term sum.
    rng = np.random.default_rng(3)
    A = inputs.uniform_pm1(5, (9, 23))
    B = rng.integers(-8, 9, size=(23, 6)).astype(np.float32)
    assert np.array_equal(oracle.sgemm_cube_four_term(A, B, s=11, kb=kb),
                          oracle.sgemm_cube(A, B, s=11, order=oracle.TERMWISE, kb=kb))
    # and with the roles exchanged (catches a transposed low-low operand)
    A2 = rng.integers(-8, 9, size=(9, 23)).astype(np.float32)
    B2 = inputs.uniform_pm1(6, (23, 6))
    assert np.array_equal(oracle.sgemm_cube_four_term(A2, B2, s=11, kb=kb),
                          oracle.sgemm_cube(A2, B2, s=11, order=oracle.TERMWISE, kb=kb))


@pytest.mark.parametrize("kb", [3, 100])
def test_brute_force_rounding_order_on_tiny_inputs(kb):
    s = 11
    A = inputs.uniform_pm1(11, (3, 10))
    B = inputs.uniform_pm1(12, (10, 2))
    Ah, Al = oracle.split(A, s)
    Bh, Bl = oracle.split(B, s)
    fr = np.vectorize(_f16_frac, otypes=[object])
    Ah, Al, Bh, Bl = fr(Ah), fr(Al), fr(Bh), fr(Bl)
    inv = Fraction(1, 2 ** s)
    want = np.empty((3, 2), dtype=object)
    for i in range(3):
        for j in range(2):
            S = [Fraction(0)] * 4
            for k0 in range(0, 10, kb):
                P = [Fraction(0)] * 4
                for k in range(k0, min(k0 + kb, 10)):
                    P[0] = _rn32(P[0] + Ah[i, k] * Bh[k, j])
                    P[1] = _rn32(P[1] + Al[i, k] * Bh[k, j])
                    P[2] = _rn32(P[2] + Ah[i, k] * Bl[k, j])
                    P[3] = _rn32(P[3] + Al[i, k] * Bl[k, j])
                S = [_rn32(S[t] + P[t]) for t in range(4)]
            small = _rn32(_rn32(S[1] + S[2]) * inv + S[3] * inv * inv)
            want[i, j] = _rn32(S[0] + small)
    got = _to_frac_matrix(oracle.sgemm_cube_four_term(A, B, s=s, kb=kb))
    assert np.all(got == want)


def test_single_products_are_nearly_correctly_rounded():
    # K = 1 and inputs with at most 22 significant bits: the split is exact, the four partial
    # products are exact, so the four-term result is the exact product rounded twice (the small
    # terms, then the total): within 2^-24 (1 + 2^-10) of it.  The three-term result misses the
    # low-low product, which reaches 2^-22 relative.
    rng = np.random.default_rng(4)
    x = (rng.integers(2 ** 21, 2 ** 22, 4000) * 2.0 ** -21).astype(np.float32)
    y = (rng.integers(2 ** 21, 2 ** 22, 4000) * 2.0 ** -21).astype(np.float32)
    A, B = x.reshape(-1, 1), y[:64].reshape(1, -1)
    exact = A.astype(np.float64) @ B.astype(np.float64)
    e4 = np.abs(oracle.sgemm_cube_four_term(A, B, s=11, kb=64) - exact) / exact
    e3 = np.abs(oracle.sgemm_cube(A, B, s=11, order=oracle.TERMWISE, kb=64) - exact) / exact
    assert e4.max() <= 2.0 ** -24 * (1 + 2.0 ** -10)
    assert e3.max() > 2.0 ** -23


@pytest.mark.parametrize("kind", ["uniform_pm1", "normal"])
def test_short_sums_gain_a_little_from_the_fourth_term(kind):
    # The dropped term has leading coefficient 2^-22 = 4 u_32 (Eq. ll_bound), the size of a
    # length-four FP32 accumulation error; at K = 8 keeping it lowers the Frobenius error by a
    # visible margin (10-15 % on these inputs), and the componentwise error stays within the
    # representation error (2 u_16^2 leading) plus 8 RN additions.
    A, B = inputs.make_pair(kind, 21, 96, 80, 8)
    C64, ABabs = oracle.dgemm_ref(A, B)
    C3 = oracle.sgemm_cube(A, B, s=11, kb=64)
    C4 = oracle.sgemm_cube_four_term(A, B, s=11, kb=64)
    assert oracle.frobenius_rel_err(C4, C64) < 0.95 * oracle.frobenius_rel_err(C3, C64)
    assert oracle.componentwise_err(C4, C64, ABabs) <= (8 + 3) * 2.0 ** -24


def test_difference_to_three_term_is_the_low_low_product():
    A, B = inputs.make_pair("uniform_pm1", 22, 40, 30, 50)
    s = 11
    Ah, Al = oracle.split(A, s)
    Bh, Bl = oracle.split(B, s)
    ll = (Al.view(np.float16).astype(np.float64) @ Bl.view(np.float16).astype(np.float64)) \
        * 2.0 ** (-2 * s)
    _, ABabs = oracle.dgemm_ref(A, B)
    d = oracle.sgemm_cube_four_term(A, B, s=s, kb=64).astype(np.float64) \
        - oracle.sgemm_cube(A, B, s=s, order=oracle.TERMWISE, kb=64).astype(np.float64)
    # equal up to the final roundings of the two results (each <= 2^-24 |C| <= 2^-24 |A||B|)
    assert np.all(np.abs(d - ll) <= 2.5 * 2.0 ** -24 * ABabs)
    assert np.all(np.abs(ll) <= 2.0 ** -22 * (1 + 2.0 ** -11) ** 2 * ABabs)     # Eq. ll_bound


def test_invalid_arguments():
    A = np.zeros((2, 3), np.float32)
    with pytest.raises(ValueError):
        oracle.sgemm_cube_four_term(A, np.zeros((4, 2), np.float32))


def test_coherent_residuals_show_the_dropped_term_in_full():
    # Constructed inputs: every entry 1.xx + (just under) half a unit in the 11th place, so every
    # residual is about +2^-11 relative and the dropped products add up coherently:
    # sum lo lo 2^-22 ~ 2^-22 / 1.05^2 of |A||B| = about 3.6 u_32, which the four-term sum recovers.
    A = inputs.coherent_residuals(1, (32, 64), 0)
    B = inputs.coherent_residuals(1, (64, 24), 1)
    _, lo = oracle.split(A, 11)
    assert np.all(lo.view(np.float16) > 0.99)
    C64, ABabs = oracle.dgemm_ref(A, B)
    e3 = (oracle.sgemm_cube(A, B, 11, oracle.TERMWISE, 64).astype(np.float64) - C64) / ABabs
    e4 = (oracle.sgemm_cube_four_term(A, B, 11, 64).astype(np.float64) - C64) / ABabs
    assert e3.mean() * 2.0 ** 24 < -3.0 and abs(e4.mean()) * 2.0 ** 24 < 0.5   # a bias, removed
    shift = (e4 - e3).mean() * 2.0 ** 24
    assert 3.0 < shift < 4.0
    assert np.abs(e4).max() < np.abs(e3).max()
