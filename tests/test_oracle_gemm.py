"""Pins for the oracle's three-product reconstruction (Sec. 4.3-4.5) and for the bound helpers.

Independent anchors used here: exact rational arithmetic with an explicit FP32 rounding step
written in this file (brute force on tiny inputs), inputs on which every partial sum is exact,
the FP64 reference, and the constants the paper states for its bounds.
"""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import bounds
from paper_2507_23387_b200 import inputs


# ------------------------------------------------------------------ helpers (independent of oracle)
def _f16_frac(bits16):
    b = int(bits16)
    sign = -1 if b & 0x8000 else 1
    E, M = (b >> 10) & 0x1F, b & 0x3FF
    assert E != 0x1F
    if E == 0:
        return sign * Fraction(M, 2 ** 24)
    return sign * Fraction(1024 + M, 1024) * Fraction(2) ** (E - 15)


def _rn32(q: Fraction) -> Fraction:
    """Round an exact rational to the nearest FP32 value, ties to even (normal range only)."""
    if q == 0:
        return Fraction(0)
    sign = -1 if q < 0 else 1
    a = abs(q)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    assert -126 <= e <= 127
    ulp = Fraction(2) ** (e - 23)
    n = a / ulp                                  # in [2^23, 2^24)
    fl = n.numerator // n.denominator
    rem = n - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        fl += 1
    return sign * fl * ulp


def _brute_force(A, B, s, order, kb):
    """Eq. termwise / Eq. elementwise evaluated with exact rationals and explicit FP32 rounding
    of every addition.  hi/lo words come from the (separately pinned) split."""
    M, K = A.shape
    _, N = B.shape
    Ah, Al = oracle.split(A, s)
    Bh, Bl = oracle.split(B, s)
    fr = np.vectorize(_f16_frac, otypes=[object])
    Ah, Al, Bh, Bl = fr(Ah), fr(Al), fr(Bh), fr(Bl)
    inv = Fraction(1, 2 ** s)
    C = np.empty((M, N), dtype=object)
    for i in range(M):
        for j in range(N):
            S = [Fraction(0)] * 3
            acc = Fraction(0)
            for k0 in range(0, K, kb):
                P = [Fraction(0)] * 3
                for k in range(k0, min(k0 + kb, K)):
                    P[0] = _rn32(P[0] + Ah[i, k] * Bh[k, j])
                    P[1] = _rn32(P[1] + Al[i, k] * Bh[k, j])
                    P[2] = _rn32(P[2] + Ah[i, k] * Bl[k, j])
                if order == oracle.TERMWISE:
                    S = [_rn32(S[t] + P[t]) for t in range(3)]
                elif order == oracle.ELEMENTWISE_REORDERED:
                    block = _rn32(_rn32(P[1] + P[2]) * inv + P[0])
                    acc = _rn32(acc + block)
                else:
                    acc = _rn32(acc + P[0])
                    acc = _rn32(acc + P[1] * inv)
                    acc = _rn32(acc + P[2] * inv)
            if order == oracle.TERMWISE:
                C[i, j] = _rn32(S[0] + _rn32(S[1] + S[2]) * inv)
            else:
                C[i, j] = acc
    return C


def _to_frac_matrix(C):
    return np.vectorize(lambda v: Fraction(float(v)), otypes=[object])(C)


# ------------------------------------------------------------------------------------ the pins
def test_rn32_helper_agrees_with_numpy_float32():
    rng = np.random.default_rng(0)
    for v in rng.standard_normal(200) * 10.0 ** rng.integers(-5, 5, 200):
        assert _rn32(Fraction(float(v))) == Fraction(float(np.float32(v)))
    assert _rn32(Fraction(2 ** 24 + 1)) == 2 ** 24            # tie -> even
    assert _rn32(Fraction(2 ** 24 + 3)) == 2 ** 24 + 4


@pytest.mark.parametrize("order", [oracle.TERMWISE, oracle.ELEMENTWISE, oracle.ELEMENTWISE_REORDERED])
@pytest.mark.parametrize("kb", [1, 3, 64])
def test_small_integers_give_the_exact_product(order, kb):
    # Integers of magnitude <= 8: hi = x, lo = 0, every partial sum exact.  Non-square shapes and
    # non-symmetric data catch transposed operands and index slips.
    rng = np.random.default_rng(1)
    M, N, K = 5, 7, 11
    A = rng.integers(-8, 9, size=(M, K)).astype(np.float32)
    B = rng.integers(-8, 9, size=(K, N)).astype(np.float32)
    C = oracle.sgemm_cube(A, B, s=11, order=order, kb=kb)
    want = A.astype(np.int64) @ B.astype(np.int64)
    assert np.array_equal(C.astype(np.int64), want) and np.array_equal(C, want.astype(np.float32))


@pytest.mark.parametrize("order", [oracle.TERMWISE, oracle.ELEMENTWISE, oracle.ELEMENTWISE_REORDERED])
@pytest.mark.parametrize("s", [9, 11, 12])
def test_three_terms_kept_and_low_low_dropped_exactly(order, s):
    # x = p + q 2^-13 with p in {4..7}, q in {-3..3}: hi = p, residual q 2^-13 exactly, and all
    # partial sums of the three computed products are exact in FP32.  The result must therefore be
    # EXACTLY  sum(p p' + (p q' + q p') 2^-13): the full product minus the dropped q q' 2^-26 term
    # (Eq. recover_eqn), for either accumulation order and any scale exponent.
    rng = np.random.default_rng(2)
    M, N, K = 4, 3, 6
    pA, qA = rng.integers(4, 8, (M, K)), rng.integers(-3, 4, (M, K))
    pB, qB = rng.integers(4, 8, (K, N)), rng.integers(-3, 4, (K, N))
    sgnA, sgnB = rng.choice([-1, 1], (M, K)), rng.choice([-1, 1], (K, N))
    A = (sgnA * (pA + qA * 2.0 ** -13)).astype(np.float32)
    B = (sgnB * (pB + qB * 2.0 ** -13)).astype(np.float32)
    assert np.array_equal(A.astype(np.float64), sgnA * (pA + qA * 2.0 ** -13))
    hh = (sgnA * pA) @ (sgnB * pB)
    cross = (sgnA * pA) @ (sgnB * qB) + (sgnA * qA) @ (sgnB * pB)
    want = hh + cross * 2.0 ** -13
    C = oracle.sgemm_cube(A, B, s=s, order=order, kb=4)
    assert np.array_equal(C.astype(np.float64), want)
    full = A.astype(np.float64) @ B.astype(np.float64)
    dropped = ((sgnA * qA) @ (sgnB * qB)) * 2.0 ** -26
    assert np.allclose(full - C, dropped, rtol=0, atol=1e-15) and np.any(dropped != 0)


@pytest.mark.parametrize("order", [oracle.TERMWISE, oracle.ELEMENTWISE, oracle.ELEMENTWISE_REORDERED])
@pytest.mark.parametrize("kb", [3, 7, 100])
def test_brute_force_rounding_order_on_tiny_inputs(order, kb):
    M, N, K = 3, 2, 7
    A, B = inputs.make_pair("normal", 5, M, N, K)
    want = _brute_force(A, B, 11, order, kb)
    got = _to_frac_matrix(oracle.sgemm_cube(A, B, s=11, order=order, kb=kb))
    assert np.array_equal(got, want)


def test_orders_differ_matches_brute_force():
    # Small corrections meeting a large accumulator: elementwise adds each correction to the
    # running sum (swamping), termwise sums the corrections first (Sec. 4.5).  Exact brute force
    # decides the expected bits; the termwise result must also be the more accurate one here.
    # Block 0 makes the accumulator 1.  Each of blocks 1..3 adds a high product 2^-12 and a
    # correction of 0.375 ulp(1): elementwise loses every one of them, termwise sums them to
    # 1.125 ulp first and keeps one ulp.
    s = 11
    x = 2.0 ** -12 * (1 + 3 * 2.0 ** -14)        # hi = 2^-12, residual 3 * 2^-26
    A = np.array([[1.0, x, x, x]], dtype=np.float32)
    B = np.ones((4, 1), dtype=np.float32)
    for kb in (1, 2):
        for order in (oracle.TERMWISE, oracle.ELEMENTWISE):
            got = _to_frac_matrix(oracle.sgemm_cube(A, B, s=s, order=order, kb=kb))
            assert np.array_equal(got, _brute_force(A, B, s, order, kb))
    el = oracle.sgemm_cube(A, B, s=s, order=oracle.ELEMENTWISE, kb=1)
    tw = oracle.sgemm_cube(A, B, s=s, order=oracle.TERMWISE, kb=1)
    assert float(el[0, 0]) == 1 + 3 * 2.0 ** -12
    assert float(tw[0, 0]) == 1 + 3 * 2.0 ** -12 + 2.0 ** -23


def test_reordered_elementwise_keeps_what_the_plain_order_loses_inside_a_block():
    # Sec. 4.5, last paragraph: summing the two corrections of a block before they meet the large
    # accumulator removes the swamping inside a block.  Block 0 makes the accumulator 1; block 1
    # has hi*hi = 2^-12 and two corrections of 0.375 ulp(1) each: added one by one to 1 + 2^-12
    # both are lost, added together (0.75 ulp) they round up.
    u = 2.0 ** -23
    a = 2.0 ** -12 * (1 + 3 * 2.0 ** -14)          # hi = 2^-12, residual 3 * 2^-26
    b = 1 + 3 * 2.0 ** -14                          # hi = 1,     residual 3 * 2^-14
    A = np.array([[1.0, a]], dtype=np.float32)
    B = np.array([[1.0], [b]], dtype=np.float32)
    el = float(oracle.sgemm_cube(A, B, s=11, order=oracle.ELEMENTWISE, kb=1)[0, 0])
    ro = float(oracle.sgemm_cube(A, B, s=11, order=oracle.ELEMENTWISE_REORDERED, kb=1)[0, 0])
    tw = float(oracle.sgemm_cube(A, B, s=11, order=oracle.TERMWISE, kb=1)[0, 0])
    assert el == 1 + 2.0 ** -12
    assert ro == 1 + 2.0 ** -12 + u and tw == ro
    for order in (oracle.ELEMENTWISE, oracle.ELEMENTWISE_REORDERED):
        got = _to_frac_matrix(oracle.sgemm_cube(A, B, s=11, order=order, kb=1))
        assert np.array_equal(got, _brute_force(A, B, 11, order, 1))


def test_reordered_elementwise_adds_a_block_to_the_accumulator_once():
    # Accumulator 2^10 (ulp 2^-13) after block 0; block 1 holds hi*hi = 2^-14 (1 - 2^-20), just
    # under half an ulp, and a correction of about 2^-29.  Eq. elementwise adds them one by one
    # and loses both; the termwise hi*hi stream loses the product as well; the reordered order
    # adds the block's own sum, which exceeds half an ulp, and rounds up.
    a_hi = 2.0 ** -7 * (1 + 2.0 ** -10)
    b = 2.0 ** -7 * (1 - 2.0 ** -10)
    a = a_hi + 2.0 ** -22
    A = np.array([[32.0, a]], dtype=np.float32)
    B = np.array([[32.0], [b]], dtype=np.float32)
    res = {o: float(oracle.sgemm_cube(A, B, s=11, order=o, kb=1)[0, 0])
           for o in (oracle.TERMWISE, oracle.ELEMENTWISE, oracle.ELEMENTWISE_REORDERED)}
    assert res[oracle.TERMWISE] == 1024.0 and res[oracle.ELEMENTWISE] == 1024.0
    assert res[oracle.ELEMENTWISE_REORDERED] == 1024.0 + 2.0 ** -13
    exact = 1024.0 + float(A[0, 1]) * float(B[1, 0])
    assert abs(res[oracle.ELEMENTWISE_REORDERED] - exact) < abs(res[oracle.TERMWISE] - exact)


@pytest.mark.parametrize("kind", ["uniform_pm1", "exponent_spread", "normal"])
@pytest.mark.parametrize("K", [15, 64, 300])
def test_main_bound_holds_entrywise_for_termwise(kind, K):
    # Eq. main_bound (valid under RN accumulation, which the oracle has by construction).  Blocked
    # summation only shortens the chains, so the bound for length K covers every kb.
    M, N = 24, 40
    A, B = inputs.make_pair(kind, 11, M, N, K)
    if kind == "normal":     # keep inside the window where Eq. split_error holds (|x| >= 2^-14)
        A = np.where(np.abs(A) < 2.0 ** -14, np.float32(2.0 ** -14), A).astype(np.float32)
        B = np.where(np.abs(B) < 2.0 ** -14, np.float32(2.0 ** -14), B).astype(np.float32)
    if kind == "uniform_pm1":
        A = np.where(np.abs(A) < 2.0 ** -14, np.float32(0), A).astype(np.float32)
        B = np.where(np.abs(B) < 2.0 ** -14, np.float32(0), B).astype(np.float32)
    C64, AB = oracle.dgemm_ref(A, B)
    coeff = float(bounds.main_bound_coeff(K))
    for kb in (K, 64, 16):
        C = oracle.sgemm_cube(A, B, s=11, order=oracle.TERMWISE, kb=kb)
        assert np.all(np.abs(C.astype(np.float64) - C64) <= coeff * AB * (1 + 1e-12))
        eta = oracle.componentwise_err(C, C64, AB)
        assert eta <= 2 * K * 2.0 ** -24          # the looser gate used for the CUDA path
        assert eta > 2.0 ** -30                   # ... and the error is not implausibly small


def test_dropped_low_low_term_obeys_ll_bound():
    # Eq. ll_bound: |R_A R_B / s_f^2| <= u16^2 (1 + u16)^2 |A||B| entrywise.
    s = 11
    A, B = inputs.make_pair("exponent_spread", 3, 16, 16, 50)
    Ah, Al = oracle.split(A, s)
    Bh, Bl = oracle.split(B, s)
    f = lambda b: b.view(np.float16).astype(np.float64)
    ll = np.abs((f(Al) * 2.0 ** -s) @ (f(Bl) * 2.0 ** -s))
    _, AB = oracle.dgemm_ref(A, B)
    assert np.all(ll <= float(bounds.ll_coeff()) * AB)
    assert ll.max() > 0


def test_bound_constants_stated_in_the_paper():
    # Sec. 4.3: the exact low-low coefficient lies between gamma_4 and gamma_5.
    assert bounds.gamma(4) < bounds.ll_coeff() < bounds.gamma(5)
    # Sec. 4.4: the ratio of Eq. main_bound's coefficient to the classical gamma_k falls below 2
    # at k = 15 (so it is >= 2 at k = 14) and tends to 1.
    assert bounds.main_bound_coeff(14) / bounds.gamma(14) >= 2
    assert bounds.main_bound_coeff(15) / bounds.gamma(15) < 2
    assert bounds.main_bound_coeff(10 ** 6) / bounds.gamma(10 ** 6) < 1.002
    # Eq. main_bound_first_order: gamma_k + 14 u32 is the first-order part; the exact
    # coefficient is slightly larger.
    for k in (15, 64, 4096):
        first = bounds.main_bound_first_order(k)
        exact = bounds.main_bound_coeff(k)
        assert first < exact < first * (1 + Fraction(1, 100))
    # tau = u16^2 (3 + 2 u16 + 2 u16^2); u16^2 = 4 u32
    assert bounds.U16 ** 2 == 4 * bounds.U32
    assert 3 * 4 * bounds.U32 < bounds.tau() < Fraction(1201, 100) * bounds.U32 * Fraction(101, 100)


def test_accuracy_against_fp64_and_native_fp16_contrast():
    # Sec. 6.2: native FP16 GEMM has Frobenius error ~1e-4; SGEMM-cube is comparable to an FP32 GEMM.
    A, B = inputs.make_pair("uniform_pm1", 0, 256, 256, 256)
    C64, AB = oracle.dgemm_ref(A, B)
    C, H = oracle.sgemm_cube(A, B, s=11, order=oracle.TERMWISE, kb=256, return_hgemm=True)
    e_cube = oracle.frobenius_rel_err(C, C64)
    e_h = oracle.frobenius_rel_err(H, C64)
    e_f32 = oracle.frobenius_rel_err(oracle.sgemm_f32(A, B), C64)
    assert 3e-5 < e_h < 1e-3
    assert e_cube < 1e-6 and e_cube < e_h / 100
    assert e_cube < 4 * e_f32 and e_f32 < 4 * e_cube
    # hi*hi alone equals an FP16-input GEMM done in float64 up to FP32 accumulation error
    Ah, _ = oracle.split(A, 11)
    Bh, _ = oracle.split(B, 11)
    f = lambda b: b.view(np.float16).astype(np.float64)
    assert np.allclose(H, f(Ah) @ f(Bh), rtol=0, atol=256 * 2.0 ** -24 * 256)


def test_scaling_matters_at_low_exponents():
    # Sec. 6.2: with s_b = 0 the method trails FP32 at low exponents; s_b = 12 recovers 1-2 orders.
    A = inputs.uniform_range(1, (64, 256), e=-8, stream=0)
    B = inputs.uniform_range(1, (256, 64), e=-8, stream=1)
    C64 = oracle.dgemm_ref(A, B, with_abs=False)
    err = {s: oracle.frobenius_rel_err(oracle.sgemm_cube(A, B, s=s, kb=64), C64) for s in (0, 6, 12)}
    assert err[12] < err[6] < err[0]
    assert err[0] > 10 * err[12]


def test_sgemm_f32_and_dgemm_reference_against_numpy():
    A, B = inputs.make_pair("normal", 9, 17, 13, 29)
    C64, AB = oracle.dgemm_ref(A, B)
    assert np.allclose(C64, A.astype(np.float64) @ B.astype(np.float64), rtol=1e-13, atol=1e-13)
    assert np.allclose(AB, np.abs(A).astype(np.float64) @ np.abs(B).astype(np.float64), rtol=1e-13)
    C32 = oracle.sgemm_f32(A, B)
    assert np.all(np.abs(C32 - C64) <= float(bounds.gamma(29)) * AB)


def test_leading_dimensions_are_honoured():
    rng = np.random.default_rng(4)
    bigA = rng.standard_normal((9, 40)).astype(np.float32)
    bigB = rng.standard_normal((40, 30)).astype(np.float32)
    A, B = bigA[:, :33], bigB[:33, :21]
    C1 = oracle.sgemm_cube(A, B, kb=8)
    C2 = oracle.sgemm_cube(np.ascontiguousarray(A), np.ascontiguousarray(B), kb=8)
    assert np.array_equal(C1, C2)


# ------------------------------------------------------------------ metric helpers, by hand
def test_error_metrics_on_cases_worked_by_hand():
    """componentwise_err = max |C - C64| / (|A||B|) (the measure Eq. main_bound is stated in) and
    frobenius_rel_err = ||C - C64||_F / ||C64||_F (Eq. err), on 2 x 2 cases small enough to do on
    paper.  A = [[1, -2], [0, 4]], B = [[3, 1], [1, -1]]:
        C64    = [[1, 3], [4, -4]]         |A||B| = [[5, 3], [4, 4]]   (differs from |C64|)
    and a result that is off by [[0.5, 0], [0, -1]]."""
    C64 = np.array([[1.0, 3.0], [4.0, -4.0]])
    AB = np.array([[5.0, 3.0], [4.0, 4.0]])
    A = np.array([[1, -2], [0, 4]], dtype=np.float32)
    B = np.array([[3, 1], [1, -1]], dtype=np.float32)
    C64_o, AB_o = oracle.dgemm_ref(A, B)
    assert np.array_equal(C64_o, C64) and np.array_equal(AB_o, AB)
    C = C64 + np.array([[0.5, 0.0], [0.0, -1.0]])
    # componentwise: max(0.5 / 5, 1 / 4) = 0.25; dividing by |C64| instead would give 0.5
    assert oracle.componentwise_err(C, C64, AB) == 0.25
    # Frobenius: sqrt(0.25 + 1) / sqrt(1 + 9 + 16 + 16) = sqrt(1.25 / 42); without the square
    # roots it would be 1.25 / 42
    assert oracle.frobenius_rel_err(C, C64) == pytest.approx((1.25 / 42.0) ** 0.5, rel=1e-15)
    assert oracle.frobenius_rel_err(C64, C64) == 0.0 and oracle.componentwise_err(C64, C64, AB) == 0.0
    # the largest quotient decides, not the largest difference
    C2 = C64 + np.array([[1.0, 0.9], [0.0, 0.0]])            # quotients 0.2 and 0.3
    assert oracle.componentwise_err(C2, C64, AB) == pytest.approx(0.3, rel=1e-15)


def test_componentwise_error_where_the_bound_is_zero():
    """An entry with (|A||B|)_ij = 0 has no tolerance at all: every product in it is zero, so any
    non-zero result there is an infinite error, and a zero result does not count."""
    A = np.array([[0, 0], [1, 2]], dtype=np.float32)
    B = np.array([[1, 0], [1, 0]], dtype=np.float32)          # |A||B| = [[0, 0], [3, 0]]
    C64, AB = oracle.dgemm_ref(A, B)
    assert np.array_equal(AB, np.array([[0.0, 0.0], [3.0, 0.0]]))
    good = np.array([[0.0, 0.0], [3.75, 0.0]])
    assert oracle.componentwise_err(good, C64, AB) == 0.25
    bad = good.copy()
    bad[0, 1] = 1e-30
    assert oracle.componentwise_err(bad, C64, AB) == float("inf")
    assert oracle.componentwise_err(np.zeros((1, 2)), np.zeros((1, 2)), np.zeros((1, 2))) == 0.0


def test_sgemm_f32_rounds_every_addition_to_fp32_in_k_order():
    """oracle.sgemm_f32 is the plain FP32 GEMM: products rounded to FP32, then added one after the
    other in ascending k with a rounding after each addition.  Brute force with exact rationals
    and the explicit rounding step above; K = 7 on inputs whose partial sums are not exact, so an
    implementation that accumulates in double (or in another order) gives different bits."""
    A, B = inputs.make_pair("normal", 3, 4, 5, 7)
    C = oracle.sgemm_f32(A, B)
    for i in range(A.shape[0]):
        for j in range(B.shape[1]):
            acc = Fraction(0)
            for k in range(A.shape[1]):
                prod = _rn32(Fraction(float(A[i, k])) * Fraction(float(B[k, j])))
                acc = _rn32(acc + prod)
            assert Fraction(float(C[i, j])) == acc, (i, j)
    # the two accumulation precisions really differ on this input
    C_double = (A.astype(np.float64) @ B.astype(np.float64)).astype(np.float32)
    assert not np.array_equal(C, C_double)
