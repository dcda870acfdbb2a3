"""Pins for the oracle's exponent-window helpers (Sec. 4.2, Rules 1-2, Eq. sf_bounds)."""
import numpy as np

import oracle


def test_sf_bounds_statements_of_the_paper():
    # full normal FP16 range of the high words: the unique fixed choice is 11
    lo, hi = oracle.scale_exp_bounds(-14, 15)
    assert lo == 11 and hi == 11
    # s_b = 12 is admissible exactly when e_max <= 14 (Rule 2: s_b <= 26 - e_max)
    assert oracle.scale_exp_bounds(-14, 14)[1] == 12 and oracle.scale_exp_bounds(-14, 15)[1] < 12
    # Rule 1: below 2^-2 (e <= -3) the residual needs scaling, i.e. the lower bound becomes positive
    assert oracle.scale_exp_bounds(-2, 0)[0] <= 0 < oracle.scale_exp_bounds(-4, 0)[0]


def test_upper_bound_is_exactly_where_the_scaled_residual_overflows():
    # For every exponent e, the worst residual of a high word with exponent e is 2^(e-11)
    # (midpoint tie); scaled by 2^s it overflows FP16 (>= 65520 -> inf) iff s > 26 - e - ... :
    # the paper's sufficient bound e - 11 + s <= 15 must be safe, and s = 27 - e must overflow for
    # the tie input.
    for e in range(-10, 16):
        x = np.float32(2.0 ** e * (1 + 2.0 ** -11))          # midpoint between two FP16 values
        win = oracle.exponent_window([[x]])
        s_hi = oracle.scale_exp_bounds(win[0], win[1])[1]
        if 0 <= s_hi <= 24:
            _, lo = oracle.split(np.array([[x]], dtype=np.float32), s_hi)
            assert (lo[0, 0] & 0x7FFF) < 0x7C00                     # in range at the bound
        if 0 <= s_hi + 1 <= 24:
            _, lo = oracle.split(np.array([[x]], dtype=np.float32), s_hi + 1)
            assert (lo[0, 0] & 0x7FFF) == 0x7C00                    # overflows one above it
    # the paper's worked example: 32784 has e_max = 15, so 12 is out and 11 is in
    assert oracle.scale_exp_bounds(*oracle.exponent_window([[32784.0]])[:2])[1] == 11


def test_exponent_window_counts():
    X = np.array([[1.0, -3.0, 0.0, -0.0, 2.0 ** -15, 2.0 ** -30, 65504.0, 65520.0, np.inf, np.nan,
                   2.0 ** -14, 1e-3]], dtype=np.float32)
    win = oracle.exponent_window(X)
    assert win == [-14, 15, 1, 3, 3]      # 2^-15 subnormal; 65520, inf, nan non-finite; 0, -0, 2^-30 zero
    assert oracle.exponent_window(np.zeros((2, 2), dtype=np.float32)) == [127, -127, 0, 0, 4]
    # rounding carry: 2047.9 rounds up to 2048 = 2^11
    assert oracle.exponent_window([[2047.9]])[:2] == [11, 11]


# ------------------------------------------------------------------ whole-input scaling
from paper_2507_23387_b200 import inputs  # noqa: E402


def test_hi_exponent_range_agrees_with_the_fp16_window_inside_the_normal_range():
    # Where every high word is a normal FP16 number the two notions coincide; exponent_window
    # reads the exponent field of the (separately pinned) FP16 conversion.
    X = inputs.exponent_spread(7, (64, 48))                      # exponents -10 .. 10
    win = oracle.exponent_window(X)
    assert win[2:] == [0, 0, 0]
    assert oracle.hi_exponent_range(X) == [win[0], win[1], 0]


def test_hi_exponent_range_rounding_cases():
    r = oracle.hi_exponent_range
    assert r([[1.0]]) == [0, 0, 0]
    assert r([[np.float32(2 - 2.0 ** -11)]])[:2] == [1, 1]       # tie, rounds to even = 2.0
    tie = np.array([[2 - 2.0 ** -11]], dtype=np.float32)
    assert oracle.split(tie, 0)[0][0, 0] == 0x4000               # the FP16 conversion says the same
    assert r([[np.float32(2 - 2.0 ** -10)]])[:2] == [0, 0]       # representable, stays below 2
    assert r([[65519.0]])[:2] == [15, 15] and r([[65520.0]])[:2] == [16, 16]
    assert r([[2.0 ** -30, -3.0, 0.0]]) == [-30, 1, 0]
    assert r([[2.0 ** -140]])[:2] == [-140, -140]                # FP32 subnormal input
    assert r([[0.0, np.inf, np.nan]]) == [127, -127, 2]


def test_input_scale_exps_rule():
    # largest high word to the top normal binade; whole normal window -> s_b = 11 (Eq. sf_bounds)
    assert oracle.input_scale_exps([-14, 15, 0], [-14, 15, 0]) == (0, 0, 11, True)
    assert oracle.input_scale_exps([-40, -20, 0], [3, 20, 0]) == (35, -5, 11, True)
    assert oracle.input_scale_exps([-40, -10, 0], [0, 0, 0])[3] is False     # 31 binades: too wide
    assert oracle.input_scale_exps([0, 0, 1], [0, 0, 0])[3] is False         # inf / NaN present
    assert oracle.input_scale_exps([127, -127, 0], [0, 0, 0])[:2] == (0, 15)  # all-zero operand
    lo, hi = oracle.scale_exp_bounds(-14, 15)
    assert lo <= 11 <= hi


def test_scaled_product_is_the_plain_one_when_no_scaling_is_asked():
    A, B = inputs.make_pair("uniform_pm1", 3, 20, 30, 70)
    for order in (oracle.TERMWISE, oracle.ELEMENTWISE):
        assert np.array_equal(oracle.sgemm_cube_scaled(A, B, 0, 0, 11, order, 64),
                              oracle.sgemm_cube(A, B, 11, order, 64))


def test_auto_scaled_product_is_scale_covariant_bit_for_bit():
    # Multiplying an operand by a power of two shifts its p by the same amount: the split sees
    # identical words and the result is the same up to the (exact) power of two.
    A, B = inputs.make_pair("normal", 4, 24, 16, 100)
    base = None
    for a, b in ((0, 0), (-37, 9), (20, -50), (-60, -60)):
        A2, B2 = np.ldexp(A, a).astype(np.float32), np.ldexp(B, b).astype(np.float32)
        pa, pb, s, _ = oracle.input_scale_exps(oracle.hi_exponent_range(A2), oracle.hi_exponent_range(B2))
        C = oracle.sgemm_cube_scaled(A2, B2, pa, pb, s, oracle.TERMWISE, 64)
        C0 = np.ldexp(C.astype(np.float64), -(a + b))
        if base is None:
            base = C0
        assert np.array_equal(C0, base)


def test_scaling_restores_the_accuracy_of_tiny_inputs():
    # Entries around 2^-30: every high word is zero or subnormal, the plain method loses all
    # accuracy (Sec. 4.2, remark after Rule 1); with whole-input scaling the error is back at the
    # level of well-scaled inputs.
    A = inputs.uniform_range(5, (48, 200), -30, False, stream=0)
    B = inputs.uniform_range(5, (200, 40), -30, False, stream=1)
    C64 = oracle.dgemm_ref(A, B, with_abs=False)
    plain = oracle.frobenius_rel_err(oracle.sgemm_cube(A, B, 12, oracle.TERMWISE, 64), C64)
    ra, rb = oracle.hi_exponent_range(A), oracle.hi_exponent_range(B)
    pa, pb, s, _ = oracle.input_scale_exps(ra, rb)
    assert pa == 15 - ra[1] and pa >= 44
    scaled = oracle.frobenius_rel_err(oracle.sgemm_cube_scaled(A, B, pa, pb, s, oracle.TERMWISE, 64), C64)
    assert plain > 0.5 and scaled < 5e-7


def test_residual_overflow_detection_on_the_papers_example():
    # Sec. 4.2: V = 32784 rounds to 32768, residual 16; 16 * 2^12 = 65536 overflows FP16, 16 * 2^11
    # does not.  Rule 2: s_b <= 26 - e_max with e_max = 15 here.
    V = np.array([[32784.0, 1.0, -32784.0, 0.5]], dtype=np.float32)
    assert oracle.residual_overflow_count(V, 12) == 2
    assert oracle.residual_overflow_count(V, 11) == 0
    # inputs beyond the FP16 range (hi = inf) are not residual overflows
    assert oracle.residual_overflow_count(np.array([[70000.0, np.inf, np.nan]], dtype=np.float32), 12) == 0
    # the bound of Rule 2 is exactly where overflow can start: ties at exponent e overflow at 27 - e
    for e in range(3, 16):
        x = np.array([[2.0 ** e * (1 + 2.0 ** -11)]], dtype=np.float32)
        assert oracle.residual_overflow_count(x, min(26 - e, 24)) == 0
        if 27 - e <= 24:
            assert oracle.residual_overflow_count(x, 27 - e) == 1
