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
