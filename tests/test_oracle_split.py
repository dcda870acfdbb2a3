"""Pins for the oracle's two-word split (Sec. 3.3, Sec. 4.1, Sec. 4.2, Eq. split_ineqs).

All checks are done in float64, where x, hi, lo * 2^-s and their differences are exact.
"""
import math
import os

import numpy as np
import pytest

import oracle

HERE = os.path.dirname(os.path.abspath(__file__))


def _f16_val(bits16):
    """FP16 bit patterns -> float64 values via numpy's own float16 (not the oracle)."""
    return np.asarray(bits16, dtype=np.uint16).view(np.float16).astype(np.float64)


def _x_with_exponent(e, mant):
    mant = np.asarray(mant, dtype=np.uint32)
    return (np.uint32((e + 127) << 23) | mant).view(np.float32)


def _split(x, s):
    x = np.asarray(x, dtype=np.float32).reshape(1, -1)
    hi, lo = oracle.split(x, s)
    return hi.ravel(), lo.ravel()


ALL_MANT = np.arange(1 << 23, dtype=np.uint32)
SOME_MANT = np.concatenate([np.arange(0, 1 << 23, 509, dtype=np.uint32),
                            np.arange(0, 1 << 14, dtype=np.uint32),
                            (1 << 23) - 1 - np.arange(0, 1 << 14, dtype=np.uint32)])


def test_worked_example_32784():
    # Sec. 4.2: V = 32784 -> V_high = 32768, residual 16; 16 * 2^12 overflows FP16.
    hi, lo = _split([32784.0], 12)
    assert hi[0] == 0x7800 and lo[0] == 0x7C00
    hi, lo = _split([32784.0], 11)            # 16 * 2^11 = 32768 is in range
    assert hi[0] == 0x7800 and lo[0] == 0x7800
    hi, lo = _split([-32784.0], 11)
    assert hi[0] == 0xF800 and lo[0] == 0xF800


@pytest.mark.parametrize("s", [0, 11, 12])
def test_lo_is_rounded_exact_scaled_residual(s):
    # lo must equal fl16 of the EXACT scaled residual (Sec. 3.3: residual and scaling are exact),
    # computed here in float64 and converted with numpy's float16.
    rng = np.random.default_rng(s)
    for e in range(-20, 16):
        x = _x_with_exponent(e, rng.integers(0, 1 << 23, size=4096, dtype=np.uint32))
        x = np.where(rng.integers(0, 2, size=x.size) == 1, -x, x).astype(np.float32)
        x = x[np.abs(x) < 65520.0]
        hi, lo = _split(x, s)
        want_hi = x.astype(np.float16)
        assert np.array_equal(hi, want_hi.view(np.uint16))
        r = x.astype(np.float64) - want_hi.astype(np.float64)
        assert np.array_equal(r.astype(np.float32).astype(np.float64), r)      # exact in FP32
        with np.errstate(over="ignore"):
            want_lo = (r * 2.0 ** s).astype(np.float16)
        assert np.array_equal(lo, want_lo.view(np.uint16))


@pytest.mark.parametrize("s", [11, 12])
def test_split_error_bound_inside_window(s):
    # Eq. split_error: |V - (V_high + V_low)| <= 2^-22 |V| while V_high is normal and the scaled
    # residual neither under- nor overflows: exponents max(-14, -3-s) <= e <= min(15, 26-s).
    e_lo, e_hi = max(-14, -3 - s), min(15, 26 - s)
    worst = 0.0
    for e in range(e_lo, e_hi + 1):
        mant = ALL_MANT if e in (e_lo, e_lo + 1, 0, e_hi) else SOME_MANT
        x = _x_with_exponent(e, mant)
        x = x[x < 65520.0]
        for sign in (1.0, -1.0):
            xs = (x * np.float32(sign)).astype(np.float32)
            hi, lo = _split(xs, s)
            err = np.abs(xs.astype(np.float64) - _f16_val(hi) - _f16_val(lo) * 2.0 ** -s)
            rel = err / np.abs(xs.astype(np.float64))
            assert rel.max() <= 2.0 ** -22
            worst = max(worst, rel.max())
    assert worst > 2.0 ** -24      # the bound is not vacuous: 22 bits, not 24


@pytest.mark.parametrize("s", [0, 11, 12])
def test_general_bound_any_exponent(s):
    # Outside the window the error is bounded by the FP16 subnormal grid of the scaled residual:
    # |x - hi - lo 2^-s| <= max(2^-22 |x|, 2^-(25+s)) whenever nothing overflows.
    for e in range(-30, min(15, 26 - s) + 1):
        x = _x_with_exponent(e, SOME_MANT)
        x = x[x < 65520.0]
        hi, lo = _split(x, s)
        err = np.abs(x.astype(np.float64) - _f16_val(hi) - _f16_val(lo) * 2.0 ** -s)
        bound = np.maximum(2.0 ** -22 * x.astype(np.float64), 2.0 ** -(25 + s))
        assert np.all(err <= bound), e


def test_rule1_thresholds_without_scaling():
    # Rule 1 (Sec. 4.2), s = 0: the leading residual class (N = 0, |r| in [2^(e-12), 2^(e-11)))
    # stays a normal FP16 number down to |x| >= 2^-2 and becomes subnormal below; it stays
    # at or above the smallest subnormal 2^-24 down to |x| >= 2^-12 and falls below it under that.
    for e, subnormal, below in [(-2, False, False), (-3, True, False),
                                (-12, True, False), (-13, True, True)]:
        mant = np.uint32(0b0000000000_0110000000000)         # low 13 bits: N = 0, truncated
        x = _x_with_exponent(e, [mant])
        hi, lo = _split(x, 0)
        r = float(x[0]) - float(_f16_val(hi)[0])
        assert 2.0 ** (e - 12) <= r < 2.0 ** (e - 11)
        assert (r < 2.0 ** -14) == subnormal
        assert (r < 2.0 ** -24) == below
        is_sub = (lo[0] & 0x7C00) == 0
        assert is_sub == subnormal


def test_split_ineqs_and_sign_flip():
    # Eq. split_ineqs: |R~_A| <= u16 (1 + u16) |A|, |A_half| <= (1 + u16) |A|;
    # Sec. 3.3: the low word's sign differs from V's exactly when the high part was rounded up.
    s = 11
    u16 = 2.0 ** -11
    rng = np.random.default_rng(7)
    for e in range(-14, 16):
        x = _x_with_exponent(e, rng.integers(0, 1 << 23, size=1 << 14, dtype=np.uint32))
        x = x[x < 65520.0]
        hi, lo = _split(x, s)
        xv, hv, lv = x.astype(np.float64), _f16_val(hi), _f16_val(lo) * 2.0 ** -s
        assert np.all(np.abs(lv) <= u16 * (1 + u16) * xv)
        assert np.all(np.abs(hv) <= (1 + u16) * xv)
        nz = lv != 0
        rounded_up = hv > xv
        assert np.array_equal((lo[nz] & 0x8000) != 0, rounded_up[nz])


def _residual_classes(e):
    """Enumerate the 13 bits below the split point and the parity of the bit above them.
    Returns arrays (X_is_R, N, r) with r the exact residual V - V_high, hi taken from the oracle."""
    low = np.arange(1 << 14, dtype=np.uint32)           # bit 13 = parity of the kept LSB
    x = _x_with_exponent(e, low)
    hi, _ = _split(x, 0)
    r = x.astype(np.float64) - _f16_val(hi)
    units = np.abs(r) / 2.0 ** (e - 23)                 # residual in FP32 ulps: 0 .. 4096
    N = np.full(r.shape, 12, dtype=np.int64)
    nzm = units > 0
    N[nzm] = 11 - np.floor(np.log2(units[nzm])).astype(np.int64)
    return r < 0, N, r


def test_residual_class_probabilities_match_paper_table():
    table = {}
    for line in open(os.path.join(HERE, "golden", "residual_class_probabilities.txt")):
        if line.strip() and not line.startswith("#"):
            X, n, lg = line.split()
            table[(X, int(n))] = 0.0 if lg == "-inf" else 2.0 ** int(lg)
    assert abs(sum(table.values()) - 1.0) < 1e-15       # "the probabilities sum to one"
    for e in (-9, 0, 7):
        is_R, N, _ = _residual_classes(e)
        for (X, n), p in table.items():
            count = np.sum((is_R == (X == "R")) & (N == n))
            assert count == p * (1 << 14), (e, X, n)


@pytest.mark.parametrize("s", [0, 12])
def test_underflow_conditions(s):
    # Sec. 4.1, second displayed equation (b_low = 15, l_Mhigh = 10), for the unscaled residual:
    #   gradual underflow  (|r| < 2^-14)  iff  E_offset - 10 + 15 - 3 < N
    #   underflow          (|r| < 2^-24)  iff  E_offset + 15 - 3 < N
    # and Sec. 4.2: multiplying by 2^12 moves both boundaries down by 12 exponents
    # (residuals enter the subnormal range once E_offset < -14, fall below 2^-24 once < -24),
    # so inside the normal range of the high word (E_offset >= -14) the leading class never does.
    for e in range(-14, 12):
        is_R, N, r = _residual_classes(e)
        rs = np.abs(r) * 2.0 ** s
        nz = r != 0
        gu = (e + s) - 10 + 15 - 3 < N
        u = (e + s) + 15 - 3 < N
        assert np.array_equal((rs < 2.0 ** -14)[nz], gu[nz])
        assert np.array_equal((rs < 2.0 ** -24)[nz], u[nz])
        lead = nz & (N == 0)
        assert np.any(gu & lead) == (e + s < -2)
        assert np.any(u & lead) == (e + s < -12)


def test_signed_zero_and_special_values():
    x = np.array([0.0, -0.0, 1.0, -1.0, np.inf, -np.inf, 70000.0], dtype=np.float32)
    hi, lo = _split(x, 11)
    assert list(hi[:4]) == [0x0000, 0x8000, 0x3C00, 0xBC00]
    assert list(lo[:4]) == [0x0000, 0x0000, 0x0000, 0x0000]   # x - hi = +0 under RN
    assert hi[4] == 0x7C00 and hi[5] == 0xFC00 and hi[6] == 0x7C00
    assert all((l & 0x7FFF) > 0x7C00 or (l & 0x7FFF) == 0x7C00 for l in lo[4:])  # inf - inf / -inf
    hi, lo = _split(np.array([np.nan], dtype=np.float32), 11)
    assert (hi[0] & 0x7FFF) > 0x7C00 and (lo[0] & 0x7FFF) > 0x7C00
    tiny = np.array([-(2.0 ** -30), -(2.0 ** -40)], dtype=np.float32)
    hi, lo = _split(tiny, 11)
    assert hi[0] == 0x8000 and lo[0] == 0x8020                # -2^-19 = -32 * 2^-24, subnormal
    assert hi[1] == 0x8000 and lo[1] == 0x8000                # -2^-29 rounds to -0 in FP16


def test_strided_input():
    rng = np.random.default_rng(3)
    big = rng.standard_normal((6, 20)).astype(np.float32)
    view = big[:, :13]
    hi, lo = oracle.split(view, 11)
    hi2, lo2 = oracle.split(np.ascontiguousarray(view), 11)
    assert np.array_equal(hi, hi2) and np.array_equal(lo, lo2)
    assert math.isclose(float(_f16_val(hi)[2, 5]), float(view[2, 5]), rel_tol=2 ** -11)
