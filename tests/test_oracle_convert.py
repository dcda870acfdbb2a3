"""Pins for the oracle's FP32 <-> FP16 conversion (Sec. 3.3 and Sec. 4.1 of the paper).

The oracle's converter is written at bit level; it is pinned against things that are not itself:
numpy's float16 conversion, the host CPU's F16C instruction on all 2^32 patterns, the ties-to-even
rule on every FP16 midpoint, and the paper's worked example.
"""
import ctypes
import os
import subprocess

import numpy as np
import pytest

import oracle

HERE = os.path.dirname(os.path.abspath(__file__))


def _bits(x):
    return np.asarray(x, dtype=np.float32).view(np.uint32)


def _same_f16(a, b):
    a = np.asarray(a, dtype=np.uint16)
    b = np.asarray(b, dtype=np.uint16)
    nan_a = (a & 0x7FFF) > 0x7C00
    nan_b = (b & 0x7FFF) > 0x7C00
    return np.array_equal(nan_a, nan_b) and np.array_equal(a[~nan_a], b[~nan_b])


def test_f16_to_f32_all_patterns_match_numpy():
    h = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    want = h.view(np.float16).astype(np.float32)
    got = oracle.f16_to_f32(h).view(np.float32)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), want[~nan].view(np.uint32))


def test_f16_roundtrip_is_identity():
    h = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    back = oracle.f16_rn(oracle.f16_to_f32(h))
    assert _same_f16(back, h)
    finite = (h & 0x7FFF) <= 0x7C00
    assert np.array_equal(back[finite], h[finite])


def test_every_midpoint_goes_to_even_and_neighbours_to_nearest():
    # Adjacent non-negative FP16 values h, h+1 (up to max finite -> inf): their midpoint is
    # exactly representable in FP32 and must round to whichever of the two has an even pattern;
    # one FP32 ulp below/above the midpoint must round down/up.
    h = np.arange(0, 0x7C00, dtype=np.uint32).astype(np.uint16)
    lo = oracle.f16_to_f32(h).view(np.float32).astype(np.float64)
    hi = np.where(h == 0x7BFF, 65536.0,
                  oracle.f16_to_f32((h + 1).astype(np.uint16)).view(np.float32).astype(np.float64))
    mid = ((lo + hi) / 2).astype(np.float32)
    assert np.array_equal(mid.astype(np.float64), (lo + hi) / 2)
    even = np.where(h % 2 == 0, h, h + 1).astype(np.uint16)
    for sign in (0, 0x8000):
        sbits = np.uint32(sign << 16)
        assert np.array_equal(oracle.f16_rn(_bits(mid) | sbits), even | np.uint16(sign))
        assert np.array_equal(oracle.f16_rn((_bits(mid) - 1) | sbits), h | np.uint16(sign))
        assert np.array_equal(oracle.f16_rn((_bits(mid) + 1) | sbits),
                              (h + 1).astype(np.uint16) | np.uint16(sign))


def test_range_ends():
    f = lambda x: oracle.f16_rn(int(_bits(x)))
    assert f(65504.0) == 0x7BFF
    assert f(65519.996) == 0x7BFF
    assert f(65520.0) == 0x7C00          # tie between 65504 and 2^16 -> even -> overflow
    assert f(-65520.0) == 0xFC00
    assert f(np.inf) == 0x7C00 and f(-np.inf) == 0xFC00
    assert (f(np.nan) & 0x7FFF) > 0x7C00
    assert f(2.0 ** -24) == 0x0001
    assert f(2.0 ** -25) == 0x0000       # exact midpoint of 0 and 2^-24 -> even -> 0 (Sec. 4.1)
    assert f(np.float32(2.0 ** -25) * np.float32(1 + 2.0 ** -23)) == 0x0001
    assert f(-(2.0 ** -26)) == 0x8000
    assert f(0.0) == 0x0000 and f(-0.0) == 0x8000
    assert f(2.0 ** -14) == 0x0400
    assert f(np.float32(2.0 ** -14) * np.float32(1 - 2.0 ** -24)) == 0x0400  # rounds up to normal
    assert f(1e-45) == 0x0000            # FP32 subnormal


def test_random_patterns_match_numpy():
    rng = np.random.default_rng(20250731)
    w = rng.integers(0, 2 ** 32, size=1 << 22, dtype=np.uint64).astype(np.uint32)
    # concentrate half of them in the FP16 window, where the interesting cases live
    e = rng.integers(127 - 27, 127 + 17, size=w.size // 2, dtype=np.uint64).astype(np.uint32)
    w[: w.size // 2] = (w[: w.size // 2] & np.uint32(0x807FFFFF)) | (e << np.uint32(23))
    with np.errstate(over="ignore", invalid="ignore"):
        want = w.view(np.float32).astype(np.float16).view(np.uint16)
    assert _same_f16(oracle.f16_rn(w), want)


def test_worked_example_from_paper():
    # tests/golden/worked_example_residual_overflow.txt (Sec. 4.2)
    rows = [l.split() for l in open(os.path.join(HERE, "golden",
                                                 "worked_example_residual_overflow.txt"))
            if l.strip() and not l.startswith("#")]
    V, Vhigh, resid, sb, scaled, overflow = (int(t) for t in rows[0])
    hi = oracle.f16_rn(int(_bits(float(V))))
    assert np.uint32(oracle.f16_to_f32(hi)).view(np.float32) == float(Vhigh)
    assert V - Vhigh == resid and resid * 2 ** sb == scaled
    got = oracle.f16_rn(int(_bits(float(scaled))))
    assert (got == 0x7C00) == bool(overflow)


def _has_f16c():
    try:
        return " f16c" in open("/proc/cpuinfo").read()
    except OSError:
        return False


@pytest.mark.skipif(not _has_f16c(), reason="host CPU has no F16C")
def test_exhaustive_sweep_against_hardware_f16c(tmp_path):
    so = tmp_path / "libf16c_sweep.so"
    subprocess.run(["gcc", "-O2", "-fopenmp", "-mf16c", "-shared", "-fPIC",
                    os.path.join(HERE, "f16c_sweep.c"), "-o", str(so)], check=True)
    helper = ctypes.CDLL(str(so))
    helper.f16c_sweep.argtypes = [ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint64,
                                  ctypes.POINTER(ctypes.c_uint32)]
    helper.f16c_sweep.restype = ctypes.c_int64
    lib = oracle._load()
    fn = ctypes.cast(lib.oracle_f16_rn, ctypes.c_void_p)
    bad_example = ctypes.c_uint32(0)
    bad = helper.f16c_sweep(fn, 0, 1 << 32, ctypes.byref(bad_example))
    assert bad == 0, "first mismatch at FP32 pattern 0x%08x" % bad_example.value
