"""SGEMM-cube CPU oracle: numpy front end of oracle/sgemm_cube_oracle.cpp.

TEST INFRASTRUCTURE.  Nothing on the product path may import this package; it exists so that
tests, the smoke check and the benchmark's CPU-baseline leg can compare the CUDA library with a
slow, plain definition of the method.  It imports nothing from the CUDA package.

Functions mirror the paper's steps:
  f16_rn / f16_to_f32     FP32 <-> FP16 conversion, RN-even             [Sec. 3.3, 4.1]
  split                   (hi, lo) two-word split with residual scale s  [Eq. recover_eqn]
  sgemm_cube              three-product reconstruction, termwise or
                          elementwise accumulation, k-block kb           [Eq. termwise, elementwise]
  dgemm_ref, sgemm_f32    FP64 reference with |A||B|; plain FP32 GEMM    [Sec. 6.1]
  frobenius_rel_err       the paper's error metric                       [Eq. err]
  componentwise_err       max |C - C64| / (|A||B|)                       [Eq. main_bound]
"""
import ctypes
import os

import numpy as np

from . import build as _build
from .bounds import (U16, U32, gamma, tau, ll_coeff, main_bound_coeff,  # noqa: F401
                     main_bound_first_order)

TERMWISE = 0
ELEMENTWISE = 1
ELEMENTWISE_REORDERED = 2      # Sec. 4.5, last paragraph: corrections of a k-block summed first

_lib = None


def _load():
    global _lib
    if _lib is None:
        path = _build.build()
        lib = ctypes.CDLL(path)
        i64, c_int = ctypes.c_int64, ctypes.c_int
        vp = ctypes.c_void_p
        lib.oracle_num_threads.restype = c_int
        lib.oracle_f16_rn.argtypes = [ctypes.c_uint32]
        lib.oracle_f16_rn.restype = ctypes.c_uint16
        lib.oracle_f16_to_f32.argtypes = [ctypes.c_uint16]
        lib.oracle_f16_to_f32.restype = ctypes.c_uint32
        lib.oracle_f16_rn_array.argtypes = [i64, vp, vp]
        lib.oracle_f16_rn_array.restype = None
        lib.oracle_f16_to_f32_array.argtypes = [i64, vp, vp]
        lib.oracle_f16_to_f32_array.restype = None
        lib.oracle_split.argtypes = [i64, i64, vp, i64, vp, vp, i64, c_int]
        lib.oracle_split.restype = None
        lib.oracle_sgemm_cube.argtypes = [i64, i64, i64, vp, i64, vp, i64, vp, i64, c_int, c_int,
                                          i64, vp, i64]
        lib.oracle_sgemm_cube.restype = c_int
        lib.oracle_sgemm_cube_four_term.argtypes = [i64, i64, i64, vp, i64, vp, i64, vp, i64,
                                                    c_int, i64]
        lib.oracle_sgemm_cube_four_term.restype = c_int
        lib.oracle_dgemm_ref.argtypes = [i64, i64, i64, vp, i64, vp, i64, vp, vp]
        lib.oracle_dgemm_ref.restype = None
        lib.oracle_sgemm_f32.argtypes = [i64, i64, i64, vp, i64, vp, i64, vp, i64]
        lib.oracle_sgemm_f32.restype = None
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _f32_2d(x):
    x = np.asarray(x)
    if x.dtype != np.float32 or x.ndim != 2:
        raise TypeError("expected a 2-D float32 array")
    if x.strides[1] != 4 or x.strides[0] % 4 or x.strides[0] < 4 * x.shape[1]:
        x = np.ascontiguousarray(x)
    return x


def f16_rn(bits32):
    """FP32 bit patterns (uint32 array or int) -> FP16 bit patterns, RN-even."""
    lib = _load()
    if np.isscalar(bits32):
        return int(lib.oracle_f16_rn(int(bits32) & 0xFFFFFFFF))
    a = np.ascontiguousarray(bits32, dtype=np.uint32)
    out = np.empty(a.shape, dtype=np.uint16)
    lib.oracle_f16_rn_array(a.size, a.ctypes.data, out.ctypes.data)
    return out


def f16_to_f32(bits16):
    """FP16 bit patterns -> FP32 bit patterns (exact)."""
    lib = _load()
    if np.isscalar(bits16):
        return int(lib.oracle_f16_to_f32(int(bits16) & 0xFFFF))
    a = np.ascontiguousarray(bits16, dtype=np.uint16)
    out = np.empty(a.shape, dtype=np.uint32)
    lib.oracle_f16_to_f32_array(a.size, a.ctypes.data, out.ctypes.data)
    return out


def split(X, s):
    """Two-word split of a 2-D float32 array; returns (hi, lo) uint16 bit patterns."""
    lib = _load()
    X = _f32_2d(X)
    rows, cols = X.shape
    hi = np.empty((rows, cols), dtype=np.uint16)
    lo = np.empty((rows, cols), dtype=np.uint16)
    lib.oracle_split(rows, cols, X.ctypes.data, X.strides[0] // 4, hi.ctypes.data,
                     lo.ctypes.data, cols, int(s))
    return hi, lo


def sgemm_cube(A, B, s=11, order=TERMWISE, kb=64, return_hgemm=False):
    """C = hi_A hi_B + 2^-s (lo_A hi_B + hi_A lo_B) with FP32 accumulation in k-blocks of kb."""
    lib = _load()
    A, B = _f32_2d(A), _f32_2d(B)
    M, K = A.shape
    K2, N = B.shape
    if K != K2:
        raise ValueError("inner dimensions differ")
    C = np.empty((M, N), dtype=np.float32)
    H = np.empty((M, N), dtype=np.float32) if return_hgemm else None
    kb = int(kb) if kb else max(K, 1)
    rc = lib.oracle_sgemm_cube(M, N, K, A.ctypes.data, A.strides[0] // 4, B.ctypes.data,
                               B.strides[0] // 4, C.ctypes.data, N, int(s), int(order), kb,
                               H.ctypes.data if return_hgemm else None, N)
    if rc != 0:
        raise ValueError("oracle_sgemm_cube: invalid argument")
    return (C, H) if return_hgemm else C


def sgemm_cube_four_term(A, B, s=11, kb=64):
    """C = hi_A hi_B + 2^-s (lo_A hi_B + hi_A lo_B) + 2^-2s lo_A lo_B, termwise, k-blocks of kb
    (Eq. recover_eqn with the low-low product of Eq. ll_bound kept)."""
    lib = _load()
    A, B = _f32_2d(A), _f32_2d(B)
    M, K = A.shape
    K2, N = B.shape
    if K != K2:
        raise ValueError("inner dimensions differ")
    C = np.empty((M, N), dtype=np.float32)
    kb = int(kb) if kb else max(K, 1)
    rc = lib.oracle_sgemm_cube_four_term(M, N, K, A.ctypes.data, A.strides[0] // 4,
                                         B.ctypes.data, B.strides[0] // 4, C.ctypes.data, N,
                                         int(s), kb)
    if rc != 0:
        raise ValueError("oracle_sgemm_cube_four_term: invalid argument")
    return C


def dgemm_ref(A, B, with_abs=True):
    """(C64, |A||B|) accumulated in double."""
    lib = _load()
    A, B = _f32_2d(A), _f32_2d(B)
    M, K = A.shape
    _, N = B.shape
    C = np.empty((M, N), dtype=np.float64)
    AB = np.empty((M, N), dtype=np.float64) if with_abs else None
    lib.oracle_dgemm_ref(M, N, K, A.ctypes.data, A.strides[0] // 4, B.ctypes.data,
                         B.strides[0] // 4, C.ctypes.data, AB.ctypes.data if with_abs else None)
    return (C, AB) if with_abs else C


def sgemm_f32(A, B):
    """Sequential FP32 GEMM of the unsplit inputs."""
    lib = _load()
    A, B = _f32_2d(A), _f32_2d(B)
    M, K = A.shape
    _, N = B.shape
    C = np.empty((M, N), dtype=np.float32)
    lib.oracle_sgemm_f32(M, N, K, A.ctypes.data, A.strides[0] // 4, B.ctypes.data,
                         B.strides[0] // 4, C.ctypes.data, N)
    return C


def frobenius_rel_err(C, C64):
    """||C_true - C||_F / ||C_true||_F  [Eq. err]."""
    d = np.asarray(C, dtype=np.float64) - C64
    return float(np.sqrt((d * d).sum()) / np.sqrt((C64 * C64).sum()))


def componentwise_err(C, C64, ABabs):
    """max_ij |C - C64| / (|A||B|)_ij; entries with (|A||B|)_ij = 0 must be exactly zero."""
    d = np.abs(np.asarray(C, dtype=np.float64) - C64)
    zero = ABabs == 0
    if np.any(d[zero] != 0):
        return float("inf")
    if np.all(zero):
        return 0.0
    return float((d[~zero] / ABabs[~zero]).max())


def exponent_window(X):
    """[e_min, e_max, #subnormal hi, #non-finite hi, #zero hi] of the FP16 high words of X:
    the exponents E' - 15 that Eq. sf_bounds is stated on (Sec. 4.2)."""
    hi, _ = split(np.atleast_2d(np.asarray(X, dtype=np.float32)), 0)
    E = (hi.astype(np.int64) >> 10) & 0x1F
    Mant = hi.astype(np.int64) & 0x3FF
    normal = (E > 0) & (E < 0x1F)
    e = E[normal] - 15
    return [int(e.min()) if e.size else 127, int(e.max()) if e.size else -127,
            int(((E == 0) & (Mant != 0)).sum()), int((E == 0x1F).sum()), int(((E == 0) & (Mant == 0)).sum())]


def scale_exp_bounds(e_min, e_max):
    """Eq. sf_bounds: -3 - e_min <= s_b <= 26 - e_max."""
    return -3 - e_min, 26 - e_max


# ------------------------------------------------------------------ whole-input scaling
# Sec. 4.2 notes that once the high word is subnormal (|x| < 2^-14) scaling the residual alone no
# longer keeps 22 bits and that whole-input scaling is then needed, and leaves it open; Sec. 7
# lists explicit exponent management as future work.  What follows is the plain definition of
# that extension: operands are multiplied by powers of two (exact) before the split and the
# product is scaled back (exact unless the FP32 result leaves the normal range).

def hi_exponent_range(X):
    """[e_min, e_max, #non-finite] over the non-zero finite entries of X, where the exponent of
    an entry is that of its value rounded (RN-even) to an 11-bit significand, i.e. the unbiased
    exponent its FP16 high word would have if FP16 had unbounded exponent range.  (127, -127)
    if no entry qualifies."""
    X = np.asarray(X, dtype=np.float32)
    finite = np.isfinite(X)
    x = np.abs(X[finite & (X != 0)].astype(np.float64))
    n_bad = int((~finite).sum())
    if x.size == 0:
        return [127, -127, n_bad]
    m, e = np.frexp(x)                         # x = m 2^e, m in [0.5, 1)
    r = np.rint(m * 2048.0)                    # 11-bit significand, ties to even
    e_hi = e - 1 + (r == 2048.0)
    return [int(e_hi.min()), int(e_hi.max()), n_bad]


def input_scale_exps(range_a, range_b):
    """(p_A, p_B, s_b, protected): each operand is scaled by 2^p with p = 15 - e_max, which puts
    its largest high word in the top normal FP16 binade; the window can then span the whole
    normal range, for which Eq. sf_bounds leaves s_b = 11.  protected: every non-zero entry of
    both scaled operands has a normal high word (e_min + p >= -14) and no entry is inf/NaN."""
    ps, ok = [], True
    for e_min, e_max, n_bad in (range_a, range_b):
        if e_max < e_min:                      # operand has no non-zero finite entry
            ps.append(0)
        else:
            p = max(-126, min(126, 15 - e_max))
            ps.append(p)
            ok = ok and (e_min + p >= -14) and (e_max + p <= 15)
        ok = ok and n_bad == 0
    return ps[0], ps[1], 11, bool(ok)


def sgemm_cube_scaled(A, B, p_a, p_b, s=11, order=TERMWISE, kb=64):
    """2^-(p_a + p_b) * sgemm_cube(2^p_a A, 2^p_b B): whole-input scaling around Eq. recover_eqn."""
    A2 = np.ldexp(np.asarray(A, dtype=np.float32), int(p_a)).astype(np.float32)
    B2 = np.ldexp(np.asarray(B, dtype=np.float32), int(p_b)).astype(np.float32)
    C = sgemm_cube(A2, B2, s=s, order=order, kb=kb)
    return np.ldexp(C, -(int(p_a) + int(p_b))).astype(np.float32)


def residual_overflow_count(X, s):
    """Number of entries whose high word is finite while the scaled residual word is inf or NaN
    (Rule 2 of Sec. 4.2 violated for that entry): counted on the words of the pinned split."""
    hi, lo = split(np.atleast_2d(np.asarray(X, dtype=np.float32)), s)
    hi_finite = (hi & 0x7C00) != 0x7C00
    lo_nonfinite = (lo & 0x7C00) == 0x7C00
    return int((hi_finite & lo_nonfinite).sum())
