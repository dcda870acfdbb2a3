"""Thin ctypes binding of libsgemm_cube.so: same names as the C ABI (include/sgemm_cube.h).

Argument marshalling only.  Tensors are torch CUDA tensors (PyTorch is used for device memory and
streams); every step of the computation runs in the library's kernels.  There is no fallback: if
the library cannot be loaded, or a call returns a non-zero status, an exception is raised.
"""
import ctypes
import os

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libsgemm_cube.so")

OK, INVALID_ARG, MISALIGNED, CUDA_ERROR, DEVICE_TIMEOUT, UNSUPPORTED_ARCH, ALLOC_FAILED, TOO_LARGE = range(8)
STATIC_SCRATCH_BYTES = 32 << 20
TERMWISE, ELEMENTWISE, ELEMENTWISE_REORDERED = 0, 1, 2
OPT_TERMWISE_K_BLOCK, OPT_ELEMENTWISE_K_BLOCK, OPT_CTA_PAIR, OPT_STRATEGY, OPT_TIME_KERNEL, OPT_SPLIT_K = range(6)
STRATEGY_AUTO, STRATEGY_FUSED, STRATEGY_TWO_PHASE = 0, 1, 2

EXPORTS = ["sgemm_cube_create", "sgemm_cube_destroy", "sgemm_cube_set_option", "sgemm_cube_split",
           "sgemm_cube", "sgemm_cube_unfused", "sgemm_cube_presplit", "sgemm_cube_hgemm",
           "sgemm_cube_four_term", "sgemm_cube_hi_exponent_range", "sgemm_cube_choose_input_scaling",
           "sgemm_cube_scaled", "sgemm_cube_auto_scaled",
           "sgemm_cube_host", "sgemm_cube_unfused_static", "sgemm_cube_check", "sgemm_cube_launch_count", "sgemm_cube_last_kernel_ms", "sgemm_cube_mean_kernel_ms",
           "sgemm_cube_exponent_window", "sgemm_cube_choose_scale_exp", "sgemm_cube_residual_overflow_count",
           "sgemm_cube_last_kernel_clock", "sgemm_cube_debug_inject_error", "sgemm_cube_debug_wait_timeout",
           "sgemm_cube_status_string", "sgemm_cube_version"]

_lib = None


class SgemmCubeError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__("%s failed: status %d (%s)" % (where, status, status_string(status)))


def load():
    """Load the shared library (raises OSError if it has not been built)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise OSError("libsgemm_cube.so is missing: build it with "
                      "`python -m paper_2507_23387_b200.build` (there is no CPU fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64
    lib.sgemm_cube_create.argtypes = [ctypes.POINTER(vp), i32]
    lib.sgemm_cube_destroy.argtypes = [vp]
    lib.sgemm_cube_set_option.argtypes = [vp, i32, i64]
    lib.sgemm_cube_split.argtypes = [vp, i32, i32, vp, i64, vp, vp, i64, i32, vp]
    gemm = [vp, i32, i32, i32, vp, i64, vp, i64, vp, i64, i32, i32, vp]
    lib.sgemm_cube.argtypes = gemm
    lib.sgemm_cube_unfused.argtypes = gemm
    lib.sgemm_cube_host.argtypes = gemm
    lib.sgemm_cube_presplit.argtypes = [vp, i32, i32, i32, vp, vp, i64, vp, vp, i64, vp, i64, i32,
                                        i32, vp]
    lib.sgemm_cube_hgemm.argtypes = [vp, i32, i32, i32, vp, i64, vp, i64, vp, i64, i32, vp]
    lib.sgemm_cube_unfused_static.argtypes = [i32, i32, i32, vp, i64, vp, i64, vp, i64, i32, vp]
    lib.sgemm_cube_four_term.argtypes = [vp, i32, i32, i32, vp, i64, vp, i64, vp, i64, i32, vp]
    lib.sgemm_cube_hi_exponent_range.argtypes = [vp, i32, i32, vp, i64, ctypes.POINTER(i64), vp]
    pi = ctypes.POINTER(i32)
    lib.sgemm_cube_choose_input_scaling.argtypes = [ctypes.POINTER(i64), ctypes.POINTER(i64), pi, pi, pi, pi]
    lib.sgemm_cube_scaled.argtypes = [vp, i32, i32, i32, vp, i64, vp, i64, vp, i64, i32, i32, i32, i32, vp]
    lib.sgemm_cube_auto_scaled.argtypes = [vp, i32, i32, i32, vp, i64, vp, i64, vp, i64, i32, vp, pi]
    lib.sgemm_cube_check.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_uint32)]
    lib.sgemm_cube_last_kernel_ms.argtypes = [vp, ctypes.POINTER(ctypes.c_float)]
    lib.sgemm_cube_mean_kernel_ms.argtypes = [vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(i32)]
    lib.sgemm_cube_exponent_window.argtypes = [vp, i32, i32, vp, i64, ctypes.POINTER(i64), vp]
    lib.sgemm_cube_residual_overflow_count.argtypes = [vp, i32, i32, vp, vp, i64, ctypes.POINTER(i64), vp]
    lib.sgemm_cube_choose_scale_exp.argtypes = [ctypes.POINTER(i64), ctypes.POINTER(i64),
                                                ctypes.POINTER(i32), ctypes.POINTER(i32)]
    lib.sgemm_cube_last_kernel_clock.argtypes = [vp, ctypes.POINTER(ctypes.c_uint64),
                                                 ctypes.POINTER(ctypes.c_uint64)]
    lib.sgemm_cube_debug_inject_error.argtypes = [vp, ctypes.c_uint32]
    lib.sgemm_cube_debug_wait_timeout.argtypes = [vp, i64, vp]
    lib.sgemm_cube_launch_count.argtypes = [vp]
    lib.sgemm_cube_launch_count.restype = i64
    lib.sgemm_cube_status_string.argtypes = [i32]
    lib.sgemm_cube_status_string.restype = ctypes.c_char_p
    lib.sgemm_cube_version.argtypes = []
    for name in EXPORTS:
        if name not in ("sgemm_cube_launch_count", "sgemm_cube_status_string"):
            getattr(lib, name).restype = i32
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load().sgemm_cube_status_string(int(status)).decode()


def sgemm_cube_version() -> int:
    return int(load().sgemm_cube_version())


def _check(status, where):
    if status != OK:
        raise SgemmCubeError(status, where)


def _stream_ptr(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _ld(t):
    assert t.dim() == 2 and t.stride(1) == 1, "row-major 2-D tensor expected"
    return t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1])


def _dev(t, dtype):
    assert t.is_cuda and t.dtype == dtype, "expected a CUDA tensor of dtype %s" % dtype
    return ctypes.c_void_p(t.data_ptr())


def sgemm_cube_unfused_static(A, B, C, scale_exp=11, stream=None):
    """Handle-free, allocation-free variant of Handle.sgemm_cube_unfused for callers that may not
    allocate device memory: it works out of a fixed 32 MiB scratch area inside the library and
    therefore only accepts problems that fit it (status TOO_LARGE otherwise).  Runs on the current
    device; calls that may overlap on the GPU must not be issued (they share the scratch)."""
    M, K = A.shape
    K2, N = B.shape
    assert K == K2 and C.shape == (M, N)
    _check(load().sgemm_cube_unfused_static(M, N, K, _dev(A, torch.float32), _ld(A),
                                            _dev(B, torch.float32), _ld(B), _dev(C, torch.float32),
                                            _ld(C), scale_exp, _stream_ptr(stream)),
           "sgemm_cube_unfused_static")


def sgemm_cube_choose_input_scaling(range_a, range_b):
    """(p_a, p_b, scale_exp, protected) for two ranges (see Handle.sgemm_cube_hi_exponent_range)."""
    ra = (ctypes.c_int64 * 3)(*[int(v) for v in range_a])
    rb = (ctypes.c_int64 * 3)(*[int(v) for v in range_b])
    pa, pb, s, prot = ctypes.c_int(0), ctypes.c_int(0), ctypes.c_int(0), ctypes.c_int(0)
    _check(load().sgemm_cube_choose_input_scaling(ra, rb, ctypes.byref(pa), ctypes.byref(pb),
                                                  ctypes.byref(s), ctypes.byref(prot)),
           "sgemm_cube_choose_input_scaling")
    return int(pa.value), int(pb.value), int(s.value), bool(prot.value)


def sgemm_cube_choose_scale_exp(window_a, window_b):
    """(scale_exp, protected) for two exponent windows (see Handle.sgemm_cube_exponent_window)."""
    wa = (ctypes.c_int64 * 5)(*[int(v) for v in window_a])
    wb = (ctypes.c_int64 * 5)(*[int(v) for v in window_b])
    s, prot = ctypes.c_int(0), ctypes.c_int(0)
    _check(load().sgemm_cube_choose_scale_exp(wa, wb, ctypes.byref(s), ctypes.byref(prot)),
           "sgemm_cube_choose_scale_exp")
    return int(s.value), bool(prot.value)


class Handle:
    """Owns one sgemm_cube_handle; methods carry the C entry points' names."""

    def __init__(self, device: int = 0):
        self._h = ctypes.c_void_p()
        self.device = int(device)
        _check(load().sgemm_cube_create(ctypes.byref(self._h), self.device), "sgemm_cube_create")

    def destroy(self):
        if self._h:
            st = load().sgemm_cube_destroy(self._h)
            self._h = ctypes.c_void_p()
            _check(st, "sgemm_cube_destroy")

    def __del__(self):
        try:
            if self._h:
                load().sgemm_cube_destroy(self._h)
                self._h = ctypes.c_void_p()
        except Exception:
            pass

    def sgemm_cube_set_option(self, option: int, value: int):
        _check(load().sgemm_cube_set_option(self._h, option, value), "sgemm_cube_set_option")

    def sgemm_cube_split(self, X, hi, lo, scale_exp=11, stream=None):
        rows, cols = X.shape
        assert hi.shape == X.shape and lo.shape == X.shape and _ld(hi) == _ld(lo)
        _check(load().sgemm_cube_split(self._h, rows, cols, _dev(X, torch.float32), _ld(X),
                                       _dev(hi, torch.float16), _dev(lo, torch.float16), _ld(hi),
                                       scale_exp, _stream_ptr(stream)), "sgemm_cube_split")

    def _gemm(self, fn, name, A, B, C, scale_exp, order, stream):
        M, K = A.shape
        K2, N = B.shape
        assert K == K2 and C.shape == (M, N)
        _check(fn(self._h, M, N, K, _dev(A, torch.float32), _ld(A), _dev(B, torch.float32), _ld(B),
                  _dev(C, torch.float32), _ld(C), scale_exp, order, _stream_ptr(stream)), name)

    def sgemm_cube(self, A, B, C, scale_exp=11, order=TERMWISE, stream=None):
        self._gemm(load().sgemm_cube, "sgemm_cube", A, B, C, scale_exp, order, stream)

    def sgemm_cube_unfused(self, A, B, C, scale_exp=11, order=TERMWISE, stream=None):
        self._gemm(load().sgemm_cube_unfused, "sgemm_cube_unfused", A, B, C, scale_exp, order, stream)

    def sgemm_cube_four_term(self, A, B, C, scale_exp=11, stream=None):
        """The variant that keeps the low-low product (termwise only)."""
        M, K = A.shape
        K2, N = B.shape
        assert K == K2 and C.shape == (M, N)
        _check(load().sgemm_cube_four_term(self._h, M, N, K, _dev(A, torch.float32), _ld(A),
                                           _dev(B, torch.float32), _ld(B), _dev(C, torch.float32),
                                           _ld(C), scale_exp, _stream_ptr(stream)),
               "sgemm_cube_four_term")

    def sgemm_cube_residual_overflow_count(self, hi, lo, stream=None):
        """Entries whose high word is finite while the scaled residual word is not."""
        rows, cols = hi.shape
        assert lo.shape == hi.shape and _ld(hi) == _ld(lo)
        out = ctypes.c_int64(0)
        _check(load().sgemm_cube_residual_overflow_count(self._h, rows, cols, _dev(hi, torch.float16),
                                                         _dev(lo, torch.float16), _ld(hi),
                                                         ctypes.byref(out), _stream_ptr(stream)),
               "sgemm_cube_residual_overflow_count")
        return int(out.value)

    def sgemm_cube_hi_exponent_range(self, X, stream=None):
        """[e_min, e_max, #inf/NaN] of the unbounded-range high-word exponents of X."""
        rows, cols = X.shape
        out = (ctypes.c_int64 * 3)()
        _check(load().sgemm_cube_hi_exponent_range(self._h, rows, cols, _dev(X, torch.float32), _ld(X),
                                                   out, _stream_ptr(stream)),
               "sgemm_cube_hi_exponent_range")
        return [int(v) for v in out]

    def sgemm_cube_scaled(self, A, B, C, p_a, p_b, scale_exp=11, order=TERMWISE, stream=None):
        M, K = A.shape
        K2, N = B.shape
        assert K == K2 and C.shape == (M, N)
        _check(load().sgemm_cube_scaled(self._h, M, N, K, _dev(A, torch.float32), _ld(A),
                                        _dev(B, torch.float32), _ld(B), _dev(C, torch.float32), _ld(C),
                                        int(p_a), int(p_b), scale_exp, order, _stream_ptr(stream)),
               "sgemm_cube_scaled")

    def sgemm_cube_auto_scaled(self, A, B, C, order=TERMWISE, stream=None):
        """Returns (p_a, p_b, scale_exp, protected) as chosen from the operands' ranges."""
        M, K = A.shape
        K2, N = B.shape
        assert K == K2 and C.shape == (M, N)
        chosen = (ctypes.c_int * 4)()
        _check(load().sgemm_cube_auto_scaled(self._h, M, N, K, _dev(A, torch.float32), _ld(A),
                                             _dev(B, torch.float32), _ld(B), _dev(C, torch.float32),
                                             _ld(C), order, _stream_ptr(stream), chosen),
               "sgemm_cube_auto_scaled")
        return int(chosen[0]), int(chosen[1]), int(chosen[2]), bool(chosen[3])

    def sgemm_cube_presplit(self, Ahi, Alo, Bhi, Blo, C, scale_exp=11, order=TERMWISE, stream=None):
        M, K = Ahi.shape
        _, N = Bhi.shape
        assert _ld(Ahi) == _ld(Alo) and _ld(Bhi) == _ld(Blo)
        h = torch.float16
        _check(load().sgemm_cube_presplit(self._h, M, N, K, _dev(Ahi, h), _dev(Alo, h), _ld(Ahi),
                                          _dev(Bhi, h), _dev(Blo, h), _ld(Bhi),
                                          _dev(C, torch.float32), _ld(C), scale_exp, order,
                                          _stream_ptr(stream)), "sgemm_cube_presplit")

    def sgemm_cube_hgemm(self, A16, B16, D, accumulate=False, stream=None):
        M, K = A16.shape
        _, N = B16.shape
        _check(load().sgemm_cube_hgemm(self._h, M, N, K, _dev(A16, torch.float16), _ld(A16),
                                       _dev(B16, torch.float16), _ld(B16), _dev(D, torch.float32),
                                       _ld(D), int(bool(accumulate)), _stream_ptr(stream)),
               "sgemm_cube_hgemm")

    def sgemm_cube_host(self, A, B, C, scale_exp=11, order=TERMWISE, stream=None):
        """A, B, C are HOST tensors (pinned memory recommended); returns when C is complete."""
        M, K = A.shape
        _, N = B.shape
        for t in (A, B, C):
            assert (not t.is_cuda) and t.dtype == torch.float32
        p = lambda t: ctypes.c_void_p(t.data_ptr())
        _check(load().sgemm_cube_host(self._h, M, N, K, p(A), _ld(A), p(B), _ld(B), p(C), _ld(C),
                                      scale_exp, order, _stream_ptr(stream)), "sgemm_cube_host")

    def sgemm_cube_check(self, stream=None):
        """Synchronise the stream; returns (status, detail) without raising."""
        detail = ctypes.c_uint32(0)
        st = load().sgemm_cube_check(self._h, _stream_ptr(stream), ctypes.byref(detail))
        return int(st), int(detail.value)

    def sgemm_cube_exponent_window(self, X, stream=None):
        """[e_min, e_max, #subnormal hi, #non-finite hi, #zero hi] of a device matrix."""
        rows, cols = X.shape
        out = (ctypes.c_int64 * 5)()
        _check(load().sgemm_cube_exponent_window(self._h, rows, cols, _dev(X, torch.float32), _ld(X),
                                                 out, _stream_ptr(stream)), "sgemm_cube_exponent_window")
        return [int(v) for v in out]

    def sgemm_cube_launch_count(self) -> int:
        return int(load().sgemm_cube_launch_count(self._h))

    def sgemm_cube_last_kernel_ms(self) -> float:
        ms = ctypes.c_float(0.0)
        _check(load().sgemm_cube_last_kernel_ms(self._h, ctypes.byref(ms)), "sgemm_cube_last_kernel_ms")
        return float(ms.value)

    def sgemm_cube_mean_kernel_ms(self):
        """(mean ms, calls averaged) over the timed sgemm_cube calls since the last query."""
        ms, n = ctypes.c_float(0.0), ctypes.c_int(0)
        _check(load().sgemm_cube_mean_kernel_ms(self._h, ctypes.byref(ms), ctypes.byref(n)),
               "sgemm_cube_mean_kernel_ms")
        return float(ms.value), int(n.value)

    def sgemm_cube_last_kernel_clock(self):
        """(SM cycles, nanoseconds) the tensor-core kernel of the last timed sgemm_cube call ran for."""
        cyc, ns = ctypes.c_uint64(0), ctypes.c_uint64(0)
        _check(load().sgemm_cube_last_kernel_clock(self._h, ctypes.byref(cyc), ctypes.byref(ns)),
               "sgemm_cube_last_kernel_clock")
        return int(cyc.value), int(ns.value)

    def sgemm_cube_debug_inject_error(self, code: int):
        _check(load().sgemm_cube_debug_inject_error(self._h, ctypes.c_uint32(code)),
               "sgemm_cube_debug_inject_error")

    def sgemm_cube_debug_wait_timeout(self, limit_clocks: int, stream=None):
        _check(load().sgemm_cube_debug_wait_timeout(self._h, ctypes.c_int64(limit_clocks),
                                                    _stream_ptr(stream)), "sgemm_cube_debug_wait_timeout")
