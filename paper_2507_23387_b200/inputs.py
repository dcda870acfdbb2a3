"""Seeded synthetic input generators (shared by the tests, the benchmark and the smoke check).

This module holds none of the method's arithmetic: it only draws matrices.  Every value is a pure
function of (seed, stream, element index) through a counter-based splitmix64 hash, so the CPU
oracle and the CUDA library are always fed identical bits, whatever the order of generation.

Workloads follow the paper's experiments, which use i.i.d. synthetic matrices only
(Sec. 6.1 "Experimental Setup": symmetric U[-2^e, 2^e] and non-negative U[0, 2^e] entries,
several seeds), plus the exponent-spread and normal inputs of the benchmark configurations.
"""
import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _mix(z):
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def raw_u64(seed: int, stream: int, n: int, offset: int = 0) -> np.ndarray:
    """n 64-bit words; word i depends only on (seed, stream, offset + i)."""
    with np.errstate(over="ignore"):
        key = _mix(np.uint64(seed & 0xFFFFFFFFFFFFFFFF) * _GOLDEN
                   + np.uint64(stream & 0xFFFFFFFF) + _GOLDEN)
        idx = np.arange(offset, offset + n, dtype=np.uint64)
        return _mix((idx + np.uint64(1)) * _GOLDEN + key)


def _shape_n(shape):
    shape = tuple(int(d) for d in shape)
    n = 1
    for d in shape:
        n *= d
    return shape, n


def _chunks(n, chunk=1 << 24):
    for o in range(0, n, chunk):
        yield o, min(chunk, n - o)


def uniform_pm1(seed: int, shape, stream: int = 0) -> np.ndarray:
    """i.i.d. uniform on the grid {(r - 2^23) / 2^23 : r in [0, 2^24)} of [-1, 1): exact in FP32."""
    shape, n = _shape_n(shape)
    out = np.empty(n, dtype=np.float32)
    for o, c in _chunks(n):
        r = (raw_u64(seed, stream, c, o) >> np.uint64(40)).astype(np.int64)
        out[o:o + c] = ((r - (1 << 23)).astype(np.float64) / float(1 << 23)).astype(np.float32)
    return out.reshape(shape)


def uniform_range(seed: int, shape, e: int, nonneg: bool = False, stream: int = 0) -> np.ndarray:
    """The paper's accuracy inputs: U[-2^e, 2^e] (symmetric) or U[0, 2^e] (non-negative)."""
    shape, n = _shape_n(shape)
    out = np.empty(n, dtype=np.float32)
    for o, c in _chunks(n):
        u = (raw_u64(seed, stream, c, o) >> np.uint64(11)).astype(np.float64) / float(1 << 53)
        v = u if nonneg else 2.0 * u - 1.0
        out[o:o + c] = (v * (2.0 ** e)).astype(np.float32)
    return out.reshape(shape)


def exponent_spread(seed: int, shape, emin: int = -10, emax: int = 10, stream: int = 0):
    """(-1)^b * 1.m * 2^e with m 23 uniform bits, e a uniform integer in [emin, emax], b a fair bit."""
    shape, n = _shape_n(shape)
    out = np.empty(n, dtype=np.uint32)
    span = np.uint64(emax - emin + 1)
    for o, c in _chunks(n):
        r = raw_u64(seed, stream, c, o)
        mant = (r & np.uint64(0x7FFFFF)).astype(np.uint32)
        sign = ((r >> np.uint64(23)) & np.uint64(1)).astype(np.uint32) << np.uint32(31)
        e = ((r >> np.uint64(32)) % span).astype(np.int64) + emin
        out[o:o + c] = sign | ((e + 127).astype(np.uint32) << np.uint32(23)) | mant
    return out.view(np.float32).reshape(shape)


def normal(seed: int, shape, stream: int = 0) -> np.ndarray:
    """i.i.d. N(0, 1): Box-Muller in double on two counter streams, rounded to FP32."""
    shape, n = _shape_n(shape)
    out = np.empty(n, dtype=np.float32)
    for o, c in _chunks(n):
        u1 = ((raw_u64(seed, 2 * stream + 101, c, o) >> np.uint64(11)).astype(np.float64) + 1.0) \
            / float(1 << 53)                      # (0, 1]
        u2 = (raw_u64(seed, 2 * stream + 102, c, o) >> np.uint64(11)).astype(np.float64) \
            / float(1 << 53)
        out[o:o + c] = (np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)).astype(np.float32)
    return out.reshape(shape)


def make_pair(kind: str, seed: int, M: int, N: int, K: int):
    """(A, B) for one named workload; A uses stream 0, B stream 1 of the same seed."""
    if kind == "uniform_pm1":
        return uniform_pm1(seed, (M, K), 0), uniform_pm1(seed, (K, N), 1)
    if kind == "exponent_spread":
        return exponent_spread(seed, (M, K), stream=0), exponent_spread(seed, (K, N), stream=1)
    if kind == "normal":
        return normal(seed, (M, K), 0), normal(seed, (K, N), 1)
    raise ValueError("unknown workload kind: %r" % (kind,))


# ---- constructed (adversarial) inputs for the max-norm study the paper names as missing (Sec. 6.2,
#      Sec. 7): no randomness in their structure, only in the values the structure is built from.

def cancellation_pair(seed: int, M: int, N: int, K: int, c: float):
    """(A, B) whose product cancels down to a fraction ~c of |A||B|:
    A = [X, -X], B = [Y; Y + c Z] with X, Y, Z uniform on [-1, 1), so that A B = -c X Z while
    |A||B| ~ 2 |X||Y|.  K must be even."""
    assert K % 2 == 0
    X = uniform_pm1(seed, (M, K // 2), 0)
    Y = uniform_pm1(seed, (K // 2, N), 1)
    Z = uniform_pm1(seed, (K // 2, N), 2)
    A = np.concatenate([X, -X], axis=1)
    B = np.concatenate([Y, (Y + np.float32(c) * Z).astype(np.float32)], axis=0)
    return np.ascontiguousarray(A), np.ascontiguousarray(B)


def coherent_residuals(seed: int, shape, stream: int = 0) -> np.ndarray:
    """Positive entries just under half a unit in the 11th place above an 11-bit value, all on the
    same side: x = g + 2^-11 - 2^-22 with g on the 11-bit grid in [1, 1.125).  Every entry then
    carries a residual of (nearly) the largest relative size, 2^-11, and of the same sign, so
    whatever a method does with residual products adds up along k instead of averaging out."""
    shape, n = _shape_n(shape)
    bits = (raw_u64(seed, stream, n) >> np.uint64(57)).astype(np.float64)      # 7 random bits
    x = 1.0 + bits * 2.0 ** -10 + 2.0 ** -11 - 2.0 ** -22
    return x.astype(np.float32).reshape(shape)


def device_normal(seed: int, shape, device="cuda:0"):
    """i.i.d. N(0, 1) FP32 generated on the device with a seeded torch generator, for the
    full-size workloads where host generation would dominate the run."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return torch.randn(tuple(shape), generator=g, device=device, dtype=torch.float32)
