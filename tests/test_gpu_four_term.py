"""GPU parity of sgemm_cube_four_term (the low-low product kept) against the oracle's four-term
function: exact where the arithmetic is exact, else the componentwise gate against FP64 and at
most twice the oracle's own error.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2507_23387_b200 import binding, inputs
from gpu_common import K_BLOCK, U32, padded_dev, to_dev

pytestmark = pytest.mark.gpu

KB = K_BLOCK[binding.TERMWISE]


@pytest.fixture(scope="module")
def handle():
    h = binding.Handle(0)
    yield h
    st, det = h.sgemm_cube_check()
    h.destroy()
    assert st == 0, hex(det)


def run4(h, A, B, s=11):
    Ad, Bd = to_dev(A), to_dev(B)
    C = torch.full((A.shape[0], B.shape[1]), float("nan"), device="cuda:0")
    h.sgemm_cube_four_term(Ad, Bd, C, s)
    st, det = h.sgemm_cube_check()
    assert st == 0, hex(det)
    return C.cpu().numpy()


def gates4(C_gpu, A, B, s, label=""):
    K = A.shape[1]
    C64, AB = oracle.dgemm_ref(A, B)
    eta_g = oracle.componentwise_err(C_gpu, C64, AB)
    frob_g = oracle.frobenius_rel_err(C_gpu, C64)
    etas, frobs = [], []
    for okb in sorted({min(KB, K), K}):
        Co = oracle.sgemm_cube_four_term(A, B, s=s, kb=okb)
        etas.append(oracle.componentwise_err(Co, C64, AB))
        frobs.append(oracle.frobenius_rel_err(Co, C64))
    msg = "%s eta_gpu=%.3e frob_gpu=%.3e oracle eta=%s frob=%s" % (label, eta_g, frob_g, etas, frobs)
    assert np.isfinite(C_gpu).all(), msg
    assert eta_g <= max(2 * K, K + 14) * U32, msg
    assert eta_g <= 2 * max(etas), msg
    assert frob_g <= 2 * max(frobs), msg
    return eta_g, frob_g


def test_low_low_term_exact_structure(handle):
    # Entries p + q 2^-13 (hi = p, residual exact); rows of A against columns of B whose hi*hi
    # stream cancels exactly, so that cross 2^-13 + low-low 2^-26 fits FP32: bit-exact equality
    # with the oracle and with the exact product shows the fourth term and its 2^-2s scale.
    rng = np.random.default_rng(5)
    M, N, K = 130, 260, 2
    p = rng.integers(1, 4, (M, 1))
    qA = rng.integers(-3, 4, (M, K))
    A = (p + qA * 2.0 ** -13).astype(np.float32)
    pb = rng.integers(1, 4, (1, N))
    qB = rng.integers(-3, 4, (K, N))
    sign = np.array([[1.0], [-1.0]])
    B = (sign * (pb + qB * 2.0 ** -13)).astype(np.float32)
    exact = A.astype(np.float64) @ B.astype(np.float64)
    assert np.array_equal(exact.astype(np.float32).astype(np.float64), exact)
    for s in (9, 11, 12):
        C = run4(handle, A, B, s)
        assert np.array_equal(C, oracle.sgemm_cube_four_term(A, B, s=s, kb=KB))
        assert np.array_equal(C.astype(np.float64), exact)
    C3 = oracle.sgemm_cube(A, B, s=11, order=oracle.TERMWISE, kb=KB)
    assert np.any(C3.astype(np.float64) != exact)


def test_small_integers_exact(handle):
    rng = np.random.default_rng(6)
    A = rng.integers(-8, 9, size=(200, 333)).astype(np.float32)
    B = rng.integers(-8, 9, size=(333, 270)).astype(np.float32)
    want = (A.astype(np.int64) @ B.astype(np.int64)).astype(np.float32)
    assert np.array_equal(run4(handle, A, B), want)


@pytest.mark.parametrize("kind,M,N,K", [
    ("uniform_pm1", 128, 256, 8),
    ("uniform_pm1", 300, 520, 200),
    ("normal", 257, 129, 1000),
    ("exponent_spread", 384, 512, 640),
    ("uniform_pm1", 1024, 1024, 1024),
    ("uniform_pm1", 130, 250, 9000),       # few tiles, long k: split-K slices + low-low term
])
def test_gates_against_four_term_oracle(handle, kind, M, N, K):
    A, B = inputs.make_pair(kind, 31, M, N, K)
    C = run4(handle, A, B, 11)
    gates4(C, A, B, 11, label="%s %dx%dx%d" % (kind, M, N, K))


def test_short_sums_closer_than_three_term(handle):
    A, B = inputs.make_pair("normal", 32, 512, 512, 8)
    C64, _ = oracle.dgemm_ref(A, B)
    C4 = run4(handle, A, B, 11)
    C3 = torch.empty((512, 512), device="cuda:0")
    handle.sgemm_cube(to_dev(A), to_dev(B), C3, 11, binding.TERMWISE)
    assert oracle.frobenius_rel_err(C4, C64) < 0.95 * oracle.frobenius_rel_err(C3.cpu().numpy(), C64)


def test_unaligned_views_and_repeat_calls(handle):
    A, B = inputs.make_pair("uniform_pm1", 33, 100, 77, 150)
    Ad, Bd = padded_dev(A, 1), padded_dev(B, 1)
    big = torch.full((100, 81), float("nan"), device="cuda:0")
    C = big[:, 1:78]
    handle.sgemm_cube_four_term(Ad, Bd, C, 11)
    first = C.cpu().numpy().copy()
    handle.sgemm_cube_four_term(Ad, Bd, C, 11)
    assert np.array_equal(first, C.cpu().numpy())
    gates4(first, A, B, 11)
    assert torch.isnan(big[:, 0]).all() and torch.isnan(big[:, 78:]).all()


def test_argument_errors(handle):
    A = torch.zeros((4, 4), device="cuda:0")
    with pytest.raises(binding.SgemmCubeError) as e:
        handle.sgemm_cube_four_term(A, A, A, 25)
    assert e.value.status == binding.INVALID_ARG
