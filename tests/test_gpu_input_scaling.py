"""GPU parity of whole-input scaling (the extension Sec. 4.2 names after Rule 1): the exponent
range reduction bit-exact against the oracle, the scaled product under the usual gates and
bit-for-bit covariant under powers of two."""
import numpy as np
import pytest
import torch

import oracle
from paper_2507_23387_b200 import binding, inputs
from gpu_common import K_BLOCK, U32, padded_dev, to_dev

pytestmark = pytest.mark.gpu
T, E = binding.TERMWISE, binding.ELEMENTWISE


@pytest.fixture(scope="module")
def handle():
    h = binding.Handle(0)
    yield h
    st, det = h.sgemm_cube_check()
    h.destroy()
    assert st == 0, hex(det)


@pytest.mark.parametrize("shape", [(1, 1), (77, 131), (1024, 2048)])
def test_range_matches_oracle(handle, shape):
    for X in (inputs.exponent_spread(1, shape, -30, 17), inputs.normal(2, shape),
              inputs.uniform_range(3, shape, -40), np.zeros(shape, dtype=np.float32),
              np.ldexp(inputs.uniform_pm1(4, shape), -120).astype(np.float32)):
        assert handle.sgemm_cube_hi_exponent_range(to_dev(X)) == oracle.hi_exponent_range(X)


def test_range_special_values_and_strides(handle):
    X = np.array([[1.0, -3.0, 0.0, -0.0, 2.0 ** -15, 2.0 ** -30, 65504.0, 65519.0, 65520.0, np.inf,
                   np.nan, 2 - 2.0 ** -11, 2 - 2.0 ** -10, 2.0 ** -140, 3e38]], dtype=np.float32)
    for sub in (X, X[:, :9], X[:, 11:14], X[:, 2:4]):
        assert handle.sgemm_cube_hi_exponent_range(to_dev(sub)) == oracle.hi_exponent_range(sub)
    Y = inputs.exponent_spread(5, (33, 50), -12, 9)
    assert handle.sgemm_cube_hi_exponent_range(padded_dev(Y, 16)) == oracle.hi_exponent_range(Y)


def test_every_binade_boundary(handle):
    # the largest 24-bit values below each power of two, the power itself, and the 11-bit tie
    for e in range(-126, 127, 7):
        vals = np.array([[2.0 ** e, np.nextafter(np.float32(2.0 ** e), np.float32(0)),
                          2.0 ** e * (2 - 2.0 ** -11), 2.0 ** e * (2 - 2.0 ** -11 - 2.0 ** -23)]],
                        dtype=np.float32)
        for j in range(4):
            one = vals[:, j:j + 1]
            assert handle.sgemm_cube_hi_exponent_range(to_dev(one)) == oracle.hi_exponent_range(one), (e, j)


def test_choice_matches_oracle_rule():
    cases = [([-14, 15, 0], [-14, 15, 0]), ([-40, -20, 0], [3, 20, 0]), ([-40, -10, 0], [0, 0, 0]),
             ([0, 0, 1], [0, 0, 0]), ([127, -127, 0], [0, 0, 0]), ([-149, -130, 0], [100, 127, 0])]
    for ra, rb in cases:
        assert binding.sgemm_cube_choose_input_scaling(ra, rb) == oracle.input_scale_exps(ra, rb)


def _gates(C_gpu, A, B, pa, pb, s, order, label=""):
    K = A.shape[1]
    C64, AB = oracle.dgemm_ref(A, B)
    eta_g = oracle.componentwise_err(C_gpu, C64, AB)
    frob_g = oracle.frobenius_rel_err(C_gpu, C64)
    etas, frobs = [], []
    for okb in sorted({min(K_BLOCK[order], K), K}):
        Co = oracle.sgemm_cube_scaled(A, B, pa, pb, s, order, okb)
        etas.append(oracle.componentwise_err(Co, C64, AB))
        frobs.append(oracle.frobenius_rel_err(Co, C64))
    msg = "%s eta_gpu=%.3e frob_gpu=%.3e oracle eta=%s frob=%s" % (label, eta_g, frob_g, etas, frobs)
    assert np.isfinite(C_gpu).all(), msg
    assert eta_g <= max(2 * K, K + 14) * U32 and eta_g <= 2 * max(etas) and frob_g <= 2 * max(frobs), msg


@pytest.mark.parametrize("order", [T, E])
@pytest.mark.parametrize("e_a,e_b", [(-30, -30), (-60, 40), (20, 5), (0, 0)])
def test_auto_scaled_product_against_oracle(handle, order, e_a, e_b):
    M, N, K = 300, 260, 700
    A = inputs.uniform_range(7, (M, K), e_a, False, stream=0)
    B = inputs.uniform_range(7, (K, N), e_b, False, stream=1)
    C = torch.full((M, N), float("nan"), device="cuda:0")
    chosen = handle.sgemm_cube_auto_scaled(to_dev(A), to_dev(B), C, order)
    want = oracle.input_scale_exps(oracle.hi_exponent_range(A), oracle.hi_exponent_range(B))
    assert chosen == want
    _gates(C.cpu().numpy(), A, B, chosen[0], chosen[1], chosen[2], order, "e=%d,%d" % (e_a, e_b))


def test_tiny_inputs_need_the_scaling(handle):
    A = inputs.uniform_range(8, (256, 512), -30, False, stream=0)
    B = inputs.uniform_range(8, (512, 256), -30, False, stream=1)
    C64 = oracle.dgemm_ref(A, B, with_abs=False)
    C = torch.empty((256, 256), device="cuda:0")
    handle.sgemm_cube(to_dev(A), to_dev(B), C, 12, T)
    plain = oracle.frobenius_rel_err(C.cpu().numpy(), C64)
    handle.sgemm_cube_auto_scaled(to_dev(A), to_dev(B), C, T)
    scaled = oracle.frobenius_rel_err(C.cpu().numpy(), C64)
    assert plain > 0.5 and scaled < 5e-7


def test_scale_covariance_bit_for_bit(handle):
    A, B = inputs.make_pair("normal", 9, 200, 300, 400)
    base = None
    for a, b in ((0, 0), (-37, 9), (20, -50), (-55, -55)):
        A2, B2 = np.ldexp(A, a).astype(np.float32), np.ldexp(B, b).astype(np.float32)
        C = torch.empty((200, 300), device="cuda:0")
        handle.sgemm_cube_auto_scaled(to_dev(A2), to_dev(B2), C, T)
        C0 = np.ldexp(C.cpu().numpy().astype(np.float64), -(a + b))
        if base is None:
            base = C0
        assert np.array_equal(C0, base), (a, b)


def test_explicit_exponents_and_plain_equivalence(handle):
    # magnitudes in [2^-3, 2^4): every high word stays normal under the shifts used below
    A = inputs.exponent_spread(10, (150, 260), -3, 3)
    B = inputs.exponent_spread(11, (260, 132), -3, 3)
    Ad, Bd = to_dev(A), to_dev(B)
    C0 = torch.empty((150, 132), device="cuda:0")
    C1 = torch.empty((150, 132), device="cuda:0")
    handle.sgemm_cube_set_option(binding.OPT_STRATEGY, binding.STRATEGY_TWO_PHASE)
    handle.sgemm_cube(Ad, Bd, C0, 11, T)
    handle.sgemm_cube_set_option(binding.OPT_STRATEGY, binding.STRATEGY_AUTO)
    handle.sgemm_cube_scaled(Ad, Bd, C1, 0, 0, 11, T)
    assert torch.equal(C0, C1)                       # p = 0: the plain two-phase path
    handle.sgemm_cube_scaled(Ad, Bd, C1, 5, -5, 11, T)
    assert torch.equal(C0, C1)                       # powers of two that cancel change nothing here
    handle.sgemm_cube_scaled(Ad, Bd, C1, 3, 4, 11, T)
    _gates(C1.cpu().numpy(), A, B, 3, 4, 11, T)


def test_results_that_leave_the_fp32_range_round_once(handle):
    # operands near 2^-70: the product is FP32-subnormal; the way back must round once, as ldexp
    A = np.ldexp(inputs.uniform_pm1(11, (64, 96)), -70).astype(np.float32)
    B = np.ldexp(inputs.uniform_pm1(12, (96, 40)), -70).astype(np.float32)
    C = torch.empty((64, 40), device="cuda:0")
    pa, pb, s, _ = handle.sgemm_cube_auto_scaled(to_dev(A), to_dev(B), C, T)
    want = oracle.sgemm_cube_scaled(A, B, pa, pb, s, T, 96)
    got = C.cpu().numpy()
    assert np.all(np.abs(got.astype(np.float64) - want.astype(np.float64)) <= 2.0 ** -149)
    assert np.any(got != 0)


def test_argument_errors(handle):
    A = torch.zeros((4, 4), device="cuda:0")
    for pa, pb in ((127, 0), (0, -127)):
        with pytest.raises(binding.SgemmCubeError) as e:
            handle.sgemm_cube_scaled(A, A, A, pa, pb, 11, T)
        assert e.value.status == binding.INVALID_ARG
