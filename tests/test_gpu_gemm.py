"""GPU parity of the SGEMM-cube GEMM entry points against the oracle.

Bit-exact where the arithmetic is exact (inputs whose partial sums need no rounding); elsewhere
the three gates of gpu_common.gates: componentwise 2 K 2^-24 (|A||B|) against FP64, and at most
twice the oracle's own componentwise and Frobenius error.  Full-size configurations are checked
on sampled rows, which the oracle computes one by one.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2507_23387_b200 import binding, inputs
from gpu_common import K_BLOCK, gates, padded_dev, to_dev

pytestmark = pytest.mark.gpu

T, E = binding.TERMWISE, binding.ELEMENTWISE


@pytest.fixture(scope="module")
def handle():
    h = binding.Handle(0)
    yield h
    st, det = h.sgemm_cube_check()
    h.destroy()
    assert st == 0, hex(det)


def run(h, path, Ad, Bd, s, order):
    """Run one entry point on device operands; returns C as numpy."""
    M, N = Ad.shape[0], Bd.shape[1]
    C = torch.full((M, N), float("nan"), device="cuda:0")
    if path in STRATEGY:
        h.sgemm_cube_set_option(binding.OPT_STRATEGY, STRATEGY[path])
        try:
            h.sgemm_cube(Ad, Bd, C, s, order)
        finally:
            h.sgemm_cube_set_option(binding.OPT_STRATEGY, binding.STRATEGY_AUTO)
    elif path == "unfused":
        h.sgemm_cube_unfused(Ad, Bd, C, s, order)
    elif path == "presplit":
        K = Ad.shape[1]
        K8, N8 = (K + 7) // 8 * 8, (N + 7) // 8 * 8
        f16 = dict(dtype=torch.float16, device="cuda:0")
        Ahi, Alo = torch.empty((M, K8), **f16)[:, :K], torch.empty((M, K8), **f16)[:, :K]
        Bhi, Blo = torch.empty((K, N8), **f16)[:, :N], torch.empty((K, N8), **f16)[:, :N]
        h.sgemm_cube_split(Ad, Ahi, Alo, s)
        h.sgemm_cube_split(Bd, Bhi, Blo, s)
        h.sgemm_cube_presplit(Ahi, Alo, Bhi, Blo, C, s, order)
    st, det = h.sgemm_cube_check()
    assert st == 0, "device error %s" % hex(det)
    return C.cpu().numpy()


# sgemm_cube with each strategy forced ("fused": converter warps; "two_phase": split kernel + one
# three-product kernel; "auto": the library's choice), and the other entry points.
STRATEGY = {"fused": binding.STRATEGY_FUSED, "two_phase": binding.STRATEGY_TWO_PHASE,
            "auto": binding.STRATEGY_AUTO}
PATHS = [("fused", T), ("fused", E), ("two_phase", T), ("two_phase", E), ("presplit", T),
         ("presplit", E), ("unfused", T)]


@pytest.mark.parametrize("path,order", PATHS)
def test_small_integers_exact(handle, path, order):
    rng = np.random.default_rng(1)
    for (M, N, K) in [(5, 7, 11), (128, 256, 64), (130, 260, 100), (300, 520, 72)]:
        A = rng.integers(-8, 9, size=(M, K)).astype(np.float32)
        B = rng.integers(-8, 9, size=(K, N)).astype(np.float32)
        C = run(handle, path, padded_dev(A, 4), padded_dev(B, 4), 11, order)
        want = (A.astype(np.int64) @ B.astype(np.int64)).astype(np.float32)
        assert np.array_equal(C, want), (M, N, K)
        assert np.array_equal(C, oracle.sgemm_cube(A, B, 11, order, K_BLOCK[order]))


@pytest.mark.parametrize("path,order", PATHS)
@pytest.mark.parametrize("s", [9, 11, 12])
def test_three_terms_kept_low_low_dropped_bit_exact(handle, path, order, s):
    # x = p + q 2^-13 (p in 4..7, q in -3..3): every partial sum of the three computed products is
    # exact in FP32, whatever the summation order or rounding mode, so the CUDA result must equal
    # the oracle's bit for bit, and both must equal the closed form without the q q' 2^-26 term.
    rng = np.random.default_rng(2)
    M, N, K = 200, 264, 48
    pA, qA = rng.integers(4, 8, (M, K)), rng.integers(-3, 4, (M, K))
    pB, qB = rng.integers(4, 8, (K, N)), rng.integers(-3, 4, (K, N))
    sgA, sgB = rng.choice([-1, 1], (M, K)), rng.choice([-1, 1], (K, N))
    A = (sgA * (pA + qA * 2.0 ** -13)).astype(np.float32)
    B = (sgB * (pB + qB * 2.0 ** -13)).astype(np.float32)
    want = ((sgA * pA) @ (sgB * pB)
            + ((sgA * pA) @ (sgB * qB) + (sgA * qA) @ (sgB * pB)) * 2.0 ** -13)
    C = run(handle, path, to_dev(A), to_dev(B), s, order)
    assert np.array_equal(C.astype(np.float64), want)
    assert np.array_equal(C, oracle.sgemm_cube(A, B, s, order, K_BLOCK[order]))


@pytest.mark.parametrize("path,order", PATHS)
@pytest.mark.parametrize("seed", [0, 1, 2, 3, 4])
def test_config1_256_cubed_uniform(handle, path, order, seed):
    A, B = inputs.make_pair("uniform_pm1", seed, 256, 256, 256)
    C = run(handle, path, to_dev(A), to_dev(B), 11, order)
    gates(C, A, B, 11, order, label="%s order %d seed %d" % (path, order, seed))


@pytest.mark.parametrize("path,order", PATHS)
@pytest.mark.parametrize("K", [1024, 4096])
def test_one_signed_inputs(handle, path, order, K):
    # U[0, 1) entries (the paper's non-negative sampling): no cancellation, so the truncation of
    # the tensor core's accumulator shows as a bias.  Same gates as everywhere else.
    A = inputs.uniform_range(2, (256, K), 0, True, stream=0)
    B = inputs.uniform_range(2, (K, 512), 0, True, stream=1)
    C = run(handle, path, to_dev(A), to_dev(B), 11, order)
    gates(C, A, B, 11, order, label="nonneg %s K=%d" % (path, K))


@pytest.mark.parametrize("path,order", PATHS)
@pytest.mark.parametrize("shape", [(1, 1, 1), (129, 257, 33), (200, 300, 136), (384, 768, 1000),
                                   (127, 8, 2049), (640, 1280, 96)])
def test_ragged_shapes(handle, path, order, shape):
    M, N, K = shape
    A, B = inputs.make_pair("normal", 11, M, N, K)
    C = run(handle, path, padded_dev(A, 4), padded_dev(B, 4), 11, order)
    gates(C, A, B, 11, order, label="%s %s" % (path, shape))


@pytest.mark.parametrize("path,order", [("fused", T), ("two_phase", T), ("two_phase", E), ("unfused", T)])
@pytest.mark.parametrize("shape", [(100003, 8, 16), (8, 100004, 24), (4, 4, 100000), (1, 4096, 1),
                                   (70000, 1, 1)])
def test_extreme_aspect_ratios(handle, path, order, shape):
    # one dimension far beyond the others: tile counts, grid sizes and 64-bit offsets
    M, N, K = shape
    A, B = inputs.make_pair("uniform_pm1", 13, M, N, K)
    C = run(handle, path, padded_dev(A, 4), padded_dev(B, 4), 11, order)
    gates(C, A, B, 11, order, label="%s %s" % (path, shape))


@pytest.mark.parametrize("path,order", [("fused", T), ("fused", E), ("presplit", T)])
def test_output_leading_dimension_and_alignment(handle, path, order):
    M, N, K = 150, 203, 77
    A, B = inputs.make_pair("normal", 5, M, N, K)
    Ad, Bd = padded_dev(A, 4), padded_dev(B, 4)
    big = torch.full((M, 211), -7.0, device="cuda:0")
    Cv = big[:, 3:3 + N]                       # ldc = 211, pointer offset 12 bytes: scalar stores
    if path == "fused":
        handle.sgemm_cube(Ad, Bd, Cv, 11, order)
    else:
        Ahi, Alo = (torch.empty((M, 80), dtype=torch.float16, device="cuda:0")[:, :K] for _ in range(2))
        Bhi, Blo = (torch.empty((K, 208), dtype=torch.float16, device="cuda:0")[:, :N] for _ in range(2))
        handle.sgemm_cube_split(Ad, Ahi, Alo, 11)
        handle.sgemm_cube_split(Bd, Bhi, Blo, 11)
        handle.sgemm_cube_presplit(Ahi, Alo, Bhi, Blo, Cv, 11, order)
    assert handle.sgemm_cube_check()[0] == 0
    gates(Cv.cpu().numpy(), A, B, 11, order)
    assert torch.all(big[:, :3] == -7.0) and torch.all(big[:, 3 + N:] == -7.0)


def test_strategies_agree_bitwise(handle):
    # Same products, same accumulation structure: the on-the-fly split must reproduce the words of
    # the split kernel exactly, so all strategies give identical results.
    A, B = inputs.make_pair("exponent_spread", 4, 384, 512, 640)
    for order in (T, E):
        C1 = run(handle, "fused", to_dev(A), to_dev(B), 11, order)
        C2 = run(handle, "presplit", to_dev(A), to_dev(B), 11, order)
        C3 = run(handle, "two_phase", to_dev(A), to_dev(B), 11, order)
        assert np.array_equal(C1, C2) and np.array_equal(C1, C3)


@pytest.mark.parametrize("s", [0, 5, 15, 16, 20, 24])
def test_in_kernel_split_matches_the_split_kernel_for_every_scale_exponent(handle, s):
    """The converter warps have two forms of the split arithmetic (s <= 15: packed multiply and
    mixed-precision FMA; s > 15: subtract and multiply), the split kernel has one; whatever the scale
    exponent, and also on entries outside the method's comfortable range (FP16-subnormal high words,
    values near the top of the FP16 range, signed zeros), the fused kernel must produce the bits of
    the two-phase route.  Values are chosen so that nothing overflows to inf at the largest s
    (where one form gives inf and the other NaN)."""
    rng = np.random.default_rng(11 + s)
    M, N, K = 260, 520, 200
    if s <= 16:          # Rule 2 of Sec. 4.2: s <= 26 - e_max, and these inputs have e_max = 10
        A = inputs.exponent_spread(21, (M, K), stream=0)
        B = inputs.exponent_spread(21, (K, N), stream=1)
    else:                # |x| < 1: residuals stay in range up to s = 24
        A, B = inputs.make_pair("uniform_pm1", 21, M, N, K)
    # a few rows / columns of awkward values
    A[3, :] = (rng.standard_normal(K) * 2.0 ** -22).astype(np.float32)        # hi subnormal in FP16
    A[7, :] = 0.0
    A[9, ::2] = -0.0
    B[:, 5] = (rng.standard_normal(K) * 2.0 ** -17).astype(np.float32)
    if s <= 11:
        A[11, :] = (rng.uniform(20000, 60000, K) * rng.choice([-1, 1], K)).astype(np.float32)
    for order in (T, E, binding.ELEMENTWISE_REORDERED):
        ref = None
        for path in ("two_phase", "fused"):
            for pair in (1, 0):
                handle.sgemm_cube_set_option(binding.OPT_CTA_PAIR, pair)
                try:
                    C = run(handle, path, to_dev(A), to_dev(B), s, order)
                finally:
                    handle.sgemm_cube_set_option(binding.OPT_CTA_PAIR, 2)
                assert np.isfinite(C).all()
                if ref is None:
                    ref = C
                else:
                    assert np.array_equal(C, ref), (s, order, path, pair)


@pytest.mark.parametrize("n", [4096, 8192])
def test_strategies_and_cta_modes_agree_on_the_full_matrix(handle, n):
    """Several waves of the persistent grid, the partly filled last wave included: the fused
    kernel, the two-phase route and the pre-split entry point, each with CTA pairs and with single
    CTAs, must produce the same M x N matrix bit for bit (compared on the device, every element).
    What that common result is worth is checked against the oracle on the rows of tile_rows()."""
    A, B = inputs.make_pair("exponent_spread", 0, n, n, n)
    Ad, Bd = to_dev(A), to_dev(B)
    rows = tile_rows(n)
    ref = {}
    try:
        handle.sgemm_cube_set_option(binding.OPT_SPLIT_K, 0)
        for order in (T, E):
            for strategy in ("two_phase", "fused"):
                for pair in (1, 0):
                    handle.sgemm_cube_set_option(binding.OPT_CTA_PAIR, pair)
                    handle.sgemm_cube_set_option(binding.OPT_STRATEGY, STRATEGY[strategy])
                    C = torch.full((n, n), float("nan"), device="cuda:0")
                    handle.sgemm_cube(Ad, Bd, C, 11, order)
                    st, det = handle.sgemm_cube_check()
                    assert st == 0, hex(det)
                    if order not in ref:
                        ref[order] = C
                        gates(C[torch.as_tensor(rows, device="cuda:0")].cpu().numpy(), A[rows], B, 11, order,
                              label="%d^3 order %d" % (n, order))
                    else:
                        assert torch.equal(C, ref[order]), (n, order, strategy, pair)
                    del C
    finally:
        handle.sgemm_cube_set_option(binding.OPT_CTA_PAIR, 2)
        handle.sgemm_cube_set_option(binding.OPT_SPLIT_K, 1)
        handle.sgemm_cube_set_option(binding.OPT_STRATEGY, binding.STRATEGY_AUTO)


@pytest.mark.parametrize("path,order", PATHS + [("fused", binding.ELEMENTWISE_REORDERED),
                                                ("two_phase", binding.ELEMENTWISE_REORDERED)])
@pytest.mark.parametrize("kblock", [64, 128])
def test_residual_carrying_inputs_exact_over_several_stages_and_k_blocks(handle, path, order, kblock):
    """Entries +-(1 + q 2^-13), q in {-1, 0, 1}: hi = +-1 and lo = +-q 2^-2 (s = 11), so every
    product and every partial sum of every stream is a small multiple of a power of two and no
    addition rounds, on the tensor core or off it.  With K = 448 (seven 64-deep stages, 3.5
    k-blocks of 128) the look-ahead at the start of a k-block, the swapped last stage, the k-block
    drains and the ragged last k-block all carry non-zero lo words, and every path must reproduce
    the oracle (Eq. recover_eqn with Eq. termwise / Eq. elementwise) bit for bit."""
    rng = np.random.default_rng(7)
    M, N, K = 384, 520, 448
    def draw(shape):
        q = rng.integers(-1, 2, size=shape).astype(np.float64)
        sgn = rng.choice([-1.0, 1.0], size=shape)
        return (sgn * (1.0 + q * 2.0 ** -13)).astype(np.float32)
    A, B = draw((M, K)), draw((K, N))
    opt = binding.OPT_TERMWISE_K_BLOCK if order == T else binding.OPT_ELEMENTWISE_K_BLOCK
    want = oracle.sgemm_cube(A, B, 11, order, kblock)
    # exact value of the three kept terms, from the words themselves
    hiA, loA = oracle.split(A, 11)
    hiB, loB = oracle.split(B, 11)
    f = lambda w: oracle.f16_to_f32(w).view(np.float32).astype(np.float64)
    exact = f(hiA) @ f(hiB) + (f(loA) @ f(hiB) + f(hiA) @ f(loB)) * 2.0 ** -11
    assert np.array_equal(want.astype(np.float64), exact)
    assert np.any(f(loA) != 0) and np.any(f(loB) != 0)
    try:
        handle.sgemm_cube_set_option(opt, kblock)
        for pair in (1, 0):
            handle.sgemm_cube_set_option(binding.OPT_CTA_PAIR, pair)
            C = run(handle, path, padded_dev(A, 4), padded_dev(B, 4), 11, order)
            assert np.array_equal(C, want), (path, order, kblock, pair)
    finally:
        handle.sgemm_cube_set_option(binding.OPT_CTA_PAIR, 2)
        handle.sgemm_cube_set_option(opt, K_BLOCK[order])


@pytest.mark.parametrize("path,order", PATHS)
def test_cta_pair_mode_is_bit_identical(handle, path, order):
    # tcgen05.mma.cta_group::2 (two CTAs per 256 x 256 tile) against one CTA per 128 x 256 tile.
    res = {}
    try:
        handle.sgemm_cube_set_option(binding.OPT_SPLIT_K, 0)     # split-K applies to single CTAs only
        for pair in (0, 1):
            handle.sgemm_cube_set_option(binding.OPT_CTA_PAIR, pair)
            res[pair] = [run(handle, path, padded_dev(A, 4), padded_dev(B, 4), 11, order)
                         for (A, B) in (inputs.make_pair("normal", 6, M, N, K)
                                        for (M, N, K) in [(512, 768, 520), (129, 300, 97), (1024, 256, 2048)])]
    finally:
        handle.sgemm_cube_set_option(binding.OPT_CTA_PAIR, 0)
        handle.sgemm_cube_set_option(binding.OPT_SPLIT_K, 1)
    for a, b in zip(res[0], res[1]):
        assert np.array_equal(a, b)
    A, B = inputs.make_pair("normal", 6, 129, 300, 97)
    gates(res[1][1], A, B, 11, order, label="pair %s" % path)


@pytest.mark.parametrize("path,order", [("two_phase", T), ("two_phase", E), ("presplit", T)])
@pytest.mark.parametrize("shape", [(256, 256, 4096), (300, 520, 3000), (128, 256, 513), (1024, 1024, 8192)])
def test_split_k_on_few_tile_shapes(handle, path, order, shape):
    # Few tiles and a long k: the k range is cut into slices that run on otherwise idle SMs and a
    # reduction kernel adds the slices' sums.  Same gates; and switching it off must still pass.
    M, N, K = shape
    A, B = inputs.make_pair("normal", 13, M, N, K)
    Ad, Bd = padded_dev(A, 4), padded_dev(B, 4)
    res = {}
    try:
        for on in (1, 0):
            handle.sgemm_cube_set_option(binding.OPT_SPLIT_K, on)
            res[on] = run(handle, path, Ad, Bd, 11, order)
            gates(res[on], A, B, 11, order, label="split-k %d %s %s" % (on, path, shape))
    finally:
        handle.sgemm_cube_set_option(binding.OPT_SPLIT_K, 1)
    # exact inputs: identical whatever the slicing
    rng = np.random.default_rng(3)
    Ai = rng.integers(-8, 9, size=(M, K)).astype(np.float32)
    Bi = rng.integers(-8, 9, size=(K, N)).astype(np.float32)
    Ci = run(handle, path, padded_dev(Ai, 4), padded_dev(Bi, 4), 11, order)
    assert np.array_equal(Ci, (Ai.astype(np.int64) @ Bi.astype(np.int64)).astype(np.float32))


def test_k_block_option_changes_bracketing_not_validity(handle):
    A, B = inputs.make_pair("uniform_pm1", 3, 256, 256, 2048)
    Ad, Bd = to_dev(A), to_dev(B)
    try:
        for kb in (64, 128, 512):
            handle.sgemm_cube_set_option(binding.OPT_TERMWISE_K_BLOCK, kb)
            C = run(handle, "fused", Ad, Bd, 11, T)
            gates(C, A, B, 11, T, kb=kb, label="kblock %d" % kb)
    finally:
        handle.sgemm_cube_set_option(binding.OPT_TERMWISE_K_BLOCK, K_BLOCK[T])
    with pytest.raises(binding.SgemmCubeError):
        handle.sgemm_cube_set_option(binding.OPT_TERMWISE_K_BLOCK, 100)


def tile_rows(M, extra=0, seed=0):
    """One row out of every 128-row block of the result (so every row tile, both CTAs of every
    256-row pair tile and, since whole rows are compared, every column tile and every wave of the
    persistent grid is looked at), at an offset inside the block that changes from block to block
    (all four lane quarters of the accumulator), plus `extra` random rows."""
    rows = {min(M - 1, b * 128 + (b * 37 + 5) % 128) for b in range((M + 127) // 128)}
    if extra:
        rows |= set(np.random.default_rng(seed).choice(M, extra, replace=False).tolist())
    return np.array(sorted(rows))


def _sampled_rows_check(handle, path, order, A_rows_np, B_np, C_dev, rows, label):
    C_rows = C_dev[torch.as_tensor(rows, device="cuda:0")].cpu().numpy()
    return gates(C_rows, A_rows_np, B_np, 11, order, label=label)


@pytest.mark.parametrize("path,order", PATHS)
def test_config2_4096_cubed_sampled_rows(handle, path, order):
    n = 4096
    A, B = inputs.make_pair("uniform_pm1", 0, n, n, n)
    rows = tile_rows(n, extra=16, seed=0)
    Ad, Bd = to_dev(A), to_dev(B)
    C = torch.from_numpy(run(handle, path, Ad, Bd, 11, order)).to("cuda:0")
    _sampled_rows_check(handle, path, order, A[rows], B, C, rows, "4096^3 %s %d" % (path, order))


def test_config2_orders_compared(handle):
    # Both orders run on the same 4096^3 input; each passes its gates (above); here their errors
    # are put side by side on sampled rows, as the configuration asks.
    n = 4096
    A, B = inputs.make_pair("uniform_pm1", 1, n, n, n)
    rows = np.arange(0, n, 128)
    Ad, Bd = to_dev(A), to_dev(B)
    C64, AB = oracle.dgemm_ref(A[rows], B)
    errs = {}
    for order in (T, E):
        C = torch.empty((n, n), device="cuda:0")
        handle.sgemm_cube(Ad, Bd, C, 11, order)
        assert handle.sgemm_cube_check()[0] == 0
        errs[order] = oracle.frobenius_rel_err(C[torch.as_tensor(rows, device="cuda:0")].cpu().numpy(), C64)
    assert errs[T] < 2e-6 and errs[E] < 2e-6
    assert 0.25 < errs[T] / errs[E] < 4.0


@pytest.mark.parametrize("path,order", [("auto", T), ("fused", T), ("presplit", T), ("unfused", T)])
def test_config3_8192_cubed_exponent_spread_sampled_rows(handle, path, order):
    n = 8192
    A, B = inputs.make_pair("exponent_spread", 0, n, n, n)
    rows = tile_rows(n)
    Ad, Bd = to_dev(A), to_dev(B)
    C = torch.from_numpy(run(handle, path, Ad, Bd, 11, order))
    gates(C[torch.as_tensor(rows)].numpy(), A[rows], B, 11, order, label="8192^3 %s" % path)


@pytest.mark.parametrize("path,order", [("auto", T), ("auto", E), ("fused", T), ("fused", E),
                                        ("presplit", T), ("unfused", T)])
def test_config4_long_k_normal(handle, path, order):
    M = N = 1024
    K = 65536
    A, B = inputs.make_pair("normal", 0, M, N, K)
    rows = np.arange(0, M, 32)
    C = run(handle, path, to_dev(A), to_dev(B), 11, order)
    gates(C[rows], A[rows], B, 11, order, label="long-K %s %d" % (path, order))


def test_config4_error_growth_termwise_vs_elementwise(handle):
    # Error as K grows (N(0,1) inputs): both orders stay far below the plain FP32 sequential sum
    # at long K, and neither grows faster than sqrt(K) x 4.
    M = N = 256
    res = {}
    for K in (1024, 16384, 65536):
        A, B = inputs.make_pair("normal", 2, M, N, K)
        C64 = oracle.dgemm_ref(A, B, with_abs=False)
        for order in (T, E):
            res[(K, order)] = oracle.frobenius_rel_err(run(handle, "fused", to_dev(A), to_dev(B), 11, order), C64)
        res[(K, "f32")] = oracle.frobenius_rel_err(oracle.sgemm_f32(A, B), C64)
    for order in (T, E):
        assert res[(65536, order)] < res[(65536, "f32")] / 2
        assert res[(65536, order)] < 4 * 8 * res[(1024, order)]


@pytest.mark.parametrize("shape", [(2048, 2048, 2048), (16384, 16384, 1024), (12288, 12288, 12288),
                                   (16384, 16384, 16384)])
def test_config5_large_shapes_sampled_rows(handle, shape):
    M, N, K = shape
    A = inputs.device_normal(0, (M, K))
    B = inputs.device_normal(1, (K, N))
    C = torch.empty((M, N), device="cuda:0")
    handle.sgemm_cube(A, B, C, 11, T)
    assert handle.sgemm_cube_check()[0] == 0
    rows = tile_rows(M)
    idx = torch.as_tensor(rows, device="cuda:0")
    gates(C[idx].cpu().numpy(), A[idx].cpu().numpy(), B.cpu().numpy(), 11, T, label=str(shape))
    # properties that hold at any size: a permutation of A's rows permutes C's rows exactly
    perm = torch.randperm(256, device="cuda:0", generator=torch.Generator("cuda:0").manual_seed(0))
    A2 = A[:256][perm].contiguous()
    C2 = torch.empty((256, N), device="cuda:0")
    handle.sgemm_cube_set_option(binding.OPT_SPLIT_K, 0)      # same k bracketing as the full problem
    try:
        handle.sgemm_cube(A2, B, C2, 11, T)
    finally:
        handle.sgemm_cube_set_option(binding.OPT_SPLIT_K, 1)
    assert torch.equal(C2, C[:256][perm])


@pytest.mark.parametrize("strategy", ["two_phase", "fused"])
def test_operands_beyond_2_pow_31_elements(handle, strategy):
    # A has 2.18e9 elements (8.7 GB): element offsets of its last rows, of the FP16 word matrices
    # and of the workspace need 64 bits.  Rows from both ends are checked against the oracle.
    M, N, K = 66000, 8, 33000
    A = inputs.device_normal(3, (M, K))
    B = inputs.device_normal(4, (K, N))
    C = torch.full((M, N), float("nan"), device="cuda:0")
    handle.sgemm_cube_set_option(binding.OPT_STRATEGY, STRATEGY[strategy])
    try:
        handle.sgemm_cube(A, B, C, 11, T)
    finally:
        handle.sgemm_cube_set_option(binding.OPT_STRATEGY, binding.STRATEGY_AUTO)
    assert handle.sgemm_cube_check()[0] == 0
    assert torch.isfinite(C).all()
    rows = np.array([0, 1, 127, 128, 32768, 65071, 65072, 65535, 65998, 65999])
    idx = torch.as_tensor(rows, device="cuda:0")
    gates(C[idx].cpu().numpy(), A[idx].cpu().numpy(), B.cpu().numpy(), 11, T, label="2^31 " + strategy)
    del A, B, C
    torch.cuda.empty_cache()


def test_b_and_c_beyond_2_pow_31_elements(handle):
    # B with 2.18e9 elements (columns of its last rows are far beyond 2^31), then C with 2.15e9.
    K, N = 33000, 66000
    A = inputs.device_normal(5, (8, K))
    B = inputs.device_normal(6, (K, N))
    C = torch.full((8, N), float("nan"), device="cuda:0")
    handle.sgemm_cube(A, B, C, 11, T)
    assert handle.sgemm_cube_check()[0] == 0 and torch.isfinite(C).all()
    cols = np.array([0, 255, 256, 40000, 65535, 65999])
    cidx = torch.as_tensor(cols, device="cuda:0")
    gates(C[:, cidx].cpu().numpy(), A.cpu().numpy(), B[:, cidx].cpu().numpy(), 11, T, label="B > 2^31")
    del A, B, C
    torch.cuda.empty_cache()
    M = N = 46400
    A = inputs.device_normal(7, (M, 16))
    B = inputs.device_normal(8, (16, N))
    C = torch.full((M, N), float("nan"), device="cuda:0")
    handle.sgemm_cube(A, B, C, 11, T)
    assert handle.sgemm_cube_check()[0] == 0
    rows = np.array([0, 127, 30000, 46271, 46272, 46399])
    ridx = torch.as_tensor(rows, device="cuda:0")
    Crows = C[ridx]
    assert torch.isfinite(Crows).all() and torch.isfinite(C[:, N - 1]).all()
    gates(Crows.cpu().numpy(), A[ridx].cpu().numpy(), B.cpu().numpy(), 11, T, label="C > 2^31")
    del A, B, C
    torch.cuda.empty_cache()


@pytest.mark.parametrize("path,order", [("fused", T), ("fused", E), ("two_phase", T), ("two_phase", E)])
def test_special_values_propagate_like_the_oracle(handle, path, order):
    # inf, NaN, values beyond the FP16 range (hi = inf), zero rows and columns: IEEE semantics end
    # to end (nothing is clamped), so every entry has the class (NaN / +inf / -inf / finite) the
    # oracle gives it, and the rows and columns that saw no special value pass the usual gates.
    A, B = inputs.make_pair("uniform_pm1", 1, 130, 260, 96)
    A, B = A.copy(), B.copy()
    A[3, 5], A[7, 9], A[11, 2], A[20, 0], A[21, 1] = np.inf, -np.inf, np.nan, 70000.0, -1e30
    B[4, 17], B[50, 100] = np.inf, np.nan
    A[40, :] = 0
    B[:, 200] = 0
    C = run(handle, path, to_dev(A), to_dev(B), 11, order)
    Co = oracle.sgemm_cube(A, B, 11, order, K_BLOCK[order])

    def cls(x):
        return np.where(np.isnan(x), 2, np.where(np.isinf(x), np.sign(x), 0)).astype(np.int8)
    assert np.array_equal(cls(C), cls(Co))
    assert np.all(C[40, np.isfinite(C[40])] == 0) and np.all(C[np.isfinite(C[:, 200]), 200] == 0)
    clean_rows = [i for i in range(130) if i not in (3, 7, 11, 20, 21)]
    clean_cols = [j for j in range(260) if j not in (17, 100)]
    sub = C[np.ix_(clean_rows, clean_cols)]
    gates(sub, np.ascontiguousarray(A[clean_rows]), np.ascontiguousarray(B[:, clean_cols]), 11, order,
          label="rows and columns without special values")


R = binding.ELEMENTWISE_REORDERED


@pytest.mark.parametrize("path", ["fused", "two_phase", "presplit"])
@pytest.mark.parametrize("shape", [(129, 257, 33), (300, 520, 200), (512, 768, 1000), (1024, 1024, 4096)])
def test_reordered_elementwise_order(handle, path, shape):
    M, N, K = shape
    A, B = inputs.make_pair("normal", 17, M, N, K)
    C = run(handle, path, padded_dev(A, 4), padded_dev(B, 4), 11, R)
    gates(C, A, B, 11, R, label="reordered %s %s" % (path, shape))
    # one-signed data: same gates
    A2 = inputs.uniform_range(3, (M, K), 0, True, stream=0)
    B2 = inputs.uniform_range(3, (K, N), 0, True, stream=1)
    gates(run(handle, path, padded_dev(A2, 4), padded_dev(B2, 4), 11, R), A2, B2, 11, R, label="nonneg")


@pytest.mark.parametrize("path", ["fused", "two_phase"])
@pytest.mark.parametrize("s,kblock", [(15, 64), (16, 64), (11, 256), (0, 64)])
def test_reordered_elementwise_both_forms_of_the_kernel(handle, path, s, kblock):
    """The reordered order has two realisations in the kernel: for s <= 15 and k-blocks short enough
    to be resident at once, a block's value P_x / s_f + P_hh is formed inside one accumulator (the
    first hi*hi MMA scales the accumulator by 2^-s as it adds) and the two accumulators alternate
    between blocks; otherwise both partial sums are read and combined in registers.  Same order of
    Sec. 4.5 (last paragraph), same gates, for scale exponents and k-blocks on both sides."""
    M, N, K = 300, 520, 1000
    A, B = inputs.make_pair("exponent_spread", 5, M, N, K)
    if s == 0:
        A, B = inputs.make_pair("uniform_pm1", 5, M, N, K)
    try:
        handle.sgemm_cube_set_option(binding.OPT_ELEMENTWISE_K_BLOCK, kblock)
        for pair in (1, 0):
            handle.sgemm_cube_set_option(binding.OPT_CTA_PAIR, pair)
            C = run(handle, path, padded_dev(A, 4), padded_dev(B, 4), s, R)
            gates(C, A, B, s, R, kb=kblock, label="reordered %s s=%d kblock=%d pair=%d" % (path, s, kblock, pair))
    finally:
        handle.sgemm_cube_set_option(binding.OPT_CTA_PAIR, 2)
        handle.sgemm_cube_set_option(binding.OPT_ELEMENTWISE_K_BLOCK, K_BLOCK[R])


def test_reordered_elementwise_keeps_what_a_block_adds_up_to(handle):
    # Block 0 makes the accumulator 2^10 (ulp 2^-13).  Block 1 holds hi*hi = 2^-14 (1 - 2^-20),
    # just under half an ulp, and a correction of 2^-29: added one after the other to the
    # accumulator both are lost (Eq. elementwise, also as the kernel realises it); added
    # together first they exceed half an ulp and the sum rounds up (Sec. 4.5, last paragraph).
    a_hi = 2.0 ** -7 * (1 + 2.0 ** -10)
    b = 2.0 ** -7 * (1 - 2.0 ** -10)
    a = a_hi + 2.0 ** -22                      # residual 2^-22, far inside half an FP16 ulp
    A = np.zeros((128, 128), dtype=np.float32)
    B = np.zeros((128, 256), dtype=np.float32)
    A[:, 0], B[0, :] = 32.0, 32.0
    A[:, 64], B[64, :] = a, b
    assert float(A[0, 64]) == a and float(B[64, 0]) == b
    for path in ("fused", "two_phase"):
        el = run(handle, path, to_dev(A), to_dev(B), 11, E)
        ro = run(handle, path, to_dev(A), to_dev(B), 11, R)
        assert np.all(el == np.float32(1024.0))
        assert np.all(ro == np.float32(1024.0 + 2.0 ** -13))
        assert np.array_equal(ro, oracle.sgemm_cube(A, B, 11, R, 64))
        assert np.array_equal(el, oracle.sgemm_cube(A, B, 11, E, 64))


def test_hgemm_matches_fp64_product_of_fp16_inputs(handle):
    for (M, N, K) in [(128, 256, 64), (200, 300, 136), (1024, 1024, 1024)]:
        A = inputs.normal(1, (M, (K + 7) // 8 * 8))[:, :K]
        B = inputs.normal(2, (K, (N + 7) // 8 * 8))[:, :N]
        Ad = padded_dev(A.astype(np.float16), 8)
        Bd = padded_dev(B.astype(np.float16), 8)
        D = torch.full((M, N), float("nan"), device="cuda:0")
        handle.sgemm_cube_hgemm(Ad, Bd, D)
        ref = A.astype(np.float16).astype(np.float64) @ B.astype(np.float16).astype(np.float64)
        AB = np.abs(A.astype(np.float16).astype(np.float64)) @ np.abs(B.astype(np.float16).astype(np.float64))
        assert np.all(np.abs(D.cpu().numpy() - ref) <= 2 * K * 2.0 ** -24 * AB)
        D2 = D.clone()
        handle.sgemm_cube_hgemm(Ad, Bd, D2, accumulate=True)
        assert np.allclose(D2.cpu().numpy(), 2 * D.cpu().numpy(), rtol=0, atol=0)


def test_argument_errors(handle):
    A = torch.zeros((8, 16), device="cuda:0")
    B = torch.zeros((16, 8), device="cuda:0")
    C = torch.zeros((8, 8), device="cuda:0")
    lib = binding.load()
    p = lambda t: t.data_ptr()
    call = lambda **kw: lib.sgemm_cube(handle._h, kw.get("M", 8), kw.get("N", 8), kw.get("K", 16),
                                       kw.get("A", p(A)), kw.get("lda", 16), kw.get("B", p(B)),
                                       kw.get("ldb", 8), kw.get("C", p(C)), kw.get("ldc", 8),
                                       kw.get("s", 11), kw.get("order", 0), None)
    assert call() == binding.OK
    assert call(M=-1) == binding.INVALID_ARG
    assert call(M=0) == binding.OK                           # empty problems are valid
    assert call(K=-1) == binding.INVALID_ARG
    assert call(lda=15) == binding.INVALID_ARG
    assert call(ldc=7) == binding.INVALID_ARG
    assert call(s=25) == binding.INVALID_ARG
    assert call(order=3) == binding.INVALID_ARG and call(order=-1) == binding.INVALID_ARG
    assert call(order=2) == binding.OK                       # the reordered elementwise order
    assert call(A=None) == binding.INVALID_ARG
    assert call(A=p(A) + 4) == binding.MISALIGNED
    assert call(lda=18) == binding.MISALIGNED
    for opt, bad in ((binding.OPT_STRATEGY, 3), (binding.OPT_CTA_PAIR, 3), (binding.OPT_TIME_KERNEL, 2), (9, 0)):
        assert lib.sgemm_cube_set_option(handle._h, opt, bad) == binding.INVALID_ARG
    assert lib.sgemm_cube_unfused(handle._h, 8, 8, 16, p(A), 16, p(B), 8, p(C), 8, 11, 1,
                                  None) == binding.INVALID_ARG       # unfused is termwise only
    assert handle.sgemm_cube_check()[0] == 0


@pytest.mark.parametrize("shape", [(300, 520, 200), (1500, 1030, 1000), (2048, 1024, 1024)])
def test_host_buffer_entry_point(handle, shape):
    # small: plain copy-compute-copy; the two larger shapes take the panel pipeline (ragged last
    # panel and ragged tiles in the middle one).  Either way bit-identical to the device call.
    M, N, K = shape
    A, B = inputs.make_pair("normal", 8, M, N, K)
    Ah, Bh = torch.from_numpy(A).pin_memory(), torch.from_numpy(B).pin_memory()
    Ch = torch.full((M, N), float("nan")).pin_memory()
    for order in (T, E):
        handle.sgemm_cube_host(Ah, Bh, Ch, 11, order)
        Cd = run(handle, "auto", padded_dev(A, 4), padded_dev(B, 4), 11, order)
        assert np.array_equal(Ch.numpy(), Cd)
    # pageable host memory works too (the copies are then staged by the driver)
    C2 = torch.empty((M, N))
    handle.sgemm_cube_host(torch.from_numpy(A), torch.from_numpy(B), C2, 11, T)
    assert np.array_equal(C2.numpy(), run(handle, "auto", padded_dev(A, 4), padded_dev(B, 4), 11, T))


def test_kernel_timing_queries(handle):
    A, B = inputs.make_pair("uniform_pm1", 2, 512, 512, 512)
    Ad, Bd = to_dev(A), to_dev(B)
    C = torch.empty((512, 512), device="cuda:0")
    with pytest.raises(binding.SgemmCubeError):
        handle.sgemm_cube_last_kernel_ms()                   # timing is off by default
    handle.sgemm_cube_set_option(binding.OPT_TIME_KERNEL, 1)
    try:
        with pytest.raises(binding.SgemmCubeError):
            handle.sgemm_cube_mean_kernel_ms()               # no timed call yet
        for _ in range(3):
            handle.sgemm_cube(Ad, Bd, C, 11, T)
        last = handle.sgemm_cube_last_kernel_ms()
        mean, n = handle.sgemm_cube_mean_kernel_ms()
        assert n == 3 and 0 < mean < 50 and 0 < last < 50
        with pytest.raises(binding.SgemmCubeError):
            handle.sgemm_cube_mean_kernel_ms()               # the average restarts after a query
        for _ in range(130):                                  # more calls than event pairs are kept
            handle.sgemm_cube(Ad, Bd, C, 11, T)
        mean, n = handle.sgemm_cube_mean_kernel_ms()
        assert n == 128 and 0 < mean < 50
    finally:
        handle.sgemm_cube_set_option(binding.OPT_TIME_KERNEL, 0)


@pytest.mark.parametrize("shape", [(0, 5, 7), (5, 0, 7), (5, 8, 0), (0, 0, 0)])
def test_empty_problems(handle, shape):
    # No output elements: nothing happens.  Empty inner dimension: the empty sum, C = 0, as the
    # oracle's loops give.
    M, N, K = shape
    f32 = dict(dtype=torch.float32, device="cuda:0")
    A, B = torch.ones((M, K), **f32), torch.ones((K, N), **f32)
    want = oracle.sgemm_cube(np.ones((M, K), np.float32), np.ones((K, N), np.float32), 11, T, 64) \
        if M and N else np.zeros((M, N), np.float32)
    calls = [lambda C: handle.sgemm_cube(A, B, C, 11, T), lambda C: handle.sgemm_cube(A, B, C, 11, E),
             lambda C: handle.sgemm_cube_unfused(A, B, C, 11, T),
             lambda C: handle.sgemm_cube_four_term(A, B, C, 11),
             lambda C: handle.sgemm_cube_scaled(A, B, C, 3, -2, 11, T),
             lambda C: handle.sgemm_cube_auto_scaled(A, B, C, T),
             lambda C: binding.sgemm_cube_unfused_static(A, B, C, 11)]
    for call in calls:
        C = torch.full((M, N), 7.0, **f32)
        call(C)
        assert handle.sgemm_cube_check()[0] == 0
        assert np.array_equal(C.cpu().numpy(), want)
    f16 = dict(dtype=torch.float16, device="cuda:0")
    Ah, Bh = torch.ones((M, K), **f16), torch.ones((K, N), **f16)
    D = torch.full((M, N), 7.0, **f32)
    handle.sgemm_cube_hgemm(Ah, Bh, D, accumulate=True)
    assert torch.all(D == 7.0)                              # nothing to add
    handle.sgemm_cube_hgemm(Ah, Bh, D)
    assert np.array_equal(D.cpu().numpy(), want)
    handle.sgemm_cube_presplit(Ah, Ah.clone(), Bh, Bh.clone(), D, 11, T)
    assert np.array_equal(D.cpu().numpy(), want)
    handle.sgemm_cube_split(A, Ah, Ah.clone(), 11)          # empty split: no-op
    Ch = torch.full((M, N), 7.0).pin_memory() if M * N else torch.empty((M, N))
    handle.sgemm_cube_host(torch.ones((M, K)), torch.ones((K, N)), Ch, 11, T)
    assert np.array_equal(Ch.numpy(), want)
    with pytest.raises(binding.SgemmCubeError):
        load = binding.load()
        binding._check(load.sgemm_cube(handle._h, -1, 4, 4, None, 4, None, 4, None, 4, 11, T, None), "neg")
