"""GPU parity of sgemm_cube_split against the oracle: bit-exact hi/lo words (NaN by class)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2507_23387_b200 import binding, inputs
from gpu_common import padded_dev, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def handle():
    h = binding.Handle(0)
    yield h
    h.destroy()


def _same_words(got, want):
    nan_g = (got & 0x7FFF) > 0x7C00
    nan_w = (want & 0x7FFF) > 0x7C00
    return np.array_equal(nan_g, nan_w) and np.array_equal(got[~nan_g], want[~nan_w])


def _gpu_split(h, Xd, s):
    hi = torch.empty(Xd.shape, dtype=torch.float16, device="cuda:0")
    lo = torch.empty_like(hi)
    h.sgemm_cube_split(Xd, hi, lo, s)
    st, det = h.sgemm_cube_check()
    assert st == 0, hex(det)
    return hi.cpu().numpy().view(np.uint16), lo.cpu().numpy().view(np.uint16)


@pytest.mark.parametrize("s", [0, 11, 12, 24])
@pytest.mark.parametrize("shape", [(256, 256), (77, 131), (1, 1), (3, 8), (513, 1032)])
def test_split_matches_oracle_bit_exact(handle, shape, s):
    X = inputs.exponent_spread(7, shape, -30, 15)
    ghi, glo = _gpu_split(handle, to_dev(X), s)
    ohi, olo = oracle.split(X, s)
    assert _same_words(ghi, ohi) and _same_words(glo, olo)


def test_split_config_inputs(handle):
    for kind in ("uniform_pm1", "exponent_spread", "normal"):
        A, _ = inputs.make_pair(kind, 0, 1024, 8, 2048)
        ghi, glo = _gpu_split(handle, to_dev(A), 11)
        ohi, olo = oracle.split(A, 11)
        assert np.array_equal(ghi, ohi) and np.array_equal(glo, olo)


def test_split_special_values(handle):
    vals = np.array([0.0, -0.0, np.inf, -np.inf, np.nan, 65504.0, 65519.99, 65520.0, 70000.0, 1e30,
                     2.0 ** -14, 2.0 ** -24, 2.0 ** -25, 2.0 ** -26, 1e-45, -1e-40, 32784.0, -32784.0,
                     1.0, 1.0 + 2.0 ** -11, 1.0 + 2.0 ** -11 + 2.0 ** -23, 1.0 + 3 * 2.0 ** -11],
                    dtype=np.float32)
    X = np.resize(vals, (4, 16)).astype(np.float32)
    for s in (0, 11, 12):
        ghi, glo = _gpu_split(handle, to_dev(X), s)
        ohi, olo = oracle.split(X, s)
        assert _same_words(ghi, ohi) and _same_words(glo, olo)


def test_split_leading_dimensions_and_unaligned_views(handle):
    X = inputs.normal(3, (64, 96))
    big = torch.zeros((64, 136), device="cuda:0")
    view = big[:, 4:100]          # ldx = 136, offset of 16 bytes, 96 columns: vector path
    view.copy_(torch.from_numpy(X))
    odd = big[:, 1:97]            # 4-byte offset: scalar path
    for src in (view, odd):
        hi = torch.zeros((64, 104), dtype=torch.float16, device="cuda:0")
        lo = torch.zeros_like(hi)
        handle.sgemm_cube_split(src, hi[:, :96], lo[:, :96], 11)
        assert handle.sgemm_cube_check()[0] == 0
        ohi, olo = oracle.split(src.cpu().numpy(), 11)
        assert np.array_equal(hi[:, :96].cpu().numpy().view(np.uint16), ohi)
        assert np.array_equal(lo[:, :96].cpu().numpy().view(np.uint16), olo)
        assert torch.count_nonzero(hi[:, 96:]) == 0       # padding untouched


def test_split_every_fp32_pattern(handle):
    # All 2^32 FP32 bit patterns, s = 11, in slabs of 2^26.
    slab = 1 << 26
    for i in range(0, 1 << 32, slab):
        w = np.arange(i, i + slab, dtype=np.uint64).astype(np.uint32).reshape(1 << 13, 1 << 13)
        ghi, glo = _gpu_split(handle, to_dev(w.view(np.float32)), 11)
        ohi, olo = oracle.split(w.view(np.float32), 11)
        assert _same_words(ghi, ohi), hex(i)
        assert _same_words(glo, olo), hex(i)


def test_split_rejects_bad_arguments(handle):
    X = torch.zeros((4, 8), device="cuda:0")
    hi = torch.zeros((4, 8), dtype=torch.float16, device="cuda:0")
    with pytest.raises(binding.SgemmCubeError) as e:
        handle.sgemm_cube_split(X, hi, hi.clone(), 25)
    assert e.value.status == binding.INVALID_ARG
    lib = binding.load()
    assert lib.sgemm_cube_split(handle._h, -1, 8, X.data_ptr(), 8, hi.data_ptr(), hi.data_ptr(), 8, 11,
                                None) == binding.INVALID_ARG
    assert lib.sgemm_cube_split(handle._h, 0, 8, None, 8, None, None, 8, 11, None) == binding.OK   # empty
    assert lib.sgemm_cube_split(handle._h, 4, 8, X.data_ptr(), 4, hi.data_ptr(), hi.data_ptr(), 8, 11,
                                None) == binding.INVALID_ARG
    assert lib.sgemm_cube_split(handle._h, 4, 8, None, 8, hi.data_ptr(), hi.data_ptr(), 8, 11,
                                None) == binding.INVALID_ARG
