"""GPU parity of the exponent-window reduction and the scale choice (Sec. 4.2, Eq. sf_bounds)."""
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


@pytest.mark.parametrize("shape", [(1, 1), (77, 131), (1024, 2048)])
def test_window_matches_oracle(handle, shape):
    for X in (inputs.exponent_spread(1, shape, -30, 17), inputs.normal(2, shape),
              inputs.uniform_range(3, shape, -9), np.zeros(shape, dtype=np.float32)):
        assert handle.sgemm_cube_exponent_window(to_dev(X)) == oracle.exponent_window(X)


def test_window_special_values_and_strides(handle):
    X = np.array([[1.0, -3.0, 0.0, -0.0, 2.0 ** -15, 2.0 ** -30, 65504.0, 65520.0, np.inf, np.nan,
                   2.0 ** -14, 1e-3, 2047.9]], dtype=np.float32)
    assert handle.sgemm_cube_exponent_window(to_dev(X)) == oracle.exponent_window(X)
    Y = inputs.exponent_spread(5, (33, 50), -12, 9)
    assert handle.sgemm_cube_exponent_window(padded_dev(Y, 16)) == oracle.exponent_window(Y)


def test_scale_choice_follows_sf_bounds(handle):
    full = [-14, 15, 0, 0, 0]
    assert binding.sgemm_cube_choose_scale_exp(full, full) == (11, True)       # unique fixed choice
    assert binding.sgemm_cube_choose_scale_exp([-14, 14, 0, 0, 0], [-3, 2, 0, 0, 7]) == (12, True)
    assert binding.sgemm_cube_choose_scale_exp([-8, -1, 0, 0, 0], [-8, 0, 0, 0, 0]) == (15, True)
    assert binding.sgemm_cube_choose_scale_exp([-8, 0, 3, 0, 0], [-8, 0, 0, 0, 0]) == (15, False)
    assert binding.sgemm_cube_choose_scale_exp([-8, 15, 0, 1, 0], [-8, 0, 0, 0, 0]) == (11, False)
    assert binding.sgemm_cube_choose_scale_exp([127, -127, 0, 0, 9], [127, -127, 0, 0, 9]) == (15, True)
    for (lo, hi) in [(-14, 15), (-10, 10), (0, 0), (-14, 3)]:
        s, ok = binding.sgemm_cube_choose_scale_exp([lo, hi, 0, 0, 0], [lo, hi, 0, 0, 0])
        b_lo, b_hi = oracle.scale_exp_bounds(lo, hi)
        assert ok and b_lo <= s <= b_hi


def test_chosen_scale_keeps_the_split_inside_its_error_bound(handle):
    # end to end: window -> scale -> split; every residual in range, Eq. split_error holds
    X = inputs.exponent_spread(9, (256, 512), -12, 12)
    win = handle.sgemm_cube_exponent_window(to_dev(X))
    s, ok = binding.sgemm_cube_choose_scale_exp(win, win)
    assert ok and s == 26 - win[1]
    hi = torch.empty((256, 512), dtype=torch.float16, device="cuda:0")
    lo = torch.empty_like(hi)
    handle.sgemm_cube_split(to_dev(X), hi, lo, s)
    rec = hi.double().cpu().numpy() + lo.double().cpu().numpy() * 2.0 ** -s
    assert np.isfinite(rec).all()
    assert np.all(np.abs(rec - X.astype(np.float64)) <= 2.0 ** -22 * np.abs(X.astype(np.float64)))


def test_residual_overflow_count_matches_oracle(handle):
    V = np.array([[32784.0, 1.0, -32784.0, 0.5, 70000.0, np.inf, np.nan, 65000.0]], dtype=np.float32)
    X = inputs.exponent_spread(9, (300, 520), 5, 15)
    for src in (V, X):
        for s in (0, 8, 11, 12, 15):
            Xd = to_dev(src)
            hi = torch.empty(Xd.shape, dtype=torch.float16, device="cuda:0")
            lo = torch.empty_like(hi)
            handle.sgemm_cube_split(Xd, hi, lo, s)
            assert handle.sgemm_cube_residual_overflow_count(hi, lo) == oracle.residual_overflow_count(src, s)
    # what sgemm_cube_choose_scale_exp returns never overflows a residual
    win = handle.sgemm_cube_exponent_window(to_dev(X))
    s, _ = binding.sgemm_cube_choose_scale_exp(win, win)
    assert oracle.residual_overflow_count(X, s) == 0 and oracle.residual_overflow_count(X, 15) > 0
