"""The path device wait -> error word -> host status, without making any GEMM kernel fail.

Every wait inside the kernels is a bounded spin; one that runs out writes a code into the
handle's device error word.  Two ways to put a code there safely: a host-made failure (the code is
copied into the word) and a one-CTA diagnostic kernel whose only thread of interest runs the very
same bounded wait, with a limit of a few thousand clocks, on a barrier that nothing signals."""
import pytest
import torch

from paper_2507_23387_b200 import binding, inputs

pytestmark = pytest.mark.gpu

PROBE_CODE = 0x1F0


def _small_gemm_ok(h):
    A, B = inputs.make_pair("uniform_pm1", 1, 130, 260, 96)
    Ad, Bd = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
    C = torch.full((130, 260), float("nan"), device="cuda:0")
    h.sgemm_cube(Ad, Bd, C, 11, binding.TERMWISE)
    st, det = h.sgemm_cube_check()
    assert (st, det) == (0, 0)
    assert torch.isfinite(C).all()
    return C


def test_check_reports_and_clears_a_host_injected_failure():
    h = binding.Handle(0)
    try:
        ref = _small_gemm_ok(h)
        h.sgemm_cube_debug_inject_error(0x102)
        st, det = h.sgemm_cube_check()
        assert st == binding.DEVICE_TIMEOUT and det == 0x102
        assert "bounded wait" in binding.status_string(st)
        # reported once, then cleared: the handle stays usable and computes the same result
        assert h.sgemm_cube_check() == (0, 0)
        assert torch.equal(_small_gemm_ok(h), ref)
    finally:
        h.destroy()


def test_destroy_reports_a_failure_that_was_never_collected():
    h = binding.Handle(0)
    _small_gemm_ok(h)
    h.sgemm_cube_debug_inject_error(0x104)
    with pytest.raises(binding.SgemmCubeError) as e:
        h.destroy()
    assert e.value.status == binding.DEVICE_TIMEOUT
    # a fresh handle on the same device is unaffected
    h2 = binding.Handle(0)
    try:
        _small_gemm_ok(h2)
    finally:
        h2.destroy()


@pytest.mark.parametrize("limit", [2000, 50000])
def test_bounded_wait_gives_up_records_its_code_and_leaves_the_context_usable(limit):
    h = binding.Handle(0)
    try:
        ref = _small_gemm_ok(h)
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record()
        h.sgemm_cube_debug_wait_timeout(limit)
        end.record()
        st, det = h.sgemm_cube_check()
        assert st == binding.DEVICE_TIMEOUT and det == PROBE_CODE
        # the wait ended by its own limit (well under a millisecond), not by anything external,
        # and the second waiter left on the abort flag instead of running out its 2-second limit
        assert start.elapsed_time(end) < 50.0
        assert h.sgemm_cube_check() == (0, 0)
        assert torch.equal(_small_gemm_ok(h), ref)
    finally:
        h.destroy()


def test_probe_arguments_are_checked():
    h = binding.Handle(0)
    try:
        for bad in (0, -5, 10 ** 9):
            with pytest.raises(binding.SgemmCubeError) as e:
                h.sgemm_cube_debug_wait_timeout(bad)
            assert e.value.status == binding.INVALID_ARG
        assert h.sgemm_cube_check() == (0, 0)
    finally:
        h.destroy()
