"""GPU test of sgemm_cube_unfused_static, the entry point for callers that cannot allocate device
memory (it works out of a fixed scratch array inside the library instead of a cudaMalloc'd
workspace).  Its result must equal that of sgemm_cube_unfused, which runs the same kernels on an
allocated workspace, on two calls in a row with different inputs: the second call finds the first
call's data in the shared scratch and must not be affected by it.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from paper_2507_23387_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _pair(seed, M, N, K):
    A, B = inputs.make_pair("normal", seed, M, N, K)
    return torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()


def test_static_scratch_variant_matches_allocating_variant_twice_in_a_row():
    torch.cuda.set_device(0)
    h = binding.Handle(0)
    try:
        # different shapes on purpose: the second problem is smaller, so stale words of the first
        # call lie right behind (and, for the padded rows, between) the regions it uses
        for seed, (M, N, K) in enumerate([(640, 520, 1000), (300, 264, 136)]):
            A, B = _pair(seed, M, N, K)
            want = torch.full((M, N), float("nan"), device="cuda:0")
            got = torch.full((M, N), float("nan"), device="cuda:0")
            h.sgemm_cube_unfused(A, B, want, 11, binding.TERMWISE)
            binding.sgemm_cube_unfused_static(A, B, got, 11)
            st, det = h.sgemm_cube_check()
            assert st == 0, hex(det)
            torch.cuda.synchronize()
            assert torch.isfinite(got).all()
            # same kernels, same order of operations: the tolerance of the other GPU tests
            # (twice the oracle's error) is met with room to spare by exact agreement
            assert np.array_equal(got.cpu().numpy(), want.cpu().numpy())
    finally:
        h.destroy()


def test_static_scratch_variant_leaves_free_device_memory_unchanged():
    """What the entry point is for: after its first (set-up) call on a device, a call takes no
    device memory.  Measured with the driver's own free-memory figure around a call, with the
    inputs and the output allocated beforehand (so that torch's allocator is not involved)."""
    torch.cuda.set_device(0)
    A, B = _pair(5, 512, 384, 256)
    C = torch.empty((512, 384), device="cuda:0")
    binding.sgemm_cube_unfused_static(A, B, C, 11)        # set-up call (the first one on this device, if no test ran before)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info(0)
    for _ in range(3):
        binding.sgemm_cube_unfused_static(A, B, C, 11)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info(0)
    assert free_after == free_before
    assert torch.isfinite(C).all()


def test_static_scratch_variant_rejects_what_does_not_fit():
    torch.cuda.set_device(0)
    M = N = K = 2048                      # needs 64 MiB of scratch; the array has 32 MiB
    A = torch.zeros((M, K), device="cuda:0")
    B = torch.zeros((K, N), device="cuda:0")
    C = torch.full((M, N), 3.0, device="cuda:0")
    with pytest.raises(binding.SgemmCubeError) as e:
        binding.sgemm_cube_unfused_static(A, B, C, 11)
    assert e.value.status == binding.TOO_LARGE
    torch.cuda.synchronize()
    assert torch.all(C == 3.0)            # nothing was enqueued
    lib = binding.load()
    assert lib.sgemm_cube_unfused_static(-1, 8, 8, A.data_ptr(), 8, B.data_ptr(), 8, C.data_ptr(), 8,
                                         11, None) == binding.INVALID_ARG
    assert lib.sgemm_cube_unfused_static(0, 8, 8, A.data_ptr(), 8, B.data_ptr(), 8, C.data_ptr(), 8,
                                         11, None) == binding.OK            # empty: nothing to do
    torch.cuda.synchronize()
    assert torch.all(C == 3.0)
