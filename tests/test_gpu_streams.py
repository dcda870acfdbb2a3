"""Stream behaviour of the library: calls are pure stream-ordered work once the workspace exists, so
they can be captured into a CUDA graph and replayed, and handles on different streams do not
interfere."""
import numpy as np
import pytest
import torch

from paper_2507_23387_b200 import binding, inputs
from gpu_common import to_dev

pytestmark = pytest.mark.gpu
T, E = binding.TERMWISE, binding.ELEMENTWISE


@pytest.mark.parametrize("strategy", [binding.STRATEGY_TWO_PHASE, binding.STRATEGY_FUSED])
def test_cuda_graph_capture_and_replay(strategy):
    h = binding.Handle(0)
    try:
        h.sgemm_cube_set_option(binding.OPT_STRATEGY, strategy)
        A, B = inputs.make_pair("uniform_pm1", 41, 640, 512, 768)
        Ad, Bd = to_dev(A), to_dev(B)
        C = torch.zeros((640, 512), device="cuda:0")
        h.sgemm_cube(Ad, Bd, C, 11, T)               # first call: workspace, kernel attributes
        torch.cuda.synchronize()
        ref = C.clone()
        C.zero_()
        side = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            h.sgemm_cube(Ad, Bd, C, 11, T)            # the binding passes the current (capturing) stream
        torch.cuda.synchronize()
        assert torch.all(C == 0)                      # captured, not executed
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(C, ref)
        Ad.mul_(2.0)                                  # same buffers, new contents: exact doubling
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(C, 2.0 * ref)
        assert h.sgemm_cube_check()[0] == 0
    finally:
        h.destroy()


def test_two_handles_on_two_streams():
    h1, h2 = binding.Handle(0), binding.Handle(0)
    try:
        A1, B1 = inputs.make_pair("normal", 42, 1024, 768, 1024)
        A2, B2 = inputs.make_pair("uniform_pm1", 43, 512, 1280, 2048)
        d = [to_dev(x) for x in (A1, B1, A2, B2)]
        C1 = torch.empty((1024, 768), device="cuda:0")
        C2 = torch.empty((512, 1280), device="cuda:0")
        h1.sgemm_cube(d[0], d[1], C1, 11, T)
        h2.sgemm_cube(d[2], d[3], C2, 11, E)
        torch.cuda.synchronize()
        ref1, ref2 = C1.clone(), C2.clone()
        s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
        for _ in range(5):
            C1.fill_(float("nan"))
            C2.fill_(float("nan"))
            torch.cuda.synchronize()
            for _ in range(3):                        # interleaved submissions
                h1.sgemm_cube(d[0], d[1], C1, 11, T, stream=s1)
                h2.sgemm_cube(d[2], d[3], C2, 11, E, stream=s2)
            torch.cuda.synchronize()
            assert torch.equal(C1, ref1) and torch.equal(C2, ref2)
        assert h1.sgemm_cube_check(s1)[0] == 0 and h2.sgemm_cube_check(s2)[0] == 0
    finally:
        h1.destroy()
        h2.destroy()
