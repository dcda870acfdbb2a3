"""Seeded random sweep over shapes, k-block options and accumulation orders: every way the library
can run sgemm_cube (fused converter kernel or split + three-product kernel, single CTAs or CTA
pairs) must give the same bits, and those bits must pass the oracle gates."""
import random

import numpy as np
import pytest
import torch

from paper_2507_23387_b200 import binding
from gpu_common import gates

pytestmark = pytest.mark.gpu

VARIANTS = [(binding.STRATEGY_FUSED, 0), (binding.STRATEGY_TWO_PHASE, 0), (binding.STRATEGY_TWO_PHASE, 1),
            (binding.STRATEGY_FUSED, 1)]


@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_variants_agree_bitwise_on_random_configurations(seed):
    rng = random.Random(seed)
    h = binding.Handle(0)
    try:
        h.sgemm_cube_set_option(binding.OPT_SPLIT_K, 0)        # split-K re-brackets by design
        for trial in range(25):
            M = rng.choice([1, 64, 127, 128, 129, 255, 256, 257, 300, 512, 777, 1024, 1500])
            N = rng.choice([1, 8, 100, 255, 256, 257, 512, 640, 1000, 1536])
            K = rng.choice([1, 16, 63, 64, 65, 128, 200, 512, 1000, 2048, 4100])
            kbt, kbe = rng.choice([64, 128, 256, 512]), rng.choice([64, 128, 256])
            order = rng.choice([binding.TERMWISE, binding.ELEMENTWISE, binding.ELEMENTWISE_REORDERED])
            h.sgemm_cube_set_option(binding.OPT_TERMWISE_K_BLOCK, kbt)
            h.sgemm_cube_set_option(binding.OPT_ELEMENTWISE_K_BLOCK, kbe)
            g = torch.Generator(device="cuda:0")
            g.manual_seed(1000 * seed + trial)
            K4, N4 = (K + 3) // 4 * 4, (N + 3) // 4 * 4
            A = torch.randn(M, K4, device="cuda:0", generator=g)[:, :K]
            B = torch.randn(K, N4, device="cuda:0", generator=g)[:, :N]
            results = []
            for strategy, pair in VARIANTS:
                h.sgemm_cube_set_option(binding.OPT_STRATEGY, strategy)
                h.sgemm_cube_set_option(binding.OPT_CTA_PAIR, pair)
                C = torch.full((M, N), float("nan"), device="cuda:0")
                h.sgemm_cube(A, B, C, 11, order)
                st, det = h.sgemm_cube_check()
                assert st == 0, (M, N, K, strategy, pair, hex(det))
                results.append(C)
            label = "M=%d N=%d K=%d kb=%d/%d order=%d" % (M, N, K, kbt, kbe, order)
            for r in results[1:]:
                assert torch.equal(results[0], r), label
            if trial % 5 == 0 and M * N * K <= 300 * 1000 * 1100:
                kb = kbt if order == binding.TERMWISE else kbe
                gates(results[0].cpu().numpy(), np.ascontiguousarray(A.cpu().numpy()),
                      np.ascontiguousarray(B.cpu().numpy()), 11, order, kb=kb, label=label)
    finally:
        h.destroy()
