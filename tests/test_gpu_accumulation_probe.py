"""How the tensor core accumulates, measured through sgemm_cube_hgemm on one output element.

The method's error analysis assumes round-to-nearest FP32 accumulation in the matrix unit and
notes that NVIDIA tensor cores do not provide it (Sec. 4.3, last paragraph).  The facts below are
what the library's design rests on: chains inside the tensor core are kept short (the k-block
options, default 128) and are added outside it with round-to-nearest, and the componentwise gate
of the parity tests is 2 K 2^-24 rather than K 2^-24.  Each case puts crafted FP16 values into row
0 of A and column 0 of B (everything else zero) and reads D[0, 0]; the whole k range is one chain
inside the tensor core (k-block option set far above K)."""
import pytest
import torch

from paper_2507_23387_b200 import binding

pytestmark = pytest.mark.gpu

ULP = 2.0 ** -23          # spacing of FP32 numbers in [1, 2)
E = 2.0 ** -12            # E * E = 2^-24 = half an ulp of 1


@pytest.fixture(scope="module")
def probe():
    h = binding.Handle(0)
    h.sgemm_cube_set_option(binding.OPT_TERMWISE_K_BLOCK, 1 << 20)

    def run(avals, bvals):
        K = len(avals)
        K8 = (K + 7) // 8 * 8
        A = torch.zeros((128, K8), dtype=torch.float16, device="cuda:0")
        B = torch.zeros((K8, 256), dtype=torch.float16, device="cuda:0")
        a = torch.tensor(avals, dtype=torch.float64)
        b = torch.tensor(bvals, dtype=torch.float64)
        assert torch.equal(a.half().double(), a) and torch.equal(b.half().double(), b)   # exact in FP16
        A[0, :K] = a.half().cuda()
        B[:K, 0] = b.half().cuda()
        D = torch.full((128, 256), float("nan"), device="cuda:0")
        h.sgemm_cube_hgemm(A[:, :K], B[:K], D)
        st, det = h.sgemm_cube_check()
        assert st == 0, hex(det)
        assert torch.count_nonzero(D).item() <= 1
        return D[0, 0].item()

    yield run
    h.destroy()


def test_products_of_one_k16_group_are_summed_exactly_then_truncated(probe):
    # 1 + 15 * 2^-24 = 1 + 7.5 ulp: no intermediate rounding (fifteen separate roundings of
    # half an ulp would leave 1), one truncation at the end (7.5 -> 7)
    assert probe([1] + [E] * 15, [1] + [E] * 15) == 1.0 + 7 * ULP
    # 1 + 4 * 0.375 ulp = 1 + 1.5 ulp -> 1 + 1 ulp
    assert probe([1] + [0.75 * E] * 4, [1] + [E] * 4) == 1.0 + ULP


def test_truncation_is_toward_zero_for_both_signs(probe):
    assert probe([1, 1.5 * E], [1, E]) == 1.0           # 1 + 0.75 ulp: round-to-nearest would go up
    assert probe([-1, -1.5 * E], [1, E]) == -1.0         # -1 - 0.75 ulp: toward zero, not downward
    assert probe([1, E], [1, E]) == 1.0                  # the tie 1 + 0.5 ulp


def test_adding_a_group_to_the_accumulator_truncates_too(probe):
    z = [0] * 15
    assert probe([1] + z + [1.5 * E], [1] + z + [E]) == 1.0                  # + 0.75 ulp from the second group
    assert probe([1] + z + [3.5 * E], [1] + z + [E]) == 1.0 + ULP           # + 1.75 ulp -> + 1 ulp
    # sixteen groups each adding 0.75 ulp (12 ulp in exact arithmetic) leave the sum unchanged:
    # the bias of a long chain on one-signed data
    a = [1] + z + ([1.5 * E] + z) * 16
    b = [1] + z + ([E] + z) * 16
    assert probe(a, b) == 1.0


def test_small_addends_survive_cancellation_inside_a_group(probe):
    # 2^10 - 2^10 + 2^-14: the group is summed exactly, so the small product is not absorbed
    assert probe([2.0 ** 5, -2.0 ** 5, 2.0 ** -7], [2.0 ** 5, 2.0 ** 5, 2.0 ** -7]) == 2.0 ** -14
    # eight products of 2^-30 next to 1: below half an ulp in total, truncated away
    assert probe([1] + [2.0 ** -15] * 8, [1] + [2.0 ** -15] * 8) == 1.0


def test_fp16_subnormal_operands_are_honoured(probe):
    # the residual words rely on gradual underflow (Sec. 4.1): a subnormal FP16 operand must
    # enter the product with its value, not as zero
    assert probe([2.0 ** -24], [1.0]) == 2.0 ** -24
    assert probe([2.0 ** -24, 2.0 ** -20], [2.0 ** -24, 2.0 ** -24]) == 2.0 ** -48 + 2.0 ** -44
