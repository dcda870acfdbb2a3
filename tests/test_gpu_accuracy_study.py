"""GPU test of the accuracy-study harness (the paper's Sec. 6.2 experiments at reduced size):
the qualitative findings the paper reports must reproduce, and the harness's own error numbers
must agree with errors computed against the oracle's FP64 reference."""
import numpy as np
import pytest
import torch

import oracle
from paper_2507_23387_b200 import accuracy_study, binding, inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def handle():
    h = binding.Handle(0)
    yield h
    h.destroy()


def test_exponent_sweep_reproduces_the_papers_findings(handle):
    rows = {r["offset_exponent"]: r for r in
            accuracy_study.exponent_sweep(handle, size=512, exponents=(-12, -8, 0), seeds=2)}
    for e in (-8, 0):
        assert 3e-5 < rows[e]["fp16_hgemm"] < 1e-3            # "FP16 HGEMM ... ~1e-4"
    for e in (-12, -8):
        # residual amplification is needed: s_b = 0 trails FP32, s_b = 12 gains 1-2 orders
        assert rows[e]["termwise_s0"] > 3 * rows[e]["fp32_gemm"]
        assert rows[e]["termwise_s12"] < rows[e]["termwise_s0"] / 10
    assert rows[-12]["termwise_s6"] > 3 * rows[-12]["termwise_s12"]     # "s_b = 6 is insufficient"
    for e in (-12, -8, 0):
        assert rows[e]["termwise_s12"] < 2 * rows[e]["fp32_gemm"]       # comparable to FP32 SGEMM
        assert rows[e]["elementwise_s12"] < 2 * rows[e]["fp32_gemm"]
        assert abs(rows[e]["termwise_s11"] / rows[e]["termwise_s12"] - 1) < 0.5


def test_nonnegative_inputs(handle):
    sym = accuracy_study.exponent_sweep(handle, size=512, exponents=(0,), seeds=2, nonneg=False)[0]
    pos = accuracy_study.exponent_sweep(handle, size=512, exponents=(0,), seeds=2, nonneg=True)[0]
    # Sec. 6.2: with symmetric sampling cancellation depresses ||C_true|| and inflates the relative
    # error; without it the FP16 product alone is an order of magnitude better
    assert pos["fp16_hgemm"] < sym["fp16_hgemm"] / 5
    # one-signed data is the worst case for the tensor core's truncating accumulation (its bias
    # adds up along a k-block): still within a small factor of an FP32 GEMM
    assert pos["termwise_s12"] < 2.5 * pos["fp32_gemm"]
    assert pos["elementwise_s12"] < 2.5 * pos["fp32_gemm"]


def test_error_depends_on_k_not_on_m_n(handle):
    mn = accuracy_study.size_sweep(handle, [(256, 256, 2816), (1024, 1024, 2816)], seeds=2)
    assert 0.5 < mn[0]["termwise_s12"] / mn[1]["termwise_s12"] < 2.0
    ks = accuracy_study.size_sweep(handle, [(512, 512, 256), (512, 512, 16384)], seeds=2)
    assert ks[1]["fp32_gemm"] > 1.5 * ks[0]["fp32_gemm"]      # plain FP32 grows with k
    assert ks[1]["termwise_s12"] < ks[1]["fp32_gemm"]         # termwise stays below it at long k


def test_harness_errors_agree_with_the_oracle_reference(handle):
    A = inputs.uniform_range(3, (256, 384), -4, False, stream=0)
    B = inputs.uniform_range(3, (384, 320), -4, False, stream=1)
    got = accuracy_study.measure(handle, torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), (12,))
    C64 = oracle.dgemm_ref(A, B, with_abs=False)
    C = torch.empty((256, 320), device="cuda:0")
    handle.sgemm_cube(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), C, 12, binding.TERMWISE)
    want = oracle.frobenius_rel_err(C.cpu().numpy(), C64)
    assert abs(got["termwise_s12"] / want - 1) < 1e-3
    want_f32 = oracle.frobenius_rel_err(oracle.sgemm_f32(A, B), C64)
    assert 0.2 < got["fp32_gemm"] / want_f32 < 5


def test_dropped_term_sweep(handle):
    # The low-low product has leading coefficient 2^-22 (Eq. ll_bound): keeping it helps only
    # while the FP32 accumulation error (which grows with k) is smaller than that.
    rows = {r["k"]: r for r in accuracy_study.dropped_term_sweep(handle, ks=(8, 2048), mn=512, seeds=2)}
    assert rows[8]["four_term_frob"] < 0.95 * rows[8]["three_term_frob"]
    assert 0.8 < rows[2048]["four_term_frob"] / rows[2048]["three_term_frob"] < 1.05
    for r in rows.values():
        assert r["four_term_cw"] <= 2 * r["k"] * 2.0 ** -24 and r["three_term_cw"] <= 2 * r["k"] * 2.0 ** -24


def test_adversarial_sweep_stays_inside_the_componentwise_bound(handle):
    rows = accuracy_study.adversarial_sweep(handle, mn=256, seeds=1, cancellations=(1.0, 2.0 ** -12),
                                            k_cancel=512, ks_coherent=(16, 512))
    by = {r["case"]: r for r in rows}
    for r in rows:
        # truncating accumulation doubles the unit roundoff of the k additions (the test gate)
        for m in ("termwise", "elementwise", "four_term"):
            assert r[m + "_eta"] <= max(2 * r["k"], r["k"] + 14), (r["case"], m, r[m + "_eta"])
    # cancellation leaves the componentwise error alone and ruins the relative error of entries
    assert by["cancel c=2^-12"]["termwise_eta"] < 4 * by["cancel c=2^0"]["termwise_eta"] + 2
    assert by["cancel c=2^-12"]["termwise_maxrel"] > 50 * by["cancel c=2^0"]["termwise_maxrel"]
    # coherent residuals: the dropped term shows in full (about 2^-22 = 4 u_32 / 1.05^2), the
    # four-term variant removes it
    r = by["coherent residuals k=16"]
    assert r["termwise_eta"] - r["four_term_eta"] > 2.0


def test_harness_componentwise_errors_agree_with_the_oracle_helpers(handle):
    """The adversarial sweep reports max |C - C64| / (|A||B|) computed with torch FP64 products on the
    device; the same quantity from the oracle's FP64 reference and its (hand-pinned)
    componentwise_err on the same inputs must agree, so the harness's tables are tied to the oracle."""
    mn, K = 128, 256
    rows = accuracy_study.adversarial_sweep(handle, mn=mn, seeds=1, cancellations=(2.0 ** -6,),
                                            k_cancel=K, ks_coherent=(64,))
    by = {r["case"]: r for r in rows}
    cases = {"cancel c=2^-6": inputs.cancellation_pair(0, mn, mn, K, 2.0 ** -6),
             "coherent residuals k=64": (inputs.coherent_residuals(0, (mn, 64), 0),
                                         inputs.coherent_residuals(0, (64, mn), 1))}
    for name, (A, B) in cases.items():
        C64, AB = oracle.dgemm_ref(A, B)
        C = torch.empty((mn, mn), device="cuda:0")
        for mname, order in (("termwise", binding.TERMWISE), ("elementwise", binding.ELEMENTWISE)):
            handle.sgemm_cube(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), C, 11, order)
            want = oracle.componentwise_err(C.cpu().numpy(), C64, AB) * 2.0 ** 24
            got = by[name][mname + "_eta"]
            assert abs(got - want) <= 1e-6 * max(want, 1.0), (name, mname, got, want)
