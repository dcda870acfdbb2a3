"""Shared helpers of the GPU parity tests: gates and the oracle comparison on sampled rows."""
import numpy as np
import torch

import oracle
from paper_2507_23387_b200 import binding

U32 = 2.0 ** -24

# k-block lengths the library uses by default (include/sgemm_cube.h, SGEMM_CUBE_OPT_*); the
# oracle is run with the same block length so that both sides realise the same Eq. termwise /
# Eq. elementwise bracketing.
K_BLOCK = {binding.TERMWISE: 128, binding.ELEMENTWISE: 64, binding.ELEMENTWISE_REORDERED: 64}


def to_dev(x):
    return torch.from_numpy(np.ascontiguousarray(x)).to("cuda:0")


def padded_dev(x, mult):
    """Device copy whose leading dimension is a multiple of `mult` elements."""
    r, c = x.shape
    cp = (c + mult - 1) // mult * mult
    buf = torch.zeros((r, cp), dtype=torch.from_numpy(x[:1, :1]).dtype, device="cuda:0")
    view = buf[:, :c]
    view.copy_(torch.from_numpy(np.ascontiguousarray(x)))
    return view


def gates(C_gpu, A_rows, B, s, order, kb=None, label=""):
    """The three gates every CUDA result must pass on the rows it is checked on:
       (1) componentwise  |C - C64| <= 2 K 2^-24 (|A||B|)      (covers truncating accumulation;
           for K < 14 the representation error outweighs the accumulation error and the bound is
           the first-order form of Eq. main_bound, (K + 14) 2^-24, which equals 2 K 2^-24 at K = 14)
       (2) eta_gpu  <= 2 x eta_oracle,  (3) frob_gpu <= 2 x frob_oracle, the oracle run in the same
       order with the same k-block (the larger of that and the plain sequential sum, kb = K)."""
    K = A_rows.shape[1]
    kb = kb or K_BLOCK[order]
    C64, AB = oracle.dgemm_ref(A_rows, B)
    eta_g = oracle.componentwise_err(C_gpu, C64, AB)
    frob_g = oracle.frobenius_rel_err(C_gpu, C64)
    etas, frobs = [], []
    for okb in sorted({min(kb, K), K}):
        Co = oracle.sgemm_cube(A_rows, B, s=s, order=order, kb=okb)
        etas.append(oracle.componentwise_err(Co, C64, AB))
        frobs.append(oracle.frobenius_rel_err(Co, C64))
    msg = "%s eta_gpu=%.3e frob_gpu=%.3e oracle eta=%s frob=%s" % (label, eta_g, frob_g, etas, frobs)
    assert np.isfinite(C_gpu).all(), msg
    assert eta_g <= max(2 * K, K + 14) * U32, msg
    assert eta_g <= 2 * max(etas), msg
    assert frob_g <= 2 * max(frobs), msg
    return eta_g, frob_g
