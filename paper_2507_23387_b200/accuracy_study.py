"""Accuracy study of SGEMM-cube on the GPU, after the paper's Sec. 6.2 experiments.

Two sweeps, both with the paper's metric (Frobenius-norm relative error against an FP64 product,
Eq. err, mean over seeds):

  exponent sweep   entries U[-2^e, 2^e] (symmetric) or U[0, 2^e] (non-negative) for a range of
                   offset exponents e, scale exponents s_b in {0, 6, 11, 12}; compared methods:
                   termwise, elementwise and reordered-elementwise SGEMM-cube, the hi*hi product alone ("FP16 HGEMM"),
                   and an FP32 GEMM                                  (Fig. scaling_bit_error)
  size sweep       error against m = n, against k, and against all three, at offset exponent 0
                                                                      (Fig. mkn_error)
  dropped term     three-term SGEMM-cube against the four-term variant that keeps lo_A lo_B
                   (the term Eq. ll_bound bounds), against k
  adversarial      the max-norm study on constructed inputs that Sec. 6.2 and Sec. 7 name as
                   missing: products that cancel down to a fraction c of |A||B|, and entries whose
                   residuals all have the largest size and the same sign; reported is the largest
                   componentwise error max |C - C64| / (|A||B|) in units of u_32 = 2^-24 (the
                   quantity Eq. main_bound bounds) and the largest relative error of an entry

Everything runs through the library's C ABI (`sgemm_cube`, `sgemm_cube_split`,
`sgemm_cube_hgemm`, `sgemm_cube_four_term`); the FP64 reference and the FP32 baseline are torch matmuls on the device.
Run as a script for a markdown report:

    python -m paper_2507_23387_b200.accuracy_study [--size 1024] [--seeds 5] [--quick]
"""
import argparse
import json

import torch

from . import binding, inputs


def frobenius_rel_err(C, C64):
    d = C.double() - C64
    return float(d.norm() / C64.norm())


def _reference(A, B):
    return A.double() @ B.double()


def _fp32_gemm(A, B):
    prev = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = False
    try:
        return A @ B
    finally:
        torch.backends.cuda.matmul.allow_tf32 = prev


def _hgemm_hi_only(h, A, B, s):
    """hi_A * hi_B alone: what a native FP16 GEMM with FP32 accumulation computes."""
    M, K = A.shape
    _, N = B.shape
    f16 = dict(dtype=torch.float16, device=A.device)
    Ahi, Alo = torch.empty((M, K), **f16), torch.empty((M, K), **f16)
    Bhi, Blo = torch.empty((K, N), **f16), torch.empty((K, N), **f16)
    h.sgemm_cube_split(A, Ahi, Alo, s)
    h.sgemm_cube_split(B, Bhi, Blo, s)
    D = torch.empty((M, N), device=A.device)
    h.sgemm_cube_hgemm(Ahi, Bhi, D)
    return D


def measure(h, A, B, scale_exps=(0, 6, 11, 12)):
    """Errors of every method on one (A, B) pair; keys like 'termwise_s12'."""
    C64 = _reference(A, B)
    M, N = A.shape[0], B.shape[1]
    out = {"fp32_gemm": frobenius_rel_err(_fp32_gemm(A, B), C64),
           "fp16_hgemm": frobenius_rel_err(_hgemm_hi_only(h, A, B, 0), C64)}
    C = torch.empty((M, N), device=A.device)
    for s in scale_exps:
        for name, order in (("termwise", binding.TERMWISE), ("elementwise", binding.ELEMENTWISE),
                            ("reordered", binding.ELEMENTWISE_REORDERED)):
            h.sgemm_cube(A, B, C, s, order)
            out["%s_s%d" % (name, s)] = frobenius_rel_err(C, C64)
        h.sgemm_cube_four_term(A, B, C, s)
        out["four_term_s%d" % s] = frobenius_rel_err(C, C64)
    status, detail = h.sgemm_cube_check()
    if status != 0:
        raise RuntimeError("device error %s" % hex(detail))
    return out


def _mean_over_seeds(h, make, seeds, scale_exps):
    acc = {}
    for seed in range(seeds):
        A, B = make(seed)
        for k, v in measure(h, A, B, scale_exps).items():
            acc[k] = acc.get(k, 0.0) + v / seeds
    return acc


def exponent_sweep(h, size=1024, exponents=range(-14, 3, 2), seeds=5, nonneg=False,
                   scale_exps=(0, 6, 11, 12), device="cuda:0"):
    """Error against the offset exponent e of the inputs (Fig. scaling_bit_error (a) / (b))."""
    rows = []
    for e in exponents:
        def make(seed, e=e):
            A = torch.from_numpy(inputs.uniform_range(seed, (size, size), e, nonneg, stream=0)).to(device)
            B = torch.from_numpy(inputs.uniform_range(seed, (size, size), e, nonneg, stream=1)).to(device)
            return A, B
        r = _mean_over_seeds(h, make, seeds, scale_exps)
        r["offset_exponent"] = e
        rows.append(r)
    return rows


def size_sweep(h, shapes, seeds=5, scale_exp=12, device="cuda:0"):
    """Error against the matrix sizes at offset exponent 0 (Fig. mkn_error)."""
    rows = []
    for (M, N, K) in shapes:
        def make(seed, M=M, N=N, K=K):
            A = torch.from_numpy(inputs.uniform_range(seed, (M, K), 0, False, stream=0)).to(device)
            B = torch.from_numpy(inputs.uniform_range(seed, (K, N), 0, False, stream=1)).to(device)
            return A, B
        r = _mean_over_seeds(h, make, seeds, (scale_exp,))
        r["shape"] = (M, N, K)
        rows.append(r)
    return rows


def dropped_term_sweep(h, ks=(8, 32, 128, 512, 2048, 8192), mn=1024, seeds=5, scale_exp=11,
                       device="cuda:0"):
    """Three-term against four-term error over the inner dimension (symmetric U[-1, 1) inputs):
    Frobenius error as elsewhere, plus the largest componentwise error
    max |C - C64| / (|A||B|) (the quantity Eq. main_bound and Eq. ll_bound are stated in)."""
    rows = []
    C = torch.empty((mn, mn), device=device)
    for K in ks:
        r = {"k": K, "three_term_frob": 0.0, "four_term_frob": 0.0, "three_term_cw": 0.0,
             "four_term_cw": 0.0}
        for seed in range(seeds):
            A = torch.from_numpy(inputs.uniform_range(seed, (mn, K), 0, False, stream=0)).to(device)
            B = torch.from_numpy(inputs.uniform_range(seed, (K, mn), 0, False, stream=1)).to(device)
            C64 = _reference(A, B)
            AB = A.double().abs() @ B.double().abs()
            for name, call in (("three_term", lambda: h.sgemm_cube(A, B, C, scale_exp, binding.TERMWISE)),
                               ("four_term", lambda: h.sgemm_cube_four_term(A, B, C, scale_exp))):
                call()
                r[name + "_frob"] += frobenius_rel_err(C, C64) / seeds
                r[name + "_cw"] = max(r[name + "_cw"], float(((C.double() - C64).abs() / AB).max()))
        rows.append(r)
    status, detail = h.sgemm_cube_check()
    if status != 0:
        raise RuntimeError("device error %s" % hex(detail))
    return rows


def adversarial_sweep(h, mn=1024, seeds=3, scale_exp=11, device="cuda:0",
                      cancellations=(1.0, 2.0 ** -6, 2.0 ** -12, 2.0 ** -18), k_cancel=1024,
                      ks_coherent=(16, 256, 4096)):
    """Constructed inputs (inputs.cancellation_pair, inputs.coherent_residuals).  Per case and
    method: eta = max |C - C64| / (|A||B|) in units of 2^-24 over all seeds, and the largest
    relative error of an entry (cancellation cases)."""
    methods = (("termwise", lambda A, B, C: h.sgemm_cube(A, B, C, scale_exp, binding.TERMWISE)),
               ("elementwise", lambda A, B, C: h.sgemm_cube(A, B, C, scale_exp, binding.ELEMENTWISE)),
               ("four_term", lambda A, B, C: h.sgemm_cube_four_term(A, B, C, scale_exp)),
               ("fp32_gemm", lambda A, B, C: C.copy_(_fp32_gemm(A, B))))
    cases = [("cancel c=2^%d" % round(torch.log2(torch.tensor(c)).item()), k_cancel,
              lambda seed, c=c: inputs.cancellation_pair(seed, mn, mn, k_cancel, c)) for c in cancellations]
    cases += [("coherent residuals k=%d" % k, k,
               lambda seed, k=k: (inputs.coherent_residuals(seed, (mn, k), 0),
                                  inputs.coherent_residuals(seed, (k, mn), 1))) for k in ks_coherent]
    rows = []
    C = torch.empty((mn, mn), device=device)
    for name, K, make in cases:
        r = {"case": name, "k": K, "bound_first_order": float(K + 14)}
        for seed in range(seeds):
            A, B = (torch.from_numpy(x).to(device) for x in make(seed))
            C64 = _reference(A, B)
            AB = A.double().abs() @ B.double().abs()
            for mname, call in methods:
                call(A, B, C)
                err = (C.double() - C64).abs()
                r[mname + "_eta"] = max(r.get(mname + "_eta", 0.0), float((err / AB).max()) * 2.0 ** 24)
                rel = float((err / C64.abs().clamp_min(1e-300)).max())
                r[mname + "_maxrel"] = max(r.get(mname + "_maxrel", 0.0), rel)
        rows.append(r)
    status, detail = h.sgemm_cube_check()
    if status != 0:
        raise RuntimeError("device error %s" % hex(detail))
    return rows


def config_errors(h, device="cuda:0", rows_sampled=512):
    """Errors at the benchmark configurations (sizes and input distributions of the build's five
    workloads), both accumulation orders, against an FP64 product on `rows_sampled` rows:
    Frobenius relative error and the largest componentwise error in units of 2^-24."""
    configs = [("256^3 U[-1,1)", "uniform_pm1", 256, 256, 256),
               ("4096^3 U[-1,1)", "uniform_pm1", 4096, 4096, 4096),
               ("8192^3 exponent spread", "exponent_spread", 8192, 8192, 8192),
               ("1024 x 1024 x 65536 N(0,1)", "normal", 1024, 1024, 65536),
               ("2048^3 N(0,1)", "normal", 2048, 2048, 2048),
               ("16384 x 16384 x 1024 N(0,1)", "normal", 16384, 16384, 1024)]
    rows = []
    for name, kind, M, N, K in configs:
        A_h, B_h = inputs.make_pair(kind, 0, M, N, K)
        A, B = torch.from_numpy(A_h).to(device), torch.from_numpy(B_h).to(device)
        del A_h, B_h
        C = torch.empty((M, N), device=device)
        idx = torch.arange(0, M, max(M // rows_sampled, 1), device=device)[:rows_sampled]
        A64 = A[idx].double()
        B64 = B.double()
        C64 = A64 @ B64
        AB = A64.abs() @ B64.abs()
        del B64
        r = {"config": name, "gate_2k": 2.0 * K}
        for oname, order in (("termwise", binding.TERMWISE), ("elementwise", binding.ELEMENTWISE),
                             ("reordered", binding.ELEMENTWISE_REORDERED)):
            h.sgemm_cube(A, B, C, 11, order)
            d = (C[idx].double() - C64).abs()
            r[oname + "_frob"] = float(d.norm() / C64.norm())
            r[oname + "_eta_u32"] = float((d / AB).max()) * 2.0 ** 24
        d = (_fp32_gemm(A, B)[idx].double() - C64).abs()
        r["fp32_gemm_frob"] = float(d.norm() / C64.norm())
        r["fp32_gemm_eta_u32"] = float((d / AB).max()) * 2.0 ** 24
        rows.append(r)
        del A, B, C, A64, C64, AB, d
    status, detail = h.sgemm_cube_check()
    if status != 0:
        raise RuntimeError("device error %s" % hex(detail))
    return rows


def _table(rows, key, cols):
    lines = ["| %s | %s |" % (key, " | ".join(cols)), "|" + "---|" * (len(cols) + 1)]
    for r in rows:
        lines.append("| %s | %s |" % (r[key], " | ".join("%.2e" % r[c] for c in cols)))
    return "\n".join(lines)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--size", type=int, default=1024)
    ap.add_argument("--seeds", type=int, default=5)
    ap.add_argument("--quick", action="store_true")
    ap.add_argument("--json", action="store_true")
    ap.add_argument("--configs", action="store_true",
                    help="only the error table at the benchmark configurations")
    args = ap.parse_args()
    h = binding.Handle(0)
    if args.configs:
        rows = config_errors(h)
        h.destroy()
        print("## Errors at the benchmark configurations (s_b = 11, default k-blocks), against FP64 on "
              "512 sampled rows\n")
        print(_table(rows, "config", ["gate_2k", "termwise_frob", "elementwise_frob", "reordered_frob",
                                      "fp32_gemm_frob", "termwise_eta_u32", "elementwise_eta_u32",
                                      "reordered_eta_u32", "fp32_gemm_eta_u32"]))
        return
    exps = range(-12, 3, 4) if args.quick else range(-16, 5, 2)
    cols = ["fp16_hgemm", "fp32_gemm", "termwise_s0", "elementwise_s0", "termwise_s6", "termwise_s11",
            "termwise_s12", "elementwise_s12", "reordered_s12"]
    sym = exponent_sweep(h, args.size, exps, args.seeds, nonneg=False)
    pos = exponent_sweep(h, args.size, exps, args.seeds, nonneg=True)
    k_fixed = 64 * 44
    mn = [(n, n, k_fixed) for n in ((512, 2048) if args.quick else (256, 1024, 4096))]
    ks = [(1024, 1024, k) for k in ((256, 4096) if args.quick else (256, 1024, 4096, 16384, 65536))]
    alls = [(n, n, n) for n in ((512, 2048) if args.quick else (512, 1024, 2048, 4096))]
    scol = ["fp16_hgemm", "fp32_gemm", "termwise_s12", "elementwise_s12", "reordered_s12"]
    res = {"symmetric": sym, "nonnegative": pos, "vs_mn": size_sweep(h, mn, args.seeds),
           "vs_k": size_sweep(h, ks, args.seeds), "vs_all": size_sweep(h, alls, args.seeds),
           "dropped_term": dropped_term_sweep(h, (8, 512) if args.quick else (8, 32, 128, 512, 2048, 8192),
                                              seeds=args.seeds),
           "adversarial": adversarial_sweep(h, 512 if args.quick else 1024, 1 if args.quick else 3)}
    h.destroy()
    if args.json:
        print(json.dumps(res))
        return
    print("## Relative error vs offset exponent, U[-2^e, 2^e], %d^3, %d seeds\n" % (args.size, args.seeds))
    print(_table(sym, "offset_exponent", cols))
    print("\n## Relative error vs offset exponent, U[0, 2^e]\n")
    print(_table(pos, "offset_exponent", cols))
    print("\n## Relative error vs m = n (k = %d), offset exponent 0, s_b = 12\n" % k_fixed)
    print(_table(res["vs_mn"], "shape", scol))
    print("\n## Relative error vs k (m = n = 1024)\n")
    print(_table(res["vs_k"], "shape", scol))
    print("\n## Relative error vs m = n = k\n")
    print(_table(res["vs_all"], "shape", scol))
    print("\n## Three-term against four-term (low-low product kept), m = n = 1024, U[-1, 1), s_b = 11\n")
    print(_table(res["dropped_term"], "k", ["three_term_frob", "four_term_frob", "three_term_cw",
                                            "four_term_cw"]))
    print("\n## Constructed inputs: largest componentwise error in units of 2^-24 "
          "(first-order form of Eq. main_bound: k + 14), m = n = 1024, s_b = 11\n")
    print(_table(res["adversarial"], "case", ["bound_first_order", "termwise_eta", "elementwise_eta",
                                              "four_term_eta", "fp32_gemm_eta"]))
    print("\n## Constructed inputs: largest relative error of an entry\n")
    print(_table(res["adversarial"], "case", ["termwise_maxrel", "elementwise_maxrel", "four_term_maxrel",
                                              "fp32_gemm_maxrel"]))


if __name__ == "__main__":
    main()
