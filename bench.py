#!/usr/bin/env python
"""Benchmark of the SGEMM-cube hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" is one pass of the whole hot path over one batch of synthetic input: a single call of
the `sgemm_cube` entry point with its default options (operand split, three FP16 tensor-core
products and the FP32 reconstruction; at this size the library splits both operands once with the
split kernel and forms the products in one tensor-core kernel: two launches per step) on
M = N = K = 8192 FP32 matrices whose entries are
(+/-) u * 2^e, u uniform in [1, 2), e a uniform integer in [-10, 10], with s = 11 and termwise
accumulation.  The metric is FP32-equivalent TFLOP/s = 2 M N K / t.

Prints ONE JSON line (rank 0).  `value` is measured with the operands resident in device memory;
`e2e` through the host-buffer entry point with both copies inside the timed region; `roofline`
compares the kernel's 3 x 2MNK FP16 tensor-core FLOPs per launch with the measured dense
tensor-core peak; `cpu_baseline` is the CPU oracle timed on a bounded sample of the same
workload.  With --impl reference the oracle itself is the timed arm.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

M = N = K = 8192
SCALE_EXP = 11
WORKLOAD = "M=N=K=8192 FP32 GEMM, entries (+/-)u*2^e, u~U[1,2), e~U{-10..10}, s=11, termwise"
METRIC = "FP32-equiv TFLOP/s (2MNK/t) at 8192^3"
UNIT = "TFLOP/s"

# DRAM traffic of one launch of the dominant kernel (the three-product tensor-core kernel) at this
# workload: dram__bytes_read.sum + dram__bytes_write.sum of the full-size one-pass ncu capture
# summarised in profiles/three_product_kernel_8192_cubed.md.
KERNEL_DRAM_BYTES_PER_LAUNCH = 3102864640 + 259538944


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "hbm_gbs": float(d["hbm_gbs"]), "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0,
            "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.samples = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) >= 6:
                self.samples.append((time.perf_counter(), parts))

    def stop(self, t_begin=None, t_end=None):
        """Summary of the samples taken in [t_begin, t_end] (all samples if that window is empty)."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        inside = [v for (t, v) in self.samples
                  if t_begin is not None and t_begin <= t <= t_end + 0.05]
        window = "timed region"
        if not inside:
            inside = [v for (_, v) in self.samples]
            window = "warm-up and timed region"
        for s in inside:
            try:
                sm.append(float(s[0]))
                mx.append(float(s[1]))
            except ValueError:
                continue
            for name, v in zip(names, s[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons),
                "samples": len(sm), "window": window}


def max_over_ranks(x, world, device):
    """Max of a per-rank scalar over all ranks (the job is as slow as its slowest rank)."""
    if world <= 1:
        return float(x)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(x)], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(flops_per_rank_step, ms_per_step, world):
    """Whole-job FP32-equivalent TFLOP/s: every rank runs one full problem per step (independent
    replicas, weak scaling), and the step time is the max over ranks."""
    return world * flops_per_rank_step / (ms_per_step * 1e-3) / 1e12


def cpu_oracle_sample(rows):
    """Time the oracle (as it stands) on `rows` rows of the workload; returns (TFLOP/s, s, threads)."""
    import oracle
    from paper_2507_23387_b200 import inputs
    A = inputs.exponent_spread(0, (rows, K), stream=0)
    B = inputs.exponent_spread(0, (K, N), stream=1)
    oracle.sgemm_cube(A[:1], B[:, :8].copy(), SCALE_EXP, oracle.TERMWISE, 64)      # load the library
    t0 = time.perf_counter()
    oracle.sgemm_cube(A, B, SCALE_EXP, oracle.TERMWISE, 64)
    dt = time.perf_counter() - t0
    return 2.0 * rows * N * K / dt / 1e12, dt, oracle.num_threads()


def run_reference(args, rank):
    """The reference arm: the CPU oracle, timed on a bounded sample per step."""
    if rank != 0:
        return
    import oracle
    from paper_2507_23387_b200 import inputs
    rows = args.cpu_rows                  # the same sample as the cpu_baseline leg of the other arm
    A = inputs.exponent_spread(0, (rows, K), stream=0)
    B = inputs.exponent_spread(0, (K, N), stream=1)
    for _ in range(max(1, min(args.warmup, 1))):
        oracle.sgemm_cube(A[:8], B, SCALE_EXP, oracle.TERMWISE, 64)
    steps = max(1, min(args.steps, 3))
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.sgemm_cube(A, B, SCALE_EXP, oracle.TERMWISE, 64)
    dt = (time.perf_counter() - t0) / steps
    val = 2.0 * rows * N * K / dt / 1e12
    sample = "%d of %d rows of A against the full B (split of B included), per step" % (rows, M)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-rows", type=int, default=2048)
    ap.add_argument("--sustained-seconds", type=float, default=3.0)
    ap.add_argument("--size", type=int, default=8192,
                    help="M = N = K; values other than 8192 are for profiler captures only")
    ap.add_argument("--strategy", default="auto", choices=["auto", "fused", "two_phase"],
                    help="SGEMM_CUBE_OPT_STRATEGY for sgemm_cube (the bench value uses auto)")
    ap.add_argument("--entry", default="sgemm_cube", choices=["sgemm_cube", "presplit", "unfused"],
                    help="entry point timed as the step (profiler captures; the bench value is sgemm_cube)")
    ap.add_argument("--kernel-only", action="store_true",
                    help="skip the ablation, end-to-end and CPU legs (profiler captures)")
    args = ap.parse_args()
    global M, N, K, WORKLOAD
    if args.size != 8192:
        M = N = K = args.size
        WORKLOAD = WORKLOAD.replace("8192", str(args.size)) + " (reduced size: not a bench value)"

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    from paper_2507_23387_b200 import binding, inputs

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = "cuda:%d" % local_rank
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device(dev))

    h = binding.Handle(local_rank)
    strategies = {"auto": binding.STRATEGY_AUTO, "fused": binding.STRATEGY_FUSED,
                  "two_phase": binding.STRATEGY_TWO_PHASE}
    h.sgemm_cube_set_option(binding.OPT_STRATEGY, strategies[args.strategy])
    h.sgemm_cube_set_option(binding.OPT_TIME_KERNEL, 1)
    # Same seeded workload on every rank (independent replicas of the problem: weak scaling).
    A_host = torch.from_numpy(inputs.exponent_spread(0, (M, K), stream=0))
    B_host = torch.from_numpy(inputs.exponent_spread(0, (K, N), stream=1))
    A, B = A_host.to(dev), B_host.to(dev)
    C = torch.empty((M, N), device=dev)
    warmup = max(3, args.warmup)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    if args.entry == "presplit":
        f16 = dict(dtype=torch.float16, device=dev)
        pAhi, pAlo = torch.empty((M, K), **f16), torch.empty((M, K), **f16)
        pBhi, pBlo = torch.empty((K, N), **f16), torch.empty((K, N), **f16)
        h.sgemm_cube_split(A, pAhi, pAlo, SCALE_EXP)
        h.sgemm_cube_split(B, pBhi, pBlo, SCALE_EXP)

        def step():
            h.sgemm_cube_presplit(pAhi, pAlo, pBhi, pBlo, C, SCALE_EXP, binding.TERMWISE)
    elif args.entry == "unfused":
        def step():
            h.sgemm_cube_unfused(A, B, C, SCALE_EXP, binding.TERMWISE)
    else:
        def step():
            h.sgemm_cube(A, B, C, SCALE_EXP, binding.TERMWISE)

    sampler = ClockSampler(local_rank)
    sampler.start()
    t_warm = time.perf_counter()
    for _ in range(warmup):
        step()
    barrier()
    # keep the device busy until nvidia-smi delivers (its first sample takes a few 100 ms), so that
    # the timed region starts from a loaded, sampled state
    while not sampler.samples and time.perf_counter() - t_warm < 2.0:
        step()
        torch.cuda.synchronize()
    launches0 = h.sgemm_cube_launch_count()
    if args.entry == "sgemm_cube":
        h.sgemm_cube_mean_kernel_ms()          # start a new average at the timed region
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    barrier()
    t_begin = time.perf_counter()
    ev[0].record()
    for i in range(args.steps):
        step()
        ev[i + 1].record()
    barrier()
    total_ms = ev[0].elapsed_time(ev[-1])
    clocks = sampler.stop(t_begin, time.perf_counter())
    launches = h.sgemm_cube_launch_count() - launches0
    st, det = h.sgemm_cube_check()
    if st != 0:
        raise SystemExit("device error %s" % hex(det))
    # Device time of the dominant (tensor-core) kernel: the library records a CUDA event pair
    # around that launch on the launching stream in every sgemm_cube call; the mean over the calls
    # of the timed region (the most recent 128 at most) is read here.
    kernel_samples = []
    kernel_clock = None
    if args.entry == "sgemm_cube":
        kernel_samples.append(h.sgemm_cube_mean_kernel_ms()[0])
        kernel_clock = h.sgemm_cube_last_kernel_clock()      # (SM cycles, ns) of the last timed launch
    else:
        kernel_samples = [ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps)]
    total_ms = max_over_ranks(total_ms, world, dev)
    ms_per_step = total_ms / args.steps
    flops = 2.0 * M * N * K
    value = job_throughput(flops, ms_per_step, world)

    sm_count = torch.cuda.get_device_properties(local_rank).multi_processor_count

    def clock_fracs(tflops_fp32_equiv, kclock):
        """Three-GEMM roofline at the SM clock the kernel itself measured: SMs x 8192 dense FP16
        flop/clk/SM x (cycles / ns) / 3."""
        if not kclock or not kclock[1]:
            return {}
        ghz = kclock[0] / kclock[1]
        peak3 = sm_count * 8192 * ghz * 1e9 / 1e12 / 3.0
        return {"sm_mhz_in_kernel": ghz * 1e3, "kernel_cycles": int(kclock[0]),
                "fp32_equiv_peak_at_kernel_clock": peak3,
                "frac_at_kernel_clock": tflops_fp32_equiv / peak3}

    def sustained_run(seconds, label):
        """Back-to-back steps for at least `seconds`, with their own clock samples."""
        smp = ClockSampler(local_rank)
        smp.start()
        s_ev, e_ev = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        s_ev.record()
        n = 0
        while True:
            for _ in range(20):
                step()
            n += 20
            torch.cuda.synchronize()
            if time.perf_counter() - t0 >= seconds:
                break
        e_ev.record()
        torch.cuda.synchronize()
        t1 = time.perf_counter()
        ms = s_ev.elapsed_time(e_ev) / n
        kc = h.sgemm_cube_last_kernel_clock() if args.entry == "sgemm_cube" else None
        tf = flops / ms / 1e9
        out = {"what": label, "seconds": t1 - t0, "steps": n, "ms_per_step": ms, "tflops": tf,
               "clocks": smp.stop(t0, t1)}
        out.update(clock_fracs(tf, kc))
        return out

    sustained = fused_block = None
    if rank == 0 and not args.kernel_only:
        sustained = sustained_run(args.sustained_seconds, "default strategy, steps back to back after the timed region")
        if args.strategy != "fused" and args.entry == "sgemm_cube":
            # The fused kernel (no FP16 copy of A or B in device memory) as a measurement of its own.
            h.sgemm_cube_set_option(binding.OPT_STRATEGY, binding.STRATEGY_FUSED)
            for _ in range(3):
                step()
            torch.cuda.synchronize()
            h.sgemm_cube_mean_kernel_ms()
            fe = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
            nf = max(10, min(args.steps, 50))
            fe[0].record()
            for _ in range(nf):
                step()
            fe[1].record()
            torch.cuda.synchronize()
            f_ms = fe[0].elapsed_time(fe[1]) / nf
            f_kms = h.sgemm_cube_mean_kernel_ms()[0]
            f_kc = h.sgemm_cube_last_kernel_clock()
            f_tf = flops / f_ms / 1e9
            f_peaks = measured_peaks()
            fused_block = {"what": "sgemm_cube, strategy fused: one kernel per step, %d steps" % nf,
                           "tflops": f_tf, "ms_per_step": f_ms, "kernel_ms": f_kms,
                           "fp16_tflops": 3.0 * flops / f_kms / 1e9,
                           "frac_of_measured_burst": 3.0 * flops / f_kms / 1e9 / f_peaks["bf16_tflops"],
                           "frac_of_max_clock_three_gemm_roofline": f_tf / (sm_count * 8192 * 1.965e9 / 1e12 / 3.0)}
            fused_block.update(clock_fracs(f_tf, f_kc))
            fused_block["sustained"] = sustained_run(args.sustained_seconds, "fused strategy, steps back to back")
            h.sgemm_cube_set_option(binding.OPT_STRATEGY, strategies[args.strategy])

    # Ablation legs on rank 0 (not part of `value`): pre-split kernel, unfused path, split alone.
    extra = {}
    if rank == 0 and not args.kernel_only:
        def timed(fn, n=5):
            fn()
            torch.cuda.synchronize()
            s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s.record()
            for _ in range(n):
                fn()
            e.record()
            torch.cuda.synchronize()
            return s.elapsed_time(e) / n
        f16 = dict(dtype=torch.float16, device=dev)
        Ahi, Alo = torch.empty((M, K), **f16), torch.empty((M, K), **f16)
        Bhi, Blo = torch.empty((K, N), **f16), torch.empty((K, N), **f16)
        t_split = timed(lambda: h.sgemm_cube_split(A, Ahi, Alo, SCALE_EXP))
        h.sgemm_cube_split(B, Bhi, Blo, SCALE_EXP)
        t_pre = timed(lambda: h.sgemm_cube_presplit(Ahi, Alo, Bhi, Blo, C, SCALE_EXP, binding.TERMWISE))
        t_unf = timed(lambda: h.sgemm_cube_unfused(A, B, C, SCALE_EXP, binding.TERMWISE))
        t_ele = timed(lambda: h.sgemm_cube(A, B, C, SCALE_EXP, binding.ELEMENTWISE))
        t_reo = timed(lambda: h.sgemm_cube(A, B, C, SCALE_EXP, binding.ELEMENTWISE_REORDERED))
        t_four = timed(lambda: h.sgemm_cube_four_term(A, B, C, SCALE_EXP))
        if fused_block is not None:
            t_fus = fused_block["ms_per_step"]            # the `fused` block's own timed run
        else:
            h.sgemm_cube_set_option(binding.OPT_STRATEGY, binding.STRATEGY_FUSED)
            t_fus = timed(lambda: h.sgemm_cube(A, B, C, SCALE_EXP, binding.TERMWISE), 10)
            h.sgemm_cube_set_option(binding.OPT_STRATEGY, strategies[args.strategy])
        extra = {"three_product_kernel_alone_tflops": flops / t_pre / 1e9,
                 "unfused_split_3gemm_tflops": flops / t_unf / 1e9,
                 "elementwise_order_tflops": flops / t_ele / 1e9,
                 "reordered_elementwise_order_tflops": flops / t_reo / 1e9,
                 "four_term_variant_tflops": flops / t_four / 1e9,
                 "fused_converter_kernel_tflops": flops / t_fus / 1e9,
                 "split_kernel_gbs": 8.0 * M * K / t_split / 1e6}
        del Ahi, Alo, Bhi, Blo

    if args.kernel_only:
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
                              "steps": args.steps, "ms_per_step": ms_per_step,
                              "config": {"workload": WORKLOAD, "entry": args.entry}, "kernel_only": True,
                              "gpu_launches": int(launches)}))
        h.destroy()
        if world > 1:
            dist.destroy_process_group()
        return

    # End to end through the host-buffer entry point: H2D of A and B, kernel, D2H of C per step.
    A_pin, B_pin = A_host.pin_memory(), B_host.pin_memory()
    C_pin = torch.empty((M, N)).pin_memory()
    h.sgemm_cube_host(A_pin, B_pin, C_pin, SCALE_EXP, binding.TERMWISE)
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.e2e_steps):
        h.sgemm_cube_host(A_pin, B_pin, C_pin, SCALE_EXP, binding.TERMWISE)
    barrier()
    e2e_ms = max_over_ranks((time.perf_counter() - t0) / args.e2e_steps * 1e3, world, dev)
    e2e_val = job_throughput(flops, e2e_ms, world)
    loss_probe = float(C_pin[0, 0])          # the step's result is read on the host

    if rank == 0:
        peaks = measured_peaks()
        kernel_ms = statistics.mean(kernel_samples)
        achieved = 3.0 * flops / (kernel_ms * 1e-3) / 1e12      # FP16 tensor-core TFLOP/s
        peak = peaks["bf16_tflops"]
        sm_max = clocks.get("sm_max_mhz") or 1965.0
        clock_peak = sm_count * 8192 * sm_max * 1e6 / 1e12       # dense FP16 flop/clk/SM x clock
        cpu_val, cpu_s, cpu_threads = cpu_oracle_sample(args.cpu_rows)
        # Error of the step's result against an FP64 product (the second half of the metric: "max
        # rel err vs FP64"), on one row out of every 128-row tile, computed by the CPU oracle's
        # reference and error helpers.  Componentwise: |C - C64| / (|A||B|), the quantity the
        # method's bound (Eq. main_bound) and the test gate 2 K 2^-24 are stated in.
        import numpy as np
        import oracle
        h.sgemm_cube(A, B, C, SCALE_EXP, binding.TERMWISE)
        rows_idx = np.array([min(M - 1, b * 128 + (b * 37 + 5) % 128) for b in range((M + 127) // 128)])
        C_rows = C[torch.as_tensor(rows_idx, device=dev)].cpu().numpy()
        C64, AB = oracle.dgemm_ref(A_host.numpy()[rows_idx], B_host.numpy())
        accuracy = {"rows_sampled": int(rows_idx.size), "reference": "CPU oracle (FP64)",
                    "frobenius_rel_err": oracle.frobenius_rel_err(C_rows, C64),
                    "max_componentwise_err": oracle.componentwise_err(C_rows, C64, AB),
                    "componentwise_gate_2K_u32": 2.0 * K * 2.0 ** -24}
        del C64, AB
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f16 products, f32 accumulate",
            "data": "synthetic",
            "config": {"workload": WORKLOAD, "entry_point": "sgemm_cube, strategy %s: split kernel (both operands, one launch) + three-product "
                                      "tensor-core kernel per step" % args.strategy
                       if args.strategy != "fused" else "sgemm_cube, strategy fused: one kernel per step",
                       "l2": "inputs (512 MiB) larger than L2; no flush",
                       "parallelism": "replicas x%d" % world if world > 1 else "1 GPU"},
            "clocks": clocks,
            "e2e": {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": 4 * (M * K + K * N),
                    "d2h_bytes_per_step": 4 * M * N, "result_probe": loss_probe},
            "gpu_launches": int(launches),
            "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                         "frac": achieved / peak, "traffic": KERNEL_DRAM_BYTES_PER_LAUNCH if (M == 8192 and args.strategy != "fused") else None,
                         "peak_source": "%s cuBLAS bf16 burst (fp16 has the same nominal rate)"
                                        % peaks["source"],
                         "kernel_ms": kernel_ms,
                         "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"],
                         "frac_of_max_clock_peak": achieved / clock_peak,
                         "max_clock_peak_tflops": clock_peak,
                         **{k: v for k, v in clock_fracs(flops / kernel_ms / 1e9, kernel_clock).items()
                            if k in ("sm_mhz_in_kernel", "kernel_cycles")}},
            # The three fractions of the three-GEMM roofline (FP16 tensor peak / 3): at the maximum
            # SM clock (the stated target is 0.70 of this one), at the SM clock measured inside the
            # kernel (separates kernel quality from the power cap), and against the measured cuBLAS
            # bf16 burst / 3.
            "three_gemm_roofline": {"fp32_equiv_peak_max_clock": clock_peak / 3.0,
                                    "frac": value / world / (clock_peak / 3.0),
                                    "target_frac": 0.70,
                                    "fp32_equiv_measured_burst": peak / 3.0,
                                    "frac_of_measured_burst": value / world / (peak / 3.0),
                                    **{k: v for k, v in clock_fracs(value / world, kernel_clock).items()
                                       if k != "kernel_cycles"}},
            "sustained": sustained,
            "fused": fused_block,
            "cpu_baseline": {"value": cpu_val, "unit": UNIT, "cores": cpu_threads, "kind": "oracle",
                             "sample": "%d of %d rows of A against the full B, %.1f s"
                                       % (args.cpu_rows, M, cpu_s)},
            "ablation": extra,
            "accuracy": accuracy,
            "paper_context": "65.3 TFLOP/s = 77% of 256/3 on Ascend 910A (other hardware; not a target)",
        }
        print(json.dumps(out))
    h.destroy()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
