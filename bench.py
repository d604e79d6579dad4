#!/usr/bin/env python
"""Benchmark of the GEMM hot path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

A step is one pass of the whole hot path -- one C = alpha*op(A)*op(B) + beta*C through the C ABI -- on
seeded synthetic inputs already resident in HBM.  The default workload is the bf16 4096^3 NN configuration;
`--workload bf16_8192_nn` (and the other names printed by --list) select the rest.  For N > 1 the script
is launched by torchrun, one rank per GPU; every rank runs its own copy of the workload (independent
problems, no collective on the data path, weak scaling) and the value is the sum over ranks divided by
the slowest rank's device time.

Rank 0 prints ONE JSON line: metric/value/unit, ms_per_step, `e2e` (host buffers through peak_gemm_host,
copies inside the timed region), `roofline` (tensor or ALU bound, against the measured peak),
`cpu_baseline` (the CPU oracle on a bounded sample), `clocks`, `gpu_launches`.

`--impl reference` times the CPU oracle, as it stands, on the host cores (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "GEMM TFLOP/s (device-timed, 1 B200) and fraction of dense BF16 tensor peak"
L2_BYTES = 126e6
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
SM_COUNT, SM_MAX_MHZ = 148, 1965.0
# DRAM bytes per launch (read + write) of the dominant kernel from the ncu capture summarised under
# profiles/; None where no capture exists for the workload.
NCU_TRAFFIC_BYTES = {
    "bf16_4096_nn": 86.8e6,     # profiles/umma_gemm_multicast512_bf16_4096_nn.md (74.4 MB read + 12.4 MB written)
    "bf16_8192_nn": 0.986e9,    # profiles/umma_gemm_2cta_512wide_bf16_8192_nn.md (0.866 GB read + 0.120 GB written)
    "e4m3_8192_nt": 0.461e9,    # profiles/umma_gemm_2cta_e4m3_8192_nt.md (0.344 GB read + 0.117 GB written)
    "fp32_8192_nn": 3.553e9,    # profiles/sgemm_async_fp32_8192_nn.md (3.281 GB read + 0.272 GB written)
}


def workloads_table():
    from paper_2512_19018_b200 import workloads as W
    t = {
        "fp16_512_nn": W.config0(),
        "bf16_4096_nn": W.config1(),
        "bf16_8192_nn": W.target_workload(),
        "fp32_4096_nn": W.config4_sgemm(4096),
        "fp32_8192_nn": W.config4_sgemm(8192),
    }
    for n in (1024, 2048, 4096, 8192, 16384):
        for lay in ("NN", "TN"):
            c = W.config2(n, lay)
            t[c.name] = c
    for n in (4096, 8192):
        for it in ("e4m3", "e5m2"):
            c = W.fp8_workload(n, it)
            t[c.name] = c
    for i in range(3):
        t[W.config3(i).name] = W.config3(i)
        t[W.config4_ragged(i).name] = W.config4_ragged(i)
    return t


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# --------------------------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU while the timed region runs (NVML, read-only)."""

    def __init__(self, index: int, period_s: float = 0.002):
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            uuid = None
            try:
                import torch
                uuid = str(torch.cuda.get_device_properties(index).uuid)
            except Exception:
                pass
            self.h = None
            if uuid:
                try:
                    self.h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode())
                except Exception:
                    self.h = None
            if self.h is None:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# --------------------------------------------------------------------------------------------- oracle legs
def oracle_sampler(case, A, B, C0, target_seconds: float):
    """The CPU oracle (as it stands) on a rows x cols sub-grid of the workload sized, from a short probe,
    for roughly `target_seconds` of work.  Returns (run, description, threads); run() -> (tflops, seconds)."""
    import oracle
    T = {"f16": oracle.F16, "bf16": oracle.BF16, "f32": oracle.F32, "e4m3": oracle.E4M3, "e5m2": oracle.E5M2}

    def run_pq(p, q):
        rows = np.linspace(0, case.M - 1, p).astype(np.int64)
        cols = np.linspace(0, case.N - 1, q).astype(np.int64)
        t0 = time.perf_counter()
        oracle.gemm_submatrix(T[case.in_type], T[case.out_type], case.transA, case.transB, case.M, case.N, case.K,
                              case.alpha, A, case.lda, B, case.ldb, case.beta, C0, case.ldc, rows, cols, want_S=False)
        return time.perf_counter() - t0

    p0, q0 = min(case.M, 64), min(case.N, 64)
    run_pq(p0, q0)                                         # builds / loads the shared object, warms the pages
    t_probe = max(run_pq(p0, q0), 1e-5)
    rate = p0 * q0 * case.K / t_probe                      # MAC/s on the probe
    side = int(math.sqrt(max(rate * target_seconds / max(case.K, 1), 1.0)))
    p, q = min(case.M, max(side, 16)), min(case.N, max(side, 16))

    def run():
        dt = run_pq(p, q)
        return 2.0 * p * q * case.K / dt / 1e12, dt

    desc = f"{p} x {q} sub-grid of C (all K={case.K} terms of each element), fp64 triple loop"
    return run, desc, oracle.num_threads()


def run_reference(args, case):
    """--impl reference: the oracle on the host cores; each step is a bounded sample of the workload."""
    from paper_2512_19018_b200 import workloads as W
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    A, B, C0 = W.make_inputs(case)
    per_step = max(0.02, min(20.0, 150.0 / max(args.steps + args.warmup, 1)))
    run, desc, threads = oracle_sampler(case, A, B, C0, per_step)
    times, tfl = [], []
    for i in range(args.warmup + args.steps):
        tf, dt = run()
        if i >= args.warmup:
            times.append(dt)
            tfl.append(tf)
    value = float(len(times) / np.sum(1.0 / np.array(tfl)))       # total flops / total time (equal samples)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": float(np.mean(times) * 1e3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(case, None),
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


def rank_case(case, rank: int):
    """The problem rank `rank` runs: same shape and recipe, its own seed (independent problems, no collective
    on the data path)."""
    return case.with_(case=case.case + 17 * rank)


def reduce_max(x: float, dist=None, device="cpu") -> float:
    """Max over ranks of a per-rank time (the slowest rank defines the step time)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return x
    import torch
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(case, world: int, steps: int, max_ms: float) -> float:
    """Whole-job TFLOP/s: every rank did `steps` GEMMs of `case.flops`; time is the slowest rank's."""
    return world * case.flops * steps / (max_ms * 1e-3) / 1e12


def workload_config(case, l2_note, epilogue="none"):
    cfg = {"workload": case.name, "M": case.M, "N": case.N, "K": case.K, "layout": case.layout,
           "in": case.in_type, "out": case.out_type, "alpha": case.alpha, "beta": case.beta,
           "inputs": case.dist, "seed": case.seed}
    if l2_note:
        cfg["l2"] = l2_note
    if epilogue != "none":
        cfg["fused_epilogue"] = epilogue
    return cfg


# --------------------------------------------------------------------------------------------- our arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="bf16_4096_nn")
    ap.add_argument("--variant", default="auto")
    ap.add_argument("--no-extra", action="store_true", help="skip the secondary workloads and the CPU baseline")
    ap.add_argument("--epilogue", default="none", choices=["none", "bias", "bias_relu", "bias_gelu"],
                    help="time peak_gemm_fused with this fused tail instead of peak_gemm")
    ap.add_argument("--tune", default="", help="comma-separated key=value pairs passed to peak_set_tuning")
    ap.add_argument("--list", action="store_true")
    args = ap.parse_args()

    table = workloads_table()
    if args.list:
        print("\n".join(sorted(table)))
        return 0
    case = table[args.workload]
    if args.impl == "reference":
        args.steps = 2 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        return run_reference(args, case)

    import torch
    import torch.distributed as dist

    from paper_2512_19018_b200 import binding as P
    from paper_2512_19018_b200 import workloads as W

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    distributed = world > 1
    if distributed:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    variants = {"auto": P.PEAK_VARIANT_AUTO, "umma_1cta": P.PEAK_VARIANT_UMMA_1CTA, "umma_2cta": P.PEAK_VARIANT_UMMA_2CTA,
                "sgemm": P.PEAK_VARIANT_SGEMM, "fallback": P.PEAK_VARIANT_FALLBACK}
    variant = variants[args.variant]
    P.load()
    for kv in filter(None, args.tune.split(",")):
        k, v = kv.split("=")
        P.peak_set_tuning(int(k), int(v))

    def barrier():
        if distributed:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(x: float) -> float:
        return reduce_max(x, dist if distributed else None, "cuda")

    def time_device(case, steps, warmup, sets, clocks_index=None):
        """W warm-up steps, then exactly `steps` back-to-back calls timed with CUDA events on the launching
        stream, rotating through `sets` so that no step finds its inputs in L2."""
        stream = torch.cuda.current_stream()
        act = {"none": P.PEAK_ACT_NONE, "bias": P.PEAK_ACT_NONE, "bias_relu": P.PEAK_ACT_RELU,
               "bias_gelu": P.PEAK_ACT_GELU}[args.epilogue]
        bias = None
        if args.epilogue != "none":
            rng = np.random.Generator(np.random.Philox(case.seed + 99))
            bias = torch.from_numpy(rng.standard_normal(case.N, dtype=np.float32)).cuda()
        def step(i):
            A, B, C = sets[i % len(sets)]
            if args.epilogue == "none":
                P.peak_gemm_variant(variant, case.dtype, case.transA, case.transB, case.M, case.N, case.K, case.alpha,
                                    A, case.lda, B, case.ldb, case.beta, C, case.ldc, stream)
            else:
                P.peak_gemm_fused(case.dtype, case.transA, case.transB, case.M, case.N, case.K, case.alpha, A, case.lda,
                                  B, case.ldb, case.beta, C, case.ldc, bias, act, stream, variant=variant)
        for i in range(warmup):
            step(i)
        rc, detail = P.peak_check(stream)
        assert rc == P.PEAK_OK, f"device status {rc} 0x{detail:x}"
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sampler = ClockSampler(clocks_index) if clocks_index is not None else None
        n0 = P.peak_kernel_launches()
        barrier()
        if sampler:
            sampler.__enter__()
        e0.record(stream)
        for i in range(steps):
            step(i)
        e1.record(stream)
        barrier()
        if sampler:
            sampler.__exit__()
        ms = max_over_ranks(e0.elapsed_time(e1))
        launches = P.peak_kernel_launches() - n0
        rc, detail = P.peak_check(stream)
        assert rc == P.PEAK_OK, f"device status {rc} 0x{detail:x}"
        return ms, launches, (sampler.summary() if sampler else None)

    def make_sets(case, dc):
        """Enough distinct copies of (A, B, C) that a rotation touches more than three L2 capacities."""
        per_set = dc.A.numel() * dc.A.element_size() + dc.B.numel() * dc.B.element_size() + \
            dc.C.numel() * dc.C.element_size()
        n = int(max(2, min(64, math.ceil(3 * L2_BYTES / per_set) + 1)))
        sets = [(dc.A, dc.B, dc.C)]
        for _ in range(n - 1):
            sets.append((dc.A.clone(), dc.B.clone(), dc.C.clone()))
        return sets, f"rotating {n} input/output sets ({n * per_set / 2**20:.0f} MiB) so that no step hits L2"

    class Resident:
        """One problem's seeded inputs, on the host (stored bits) and uploaded unchanged to HBM."""

        def __init__(self, case):
            self.case = case
            self.A_h, self.B_h, c0 = W.make_inputs(case)
            self.C0_h = c0 if c0 is not None else W.poison_c(case)
            self.A, self.B, self.C = (self.up(self.A_h, case.in_type), self.up(self.B_h, case.in_type),
                                      self.up(self.C0_h, case.out_type))

        @staticmethod
        def up(arr, t):
            if t in ("f32", "e4m3", "e5m2"):          # float32 values / raw bytes
                return torch.from_numpy(arr).cuda()
            return torch.from_numpy(arr.view(np.int16)).cuda().view(torch.float16 if t == "f16" else torch.bfloat16)

    def measure(case, steps, warmup, with_clocks):
        seeded = rank_case(case, rank)                            # every rank its own problem
        dc = Resident(seeded)
        sets, note = make_sets(seeded, dc)
        ms, launches, clocks = time_device(seeded, steps, warmup, sets, local_rank if with_clocks else None)
        return dc, sets, ms, launches, clocks, note

    # default K: about one second of timed work, long enough for the NVML clock samples to mean something
    # (the driver updates them every ~100 ms) and for the power cap to settle -- a sustained figure
    expected_tflops = {"f32": 55.0, "e4m3": 2500.0, "e5m2": 2500.0}.get(case.in_type, 1200.0)
    steps = args.steps if args.steps is not None else max(20, min(20000, int(1.0 * expected_tflops * 1e12 / case.flops)))
    warmup = args.warmup if args.warmup is not None else 10
    warmup = max(warmup, 3)
    dc, sets, ms, launches, clocks, l2_note = measure(case, steps, warmup, True)
    value = aggregate_value(case, world, steps, ms)
    peaks, peak_kind = measured_peaks()

    # ---- roofline of the dominant kernel (the only kernel of a step) ----------------------------------
    kernel_ms = ms / max(launches, 1)
    if case.in_type == "f32":
        alu_peak = SM_COUNT * 128 * 2 * SM_MAX_MHZ * 1e6 / 1e12      # fp32 FMA lanes x 2 flop x max SM clock
        roof = {"bound": "alu", "achieved": case.flops / (kernel_ms * 1e-3) / 1e12, "peak": alu_peak,
                "unit": "TFLOP/s", "peak_kind": "derived: 148 SMs x 128 FMA lanes x 2 x 1.965 GHz"}
    else:
        # a timed region of a second or more runs under the power cap: the sustained cuBLAS figure is the
        # denominator there, the burst figure for short runs
        long_run = ms >= 500.0
        burst, sustained = float(peaks["bf16_tflops"]), float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]))
        ratio_note = ""
        if case.in_type in ("e4m3", "e5m2"):
            # no 8-bit peak was measured: the bf16 figure times the nominal dense ratio (4.5 / 2.25 PFLOP/s)
            burst, sustained, ratio_note = 2.0 * burst, 2.0 * sustained, " x 2 (nominal fp8 : bf16 ratio)"
        roof = {"bound": "tensor", "achieved": case.flops / (kernel_ms * 1e-3) / 1e12,
                "peak": sustained if long_run else burst, "unit": "TFLOP/s",
                "peak_kind": f"{peak_kind} cuBLAS bf16 8192^3{ratio_note}, " +
                             ("sustained (timed region >= 0.5 s)" if long_run else "burst (timed region < 0.5 s)"),
                "frac_of_burst_peak": case.flops / (kernel_ms * 1e-3) / 1e12 / burst,
                "frac_of_sustained_peak": case.flops / (kernel_ms * 1e-3) / 1e12 / sustained}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["traffic"] = NCU_TRAFFIC_BYTES.get(case.name)
    roof["algorithmic_flops_per_launch"] = case.flops
    roof["kernel_ms"] = kernel_ms
    roof["min_hbm_bytes_per_launch"] = case.min_bytes()

    # ---- end to end through the host-buffer entry point -----------------------------------------------
    e2e = None
    if rank == 0 or distributed:
        c = dc.case
        two_byte = c.in_type in ("f16", "bf16")
        hA = torch.from_numpy(dc.A_h.view(np.int16) if two_byte else dc.A_h).pin_memory()
        hB = torch.from_numpy(dc.B_h.view(np.int16) if two_byte else dc.B_h).pin_memory()
        hC = torch.from_numpy(dc.C0_h.view(np.int16) if c.out_type != "f32" else dc.C0_h).clone().pin_memory()
        h2d = hA.numel() * hA.element_size() + hB.numel() * hB.element_size() + \
            (hC.numel() * hC.element_size() if c.beta != 0 else 0)
        d2h = hC.numel() * hC.element_size()
        e_steps = max(3, min(steps, 20))
        stream = torch.cuda.current_stream()
        def host_step():
            P.peak_gemm_host(c.dtype, c.transA, c.transB, c.M, c.N, c.K, c.alpha, hA, c.lda, hB, c.ldb, c.beta, hC,
                             c.ldc, stream)
        for _ in range(3):
            host_step()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(stream)
        for _ in range(e_steps):
            host_step()
        e1.record(stream)
        barrier()
        e_ms = max_over_ranks(e0.elapsed_time(e1))
        e2e = {"value": world * c.flops * e_steps / (e_ms * 1e-3) / 1e12, "unit": "TFLOP/s",
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": e_steps,
               "ms_per_step": e_ms / e_steps}
        P.peak_release_staging()
        del hA, hB, hC

    # ---- secondary workloads (context, N = 1 only) and the CPU baseline --------------------------------
    extra, cpu = None, None
    if rank == 0 and not distributed and not args.no_extra:
        extra = {}
        del sets
        torch.cuda.empty_cache()
        for name in ("bf16_8192_nn", "fp32_4096_nn"):
            if name == case.name:
                continue
            c2 = table[name]
            s2 = max(10, min(400, int(0.3 * (55.0 if c2.in_type == "f32" else 1200.0) * 1e12 / c2.flops)))
            _, _, ms2, l2, _, _ = measure(c2, s2, 5, False)
            tf = c2.flops * s2 / (ms2 * 1e-3) / 1e12
            pk = float(peaks["bf16_tflops"]) if c2.in_type != "f32" else SM_COUNT * 128 * 2 * SM_MAX_MHZ * 1e6 / 1e12
            extra[name] = {"tflops": tf, "ms_per_step": ms2 / s2, "steps": s2, "frac_of_peak": tf / pk, "peak": pk,
                           "peak_kind": "burst" if c2.in_type != "f32" else "derived fp32 FMA peak"}
            torch.cuda.empty_cache()
        # cuBLAS (torch.matmul) on the headline workload with the same protocol: a context point only
        try:
            torch.backends.cuda.matmul.allow_tf32 = False
            dcc = Resident(case)
            csets, _ = make_sets(case, dcc)
            opA = [(a.t() if case.transA else a)[:case.M, :case.K] for a, _, _ in csets]
            opB = [(b.t() if case.transB else b)[:case.K, :case.N] for _, b, _ in csets]
            if case.in_type in ("e4m3", "e5m2"):
                # the library's 8-bit GEMM (cuBLASLt through torch._scaled_mm) with unit scales
                f8 = torch.float8_e4m3fn if case.in_type == "e4m3" else torch.float8_e5m2
                opA = [a.view(f8) for a in opA]
                opB = [b.view(f8) for b in opB]
                one = torch.ones((), dtype=torch.float32, device="cuda")
                out_t = torch.bfloat16 if case.out_type == "bf16" else torch.float32
                def mm(i):
                    torch._scaled_mm(opA[i % len(csets)], opB[i % len(csets)], scale_a=one, scale_b=one,
                                     out_dtype=out_t)
            else:
                def mm(i):
                    torch.matmul(opA[i % len(csets)], opB[i % len(csets)])
            for i in range(10):
                mm(i)
            torch.cuda.synchronize()
            c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            c0.record()
            for i in range(steps):
                mm(i)
            c1.record()
            torch.cuda.synchronize()
            extra["cublas_context"] = {"workload": case.name, "tflops": case.flops * steps / (c0.elapsed_time(c1) * 1e-3) / 1e12,
                                       "steps": steps, "note": "torch.matmul (torch._scaled_mm for 8-bit inputs), same rotation and step count; not this library"}
            del dcc, csets, opA, opB
        except Exception as exc:  # context only: never fail the bench for it
            extra["cublas_context"] = {"error": str(exc)[:200]}
        run, desc, threads = oracle_sampler(dc.case, dc.A_h, dc.B_h, dc.C0_h if dc.case.beta != 0 else None, 15.0)
        tf, dt = run()
        cpu = {"value": tf, "unit": "TFLOP/s", "cores": threads, "kind": "oracle", "sample": desc, "seconds": dt}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": steps, "warmup": warmup,
            "ms_per_step": ms / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": case.in_type,
            "data": "synthetic", "config": workload_config(case, l2_note, args.epilogue),
            "variant": P.peak_variant_string(P.peak_query_variant(
                case.dtype, case.transA, case.transB, case.M, case.N, case.K, case.alpha, dc.A, case.lda, dc.B,
                case.ldb, case.beta, dc.C, case.ldc)) if variant == P.PEAK_VARIANT_AUTO else args.variant,
            "roofline": roof, "e2e": e2e, "cpu_baseline": cpu, "clocks": clocks, "gpu_launches": int(launches),
        }
        if extra:
            line["other_workloads"] = extra
        print(json.dumps(line), flush=True)
    if distributed:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
