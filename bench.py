#!/usr/bin/env python
"""Benchmark of the GEMM hot path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

A step is one pass of the whole hot path -- one C = alpha*op(A)*op(B) + beta*C through the C ABI -- on
seeded synthetic inputs already resident in HBM.  The default workload is bf16 8192^3 NN, the shape the
throughput target is stated on; `--workload NAME` (names: --list) selects another.  For N > 1 the script is
launched by torchrun, one rank per GPU; every rank runs its own copy of the workload (independent problems,
no collective on the data path, weak scaling) and the value is the sum over ranks divided by the slowest
rank's device time.

Timing.  After W (>= 3) warm-up steps the timed region is R back-to-back blocks of K steps each, R chosen so
that the region lasts at least --min-seconds (default 1 s): long enough for the power cap to settle and for
the clock sampler to collect hundreds of samples.  CUDA events on the launching stream bracket every block;
`value` and `ms_per_step` are the mean over all R*K steps (a sustained figure), `burst` is the best block.

Rank 0 prints ONE JSON line: metric/value/unit, ms_per_step, repeats, `roofline` (tensor, ALU or HBM bound,
against fixed, named denominators), `e2e` (host buffers through peak_gemm_host, copies inside the timed
region), `cpu_baseline` (the CPU oracle on a bounded sample), `clocks`, `gpu_launches`, and `other_workloads`:
every other benchmark configuration with its own throughput, clocks and a cuBLAS (torch) context figure taken
with the same protocol.

`--impl reference` times the CPU oracle, as it stands, on the host cores (rank 0 only).
"""
from __future__ import annotations

import argparse
import glob
import json
import math
import os
import re
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
NOMINAL_BF16_TFLOPS = 2250.0                       # dense, datasheet
SM_COUNT, SM_MAX_MHZ = 148, 1965.0
ALU_PEAK_TFLOPS = SM_COUNT * 128 * 2 * SM_MAX_MHZ * 1e6 / 1e12     # fp32 FMA lanes x 2 flop x max SM clock
DEFAULT_WORKLOAD = "bf16_8192_nn"
# the benchmark configurations reported beside the headline, in this order
OTHER_WORKLOADS = [
    "bf16_4096_nn",
    "fp16_2048_nn", "fp16_2048_tn", "fp16_4096_nn", "fp16_4096_tn", "fp16_8192_nn", "fp16_8192_tn",
    "bf16_tfm_16384x4096x4096_nt", "bf16_tfm_16384x14336x4096_nt", "bf16_tfm_16384x4096x14336_nt",
    "bf16_5000x3000x2500_tn", "bf16_16x4096x4096_tn", "bf16_128x14336x4096_tn", "bf16_8192x8192x128_nt",
    "fp32_4096_nn", "fp32_8192_nn",
    "e4m3_8192_nt", "e4m3_8192_nn",
]


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
    for n in (2048, 4096, 8192):
        for it in ("e4m3", "e5m2"):
            for lay in ("NT", "NN", "TN", "TT"):
                c = W.fp8_workload(n, it, lay)
                t[c.name] = c
    for i in range(3):
        t[W.config3(i).name] = W.config3(i)
        t[W.config4_ragged(i).name] = W.config4_ragged(i)
    for k in (128, 512):
        t[W.short_k_workload(k).name] = W.short_k_workload(k)
    return t


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def hbm_bound(case, peaks) -> bool:
    """A problem whose minimum HBM time exceeds its tensor time at the measured peaks."""
    if case.in_type == "f32":
        return False
    scale = 2.0 if case.in_type in ("e4m3", "e5m2") else 1.0
    t_tensor = case.flops / (scale * float(peaks["bf16_tflops"]) * 1e12)
    t_hbm = case.min_bytes() / (float(peaks["hbm_gbs"]) * 1e9)
    return t_hbm > t_tensor


def roofline_block(case, kernel_ms, peaks, peak_kind):
    """Roofline of one launch against fixed, named denominators.  Tensor-bound work is compared with the
    SUSTAINED cuBLAS figure (every timed region here is long enough to run under the power cap); the burst and
    nominal fractions are always printed beside it."""
    tfl = case.flops / (kernel_ms * 1e-3) / 1e12
    if case.in_type == "f32":
        roof = {"bound": "alu", "achieved": tfl, "peak": ALU_PEAK_TFLOPS, "unit": "TFLOP/s",
                "peak_kind": "derived: 148 SMs x 128 fp32 FMA lanes x 2 flop x 1.965 GHz (max SM clock)"}
    elif hbm_bound(case, peaks):
        gbs = case.min_bytes() / (kernel_ms * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": gbs, "peak": float(peaks["hbm_gbs"]), "unit": "GB/s",
                "peak_kind": f"{peak_kind} copy bandwidth; achieved = minimum HBM bytes of the problem / kernel time",
                "tflops": tfl}
    else:
        burst = float(peaks["bf16_tflops"])
        sustained = float(peaks.get("bf16_tflops_sustained", burst))
        nominal, note = NOMINAL_BF16_TFLOPS, ""
        if case.in_type in ("e4m3", "e5m2"):
            # no 8-bit peak was measured: the bf16 figures times the nominal dense ratio (4.5 / 2.25 PFLOP/s)
            burst, sustained, nominal, note = 2 * burst, 2 * sustained, 2 * nominal, " x 2 (nominal fp8 : bf16 ratio)"
        roof = {"bound": "tensor", "achieved": tfl, "peak": sustained, "unit": "TFLOP/s",
                "peak_kind": f"{peak_kind} cuBLAS bf16 8192^3 sustained{note} (fixed rule: every timed region runs "
                             "for >= 0.3 s back to back, under the power cap)",
                "frac_of_sustained_peak": tfl / sustained, "frac_of_burst_peak": tfl / burst,
                "frac_of_nominal_peak": tfl / nominal,
                "peaks": {"sustained": sustained, "burst": burst, "nominal_dense": nominal}}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["kernel_ms"] = kernel_ms
    roof["algorithmic_flops_per_launch"] = case.flops
    roof["min_hbm_bytes_per_launch"] = case.min_bytes()
    return roof


# ------------------------------------------------------------------------------- ncu traffic from profiles/
_UNIT = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}


def _kernel_key(name: str):
    """'void umma_gemm_kernel<2, 512, __nv_bfloat16, 0, 0, 0, 0>(...)' -> ('umma_gemm_kernel', ['2', '512', ...])."""
    m = re.search(r"(\w+)\s*<([^>]*)>", name)
    if not m:
        m2 = re.search(r"(\w+_kernel)", name)
        return (m2.group(1), []) if m2 else None
    return m.group(1), [a.strip().replace("(bool)", "").replace("false", "0").replace("true", "1")
                        for a in m.group(2).split(",")]


def profile_traffic(workload: str, launched: str):
    """DRAM bytes per launch (read + write) from the ncu summary under profiles/ that covers this workload AND
    the kernel that was actually launched; (None, reason) otherwise."""
    want = _kernel_key(launched)
    files = sorted(glob.glob(os.path.join(ROOT, "profiles", f"*_{workload}.md")))
    if not files:
        return None, f"no ncu summary for {workload} under profiles/"
    seen = []
    for path in files:
        text = open(path).read()
        km = re.search(r"^Kernel Name\s+(.*)$", text, re.M)
        rd = re.search(r"^dram__bytes_read\.sum\s+([0-9.]+)\s+(\w+)", text, re.M)
        wr = re.search(r"^dram__bytes_write\.sum\s+([0-9.]+)\s+(\w+)", text, re.M)
        if not (km and rd and wr):
            continue
        have = _kernel_key(km.group(1))
        seen.append(km.group(1).strip()[:80])
        # template arguments compare position by position ("*" = any); a list that is shorter than the other
        # (a summary taken before the kernel gained a trailing flag) matches when the extra arguments are 0
        n = min(len(want[1]), len(have[1])) if want and have else 0
        same = bool(want and have and want[0] == have[0] and
                    all(a == b or "*" in (a, b) for a, b in zip(want[1][:n], have[1][:n])) and
                    all(x in ("0", "*") for x in want[1][n:] + have[1][n:]))
        if same:
            total = float(rd.group(1)) * _UNIT[rd.group(2)] + float(wr.group(1)) * _UNIT[wr.group(2)]
            return total, f"quoted from {os.path.relpath(path, ROOT)} (one ncu capture; not measured in this run)"
    return None, f"launched kernel '{launched.split(' grid')[0]}' differs from the profiled one(s): {seen}"


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
        return {"sm_mhz": float(np.median(self.samples)), "sm_mhz_min": float(np.min(self.samples)),
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


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
    per_step = max(0.02, min(20.0, 120.0 / max(args.steps + args.warmup, 1)))
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
        "config": workload_config(case),
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


def set_bytes(case) -> int:
    """Bytes of one (A, B, C) set as stored."""
    from paper_2512_19018_b200 import workloads as W
    si, so = W.ELEM_BYTES[case.in_type], W.ELEM_BYTES[case.out_type]
    return (case.a_shape[0] * case.lda + case.b_shape[0] * case.ldb) * si + case.M * case.ldc * so


def rotation_sets(case) -> int:
    """How many distinct (A, B, C) sets the timed loop rotates through: one when a set alone is larger than
    three L2 capacities (nothing of a step's operands survives to the next step that uses them), otherwise
    enough that a full rotation touches more than three L2 capacities."""
    per_set = set_bytes(case)
    if per_set >= 3 * L2_BYTES:
        return 1
    return int(max(2, min(64, math.ceil(3 * L2_BYTES / per_set) + 1)))


def l2_note(case) -> str:
    n, per_set = rotation_sets(case), set_bytes(case)
    if n == 1:
        return f"inputs larger than L2: one input/output set of {per_set / 2**20:.0f} MiB against 126 MB of L2"
    return f"rotating {n} input/output sets ({n * per_set / 2**20:.0f} MiB) so that no step finds its operands in L2"


def workload_config(case, epilogue="none"):
    cfg = {"workload": case.name, "M": case.M, "N": case.N, "K": case.K, "layout": case.layout,
           "in": case.in_type, "out": case.out_type, "alpha": case.alpha, "beta": case.beta,
           "inputs": case.dist, "seed": case.seed, "l2": l2_note(case)}
    if epilogue != "none":
        cfg["fused_epilogue"] = epilogue
    return cfg


# --------------------------------------------------------------------------------------------- our arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--variant", default="auto")
    ap.add_argument("--min-seconds", type=float, default=1.0, help="least length of the headline's timed region")
    ap.add_argument("--extra-seconds", type=float, default=0.3, help="same for each secondary workload")
    ap.add_argument("--no-extra", action="store_true", help="skip the secondary workloads and the CPU baseline")
    ap.add_argument("--only-extra", default="", help="comma-separated subset of the secondary workloads")
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
    args.steps = max(1, args.steps)
    if args.impl == "reference":
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
    if distributed:
        # the cluster-multicast plug-in is for single-GPU processes only: never use it in a multi-rank job,
        # whether or not its file travelled with the package
        P.peak_set_tuning(P.PEAK_TUNE_MULTICAST, 1)
    for kv in filter(None, args.tune.split(",")):
        k, v = kv.split("=")
        P.peak_set_tuning(int(k), int(v))
    warmup = max(args.warmup, 3)
    peaks, peak_kind = measured_peaks()

    def barrier():
        if distributed:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(x: float) -> float:
        return reduce_max(x, dist if distributed else None, "cuda")

    def time_blocks(step, steps, warm, min_seconds, clocks_index=None, check=None):
        """`warm` warm-up steps and one untimed calibration block, then R back-to-back blocks of `steps` calls,
        R = the fewest blocks that fill `min_seconds`; CUDA events on the launching stream bracket every block.
        Returns (total ms over all blocks [max over ranks], per-block ms [this rank], R, clock summary,
        kernels this library launched inside the timed region)."""
        stream = torch.cuda.current_stream()
        for i in range(warm):
            step(i)
        if check:
            check()
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0.record(stream)
        for i in range(steps):
            step(i)
        c1.record(stream)
        torch.cuda.synchronize()
        block_ms = max_over_ranks(max(c0.elapsed_time(c1), 1e-3))
        repeats = int(max(1, min(20000, math.ceil(min_seconds * 1e3 / block_ms))))
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(repeats + 1)]
        sampler = ClockSampler(clocks_index) if clocks_index is not None else None
        barrier()
        if sampler:
            sampler.__enter__()
        n_before = P.peak_kernel_launches()
        ev[0].record(stream)
        i = 0
        for r in range(repeats):
            for _ in range(steps):
                step(i)
                i += 1
            ev[r + 1].record(stream)
        n_launched = P.peak_kernel_launches() - n_before
        barrier()
        if sampler:
            sampler.__exit__()
        total = max_over_ranks(ev[0].elapsed_time(ev[-1]))
        blocks = [ev[r].elapsed_time(ev[r + 1]) for r in range(repeats)]
        if check:
            check()
        return total, blocks, repeats, (sampler.summary() if sampler else None), n_launched

    class Resident:
        """One problem's seeded inputs, on the host (stored bits) and uploaded unchanged to HBM."""

        def __init__(self, case, keep_host=True):
            self.case = case
            A_h, B_h, c0 = W.make_inputs(case)
            C0_h = c0 if c0 is not None else W.poison_c(case)
            self.A, self.B, self.C = (self.up(A_h, case.in_type), self.up(B_h, case.in_type),
                                      self.up(C0_h, case.out_type))
            if keep_host:
                self.A_h, self.B_h, self.C0_h = A_h, B_h, C0_h

        @staticmethod
        def up(arr, t):
            if t in ("f32", "e4m3", "e5m2"):          # float32 values / raw bytes
                return torch.from_numpy(arr).cuda()
            return torch.from_numpy(arr.view(np.int16)).cuda().view(torch.float16 if t == "f16" else torch.bfloat16)

        def sets(self):
            out = [(self.A, self.B, self.C)]
            for _ in range(rotation_sets(self.case) - 1):
                out.append((self.A.clone(), self.B.clone(), self.C.clone()))
            return out

    def our_step_fn(c, sets, epilogue="none", var=None):
        stream = torch.cuda.current_stream()
        var = variant if var is None else var
        act = {"none": P.PEAK_ACT_NONE, "bias": P.PEAK_ACT_NONE, "bias_relu": P.PEAK_ACT_RELU,
               "bias_gelu": P.PEAK_ACT_GELU}[epilogue]
        bias = None
        if epilogue != "none":
            rng = np.random.Generator(np.random.Philox(c.seed + 99))
            bias = torch.from_numpy(rng.standard_normal(c.N, dtype=np.float32)).cuda()
        n = len(sets)

        def step(i):
            A, B, C = sets[i % n]
            if epilogue == "none":
                P.peak_gemm_variant(var, c.dtype, c.transA, c.transB, c.M, c.N, c.K, c.alpha, A, c.lda, B, c.ldb,
                                    c.beta, C, c.ldc, stream)
            else:
                P.peak_gemm_fused(c.dtype, c.transA, c.transB, c.M, c.N, c.K, c.alpha, A, c.lda, B, c.ldb, c.beta, C,
                                  c.ldc, bias, act, stream, variant=var)

        def check():
            rc, detail = P.peak_check(stream)
            assert rc == P.PEAK_OK, f"device status {rc} 0x{detail:x}"
        return step, check

    def cublas_step_fn(c, sets):
        """torch (cuBLAS / cuBLASLt) on the same tensors: the same operation as far as torch offers it."""
        torch.backends.cuda.matmul.allow_tf32 = False
        opA = [(a.t() if c.transA else a)[:c.M, :c.K] for a, _, _ in sets]
        opB = [(b.t() if c.transB else b)[:c.K, :c.N] for _, b, _ in sets]
        Cs = [cc[:, :c.N] for _, _, cc in sets]
        n = len(sets)
        if c.in_type in ("e4m3", "e5m2"):
            f8 = torch.float8_e4m3fn if c.in_type == "e4m3" else torch.float8_e5m2
            opA = [a.view(f8) for a in opA]
            opB = [b.view(f8) for b in opB]
            one = torch.ones((), dtype=torch.float32, device="cuda")
            out_t = torch.bfloat16 if c.out_type == "bf16" else torch.float32

            def step(i):
                torch._scaled_mm(opA[i % n], opB[i % n], scale_a=one, scale_b=one, out_dtype=out_t)
            return step, "torch._scaled_mm, unit scales"
        if c.beta != 0:
            def step(i):
                torch.addmm(Cs[i % n], opA[i % n], opB[i % n], beta=c.beta, alpha=c.alpha, out=Cs[i % n])
            return step, "torch.addmm in place"
        if c.in_type == "f16" and c.out_type == "f32":
            try:
                torch.mm(opA[0][:16, :16].contiguous(), opB[0][:16, :16].contiguous(), out_dtype=torch.float32)

                def step(i):
                    torch.mm(opA[i % n], opB[i % n], out_dtype=torch.float32, out=Cs[i % n])
                step(0)
                return step, "torch.mm with out_dtype=float32"
            except Exception:
                pass

        def step(i):
            torch.matmul(opA[i % n], opB[i % n])
        return step, "torch.matmul"

    def tflops_of(c, steps_total, ms):
        return c.flops * steps_total / (ms * 1e-3) / 1e12

    # ---- headline ----------------------------------------------------------------------------------
    seeded = rank_case(case, rank)                                 # every rank its own problem
    dc = Resident(seeded)
    sets = dc.sets()
    step, check = our_step_fn(seeded, sets, args.epilogue)
    total_ms, blocks, repeats, clocks, launches = time_blocks(step, args.steps, warmup, args.min_seconds, local_rank,
                                                              check)
    launched = P.peak_last_kernel()
    timed_steps = repeats * args.steps
    value = aggregate_value(case, world, timed_steps, total_ms)
    # one launch per step on every whole-tile path; a k-split step is the tile kernel plus its small reduction,
    # and the step time is then the time of both
    roof = roofline_block(case, total_ms / timed_steps, peaks, peak_kind)
    roof["launches_per_step"] = launches / float(timed_steps)
    roof["traffic"], roof["traffic_source"] = profile_traffic(case.name, launched)
    roof["kernel"] = launched
    best = min(blocks)
    burst = {"value": tflops_of(case, args.steps, best) * world, "unit": "TFLOP/s", "ms_per_step": best / args.steps,
             "note": "best single block of `steps` back-to-back calls inside the timed region (this rank)"}

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
        e_steps = max(3, min(args.steps, 20))
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
               "ms_per_step": e_ms / e_steps,
               "note": "peak_gemm_host: pinned host buffers in, host buffer out, copies inside the timed region"}
        P.peak_release_staging()
        del hA, hB, hC

    # ---- cuBLAS context for the headline, the other configurations, the CPU baseline (N = 1 only) ------
    extra, cpu = None, None
    if rank == 0 and not distributed and not args.no_extra:
        extra = {}

        def context(c, sets, steps_blk, seconds):
            try:
                cstep, how = cublas_step_fn(c, sets)
                ms, blk, rep, clk, _ = time_blocks(cstep, steps_blk, 3, seconds, local_rank)
                return {"tflops": tflops_of(c, rep * steps_blk, ms), "ms_per_step": ms / (rep * steps_blk),
                        "how": how + "; same buffers, rotation, block protocol; context only, not this library",
                        "sm_mhz": clk["sm_mhz"] if clk else None}
            except Exception as exc:   # context only: never fail the bench for it
                return {"error": str(exc)[:200]}

        extra["cublas_context"] = dict(workload=case.name, **context(seeded, sets, args.steps, args.min_seconds))
        run, desc, threads = oracle_sampler(dc.case, dc.A_h, dc.B_h, dc.C0_h if dc.case.beta != 0 else None, 15.0)
        tf, dt = run()
        cpu = {"value": tf, "unit": "TFLOP/s", "cores": threads, "kind": "oracle", "sample": desc, "seconds": dt}
        del sets, dc, step
        torch.cuda.empty_cache()
        names = [n for n in OTHER_WORKLOADS if n != case.name]
        if args.only_extra:
            names = [n for n in args.only_extra.split(",") if n in table]
        for name in names:
            c2 = table[name]
            try:
                d2 = Resident(c2, keep_host=False)
                s2 = d2.sets()
                st2, ck2 = our_step_fn(c2, s2, var=P.PEAK_VARIANT_AUTO)
                ms2, blk2, rep2, clk2, nl2 = time_blocks(st2, args.steps, 3, args.extra_seconds, local_rank, ck2)
                kern2 = P.peak_last_kernel()
                per = ms2 / (rep2 * args.steps)
                r2 = roofline_block(c2, per, peaks, peak_kind)
                entry = {"tflops": tflops_of(c2, rep2 * args.steps, ms2), "ms_per_step": per, "steps": args.steps,
                         "repeats": rep2, "bound": r2["bound"], "frac": r2["frac"], "peak": r2["peak"],
                         "peak_unit": r2["unit"], "achieved": r2["achieved"], "kernel": kern2,
                         "launches_per_step": nl2 / float(rep2 * args.steps),
                         "burst_tflops": tflops_of(c2, args.steps, min(blk2)),
                         "clocks": {k: clk2[k] for k in ("sm_mhz", "reasons", "samples")} if clk2 else None,
                         "l2": l2_note(c2)}
                if "frac_of_burst_peak" in r2:
                    entry["frac_of_burst_peak"] = r2["frac_of_burst_peak"]
                    entry["frac_of_nominal_peak"] = r2["frac_of_nominal_peak"]
                ctx = context(c2, s2, args.steps, args.extra_seconds)
                entry["cublas_context"] = ctx
                if "tflops" in ctx:
                    entry["vs_cublas"] = entry["tflops"] / ctx["tflops"]
                extra[name] = entry
                del d2, s2, st2
            except Exception as exc:
                extra[name] = {"error": str(exc)[:300]}
            torch.cuda.empty_cache()

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps, "warmup": warmup,
            "ms_per_step": total_ms / timed_steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": case.in_type, "data": "synthetic", "config": workload_config(case, args.epilogue),
            "repeats": repeats, "timed_steps": timed_steps, "timed_region_s": total_ms * 1e-3, "burst": burst,
            "variant": args.variant if variant != P.PEAK_VARIANT_AUTO else "auto",
            "roofline": roof, "e2e": e2e, "cpu_baseline": cpu, "clocks": clocks,
            "gpu_launches": int(launches),
        }
        if extra:
            line["other_workloads"] = extra
        print(json.dumps(line), flush=True)
    if distributed:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
