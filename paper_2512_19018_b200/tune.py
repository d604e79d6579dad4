"""Enumerating tuner: run every valid combination of the library's performance knobs on one GEMM shape and
report the fastest.  This is the paper's "performance evaluator" (section 3.3: enumerate all valid
tuning-parameter combinations, prune the invalid ones, keep the best) applied to `peak_set_tuning`.

    python -m paper_2512_19018_b200.tune --dtype bf16_bf16 --layout NN -M 4096 -N 4096 -K 4096 [--seconds 0.3]
    python -m paper_2512_19018_b200.tune --sweep [--out FILE] [--seconds 0.15]

The second form walks the benchmark shape classes, searches each one's knob space by coordinate descent
(every value of one knob with the others held at the best found so far, two rounds, every improvement
confirmed by a second measurement of both contenders) and writes the persisted table the library loads
(tuned_sm100.json beside the shared object): one entry per shape class where a setting beats the built-in
rules by more than 1.5 %.

Knobs never change results, so the tuner only times; combinations a kernel family cannot run come back as
PEAK_ERR_UNSUPPORTED and are pruned.  Timing: CUDA events around back-to-back calls on rotating buffers.
"""
from __future__ import annotations

import argparse
import itertools
import json
import sys

DTYPES = {"f16_f32": 0, "bf16_bf16": 1, "f32_f32": 2, "f16_f16": 3, "bf16_f32": 4, "e4m3_bf16": 5, "e4m3_f32": 6,
          "e5m2_bf16": 7, "e5m2_f32": 8}

# knob -> candidate values (0 = library default); keys are peak_tuning_key_t
SPACE_16BIT = {
    "variant": ["umma_1cta", "umma_2cta"],
    1: [128, 256, 512],          # PEAK_TUNE_TILE_N
    2: [1, 2, 4, 8],             # PEAK_TUNE_SPLIT_K
    3: [1, 2],                   # PEAK_TUNE_EPILOGUE
    10: [1, 2],                  # PEAK_TUNE_MULTICAST
    0: [0, 2, 16],               # PEAK_TUNE_RASTER_GROUP
    12: [1, 2],                  # PEAK_TUNE_EPILOGUE_WARPS
}
SPACE_F32 = {
    "variant": ["sgemm"],
    4: [1, 2],                   # PEAK_TUNE_SGEMM_FMA
    7: [1, 2],                   # PEAK_TUNE_SGEMM_COPY
    0: [0, 4, 16],
}
NUM_KEYS = 20


def candidates(space: dict, quick: bool = False):
    """All combinations of the space as (variant name, {key: value}) pairs; `quick` keeps the first two values
    of every knob."""
    keys = [k for k in space if k != "variant"]
    lists = [space[k][:2] if quick else space[k] for k in keys]
    for variant in space["variant"]:
        for combo in itertools.product(*lists):
            yield variant, dict(zip(keys, combo))


def prune(variant: str, knobs: dict, M: int, N: int, K: int) -> bool:
    """Static pruning of combinations that cannot differ from another one or cannot run."""
    if variant == "umma_1cta" and (knobs.get(1) == 512 or knobs.get(10) == 2):
        return False                                   # 512-wide tiles and the multicast plug-in need CTA pairs
    if knobs.get(1, 0) == 128 and knobs.get(10) == 2:
        return False                                   # the plug-in runs 256- and 512-wide tiles
    if knobs.get(2, 1) > 1 and (knobs.get(1) == 512 or knobs.get(10) == 2):
        return False                                   # no k-split with wide tiles / plug-in
    if knobs.get(2, 1) > max(1, (K + 63) // 64):
        return False
    return True


# ------------------------------------------------------------------------------------------- sweep
# knob axes of the coordinate descent (0 = the built-in rule)
AXES_TENSOR = [
    ("variant", ["auto", "umma_2cta", "umma_1cta"]),
    (1, [0, 128, 256, 512]),        # PEAK_TUNE_TILE_N
    (10, [0, 1, 2]),                # PEAK_TUNE_MULTICAST
    (12, [0, 1, 2]),                # PEAK_TUNE_EPILOGUE_WARPS
    (0, [0, 1, 2, 4, 8, 16, 32]),   # PEAK_TUNE_RASTER_GROUP
    (2, [0, 1, 2, 3, 4, 8]),        # PEAK_TUNE_SPLIT_K
    (11, [0, 1]),                   # PEAK_TUNE_BALANCED_GRID
    (3, [0, 1, 2]),                 # PEAK_TUNE_EPILOGUE
    (13, [0, 1, 2]),                # PEAK_TUNE_K_ORDER
    (14, [0, 1, 2]),                # PEAK_TUNE_SWAP_AB
    (17, [0, 1]),                   # PEAK_TUNE_CLUSTER_K
]
AXES_F32 = [
    ("variant", ["auto"]),
    (7, [0, 1, 2, 3]),              # PEAK_TUNE_SGEMM_COPY
    (4, [0, 1, 2]),                 # PEAK_TUNE_SGEMM_FMA
    (0, [0, 2, 4, 8, 16, 32]),      # PEAK_TUNE_RASTER_GROUP
    (15, [0, 1, 2]),                # PEAK_TUNE_SGEMM_TRANSPOSE
]


def sweep_cases():
    """The benchmark shape classes the table is tuned on."""
    from . import workloads as W
    cases = [W.target_workload(), W.config1()]
    for n in (1024, 2048, 4096, 8192):
        cases += [W.config2(n, "NN"), W.config2(n, "TN")]
    cases += [W.config3(i) for i in range(3)] + [W.config4_ragged(i) for i in range(3)]
    cases += [W.config4_sgemm(4096), W.config4_sgemm(8192)]
    cases += [W.fp8_workload(8192, "e4m3", lay) for lay in ("NT", "NN")] + [W.fp8_workload(4096, "e4m3", "NT")]
    return cases


def entry_for(case, variant, knobs, tflops, default_tflops):
    e = {"in": case.in_type, "out": case.out_type, "layout": case.layout, "beta": 0 if case.beta == 0 else 1,
         "M": case.M, "N": case.N, "K": case.K, "knobs": {str(k): int(v) for k, v in sorted(knobs.items()) if v},
         "tflops": round(tflops, 1), "default_tflops": round(default_tflops, 1),
         "gain": round(tflops / default_tflops, 4), "workload": case.name}
    if variant != "auto":
        e["variant"] = variant
    return e


def sweep(out_path: str, seconds: float, only=None, min_gain: float = 1.015):
    import datetime
    import math

    import numpy as np
    import torch

    from . import binding as P
    from . import workloads as W

    P.load()
    P.peak_tuned_table_load(None)                      # tune against the built-in rules, not an older table
    variants = {"umma_1cta": P.PEAK_VARIANT_UMMA_1CTA, "umma_2cta": P.PEAK_VARIANT_UMMA_2CTA,
                "sgemm": P.PEAK_VARIANT_SGEMM, "auto": P.PEAK_VARIANT_AUTO}
    entries, log = [], []
    for case in sweep_cases():
        if only and case.name not in only:
            continue
        A_h, B_h, C_h = W.make_inputs(case, need_c0=True)

        def up(a, t):
            if t in ("f32", "e4m3", "e5m2"):
                return torch.from_numpy(a).cuda()
            return torch.from_numpy(a.view(np.int16)).cuda().view(torch.float16 if t == "f16" else torch.bfloat16)

        per_set = A_h.nbytes + B_h.nbytes + C_h.nbytes
        nsets = 1 if per_set > 3.8e8 else int(max(2, min(16, math.ceil(3.8e8 / per_set) + 1)))
        sets = [(up(A_h, case.in_type), up(B_h, case.in_type), up(C_h, case.out_type)) for _ in range(nsets)]
        del A_h, B_h, C_h

        def call(variant, i):
            A, B, C = sets[i % nsets]
            return P.peak_gemm_variant(variants[variant], case.dtype, case.transA, case.transB, case.M, case.N, case.K,
                                       case.alpha, A, case.lda, B, case.ldb, case.beta, C, case.ldc, check=False)

        def timed(variant, knobs, secs=seconds):
            for k in range(NUM_KEYS):
                P.peak_set_tuning(k, knobs.get(k, 0))
            if call(variant, 0) != P.PEAK_OK:
                return None
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(3):
                call(variant, i)
            e1.record()
            torch.cuda.synchronize()
            per = max(e0.elapsed_time(e1) / 3, 1e-3)
            steps = int(max(5, min(20000, secs * 1e3 / per)))
            e0.record()
            for i in range(steps):
                call(variant, i)
            e1.record()
            torch.cuda.synchronize()
            if P.peak_check()[0] != P.PEAK_OK:
                return None
            return e0.elapsed_time(e1) / steps

        def better(cand, inc):
            """cand = (variant, knobs) beats inc, measured twice each, alternating."""
            tc, ti = timed(*cand), timed(*inc)
            if tc is None or ti is None or tc > ti / 1.01:
                return False, tc, ti
            tc2, ti2 = timed(*cand), timed(*inc)
            return (tc2 is not None and ti2 is not None and tc2 < ti2 / 1.005), min(tc, tc2 or tc), min(ti, ti2 or ti)

        axes = AXES_F32 if case.in_type == "f32" else AXES_TENSOR
        timed("auto", {})                              # clocks and caches settle
        best = ("auto", {})
        for _round in range(2):
            changed = False
            for key, values in axes:
                for v in values:
                    cand_knobs = dict(best[1])
                    cand_variant = best[0]
                    if key == "variant":
                        if v == best[0]:
                            continue
                        cand_variant = v
                    else:
                        if cand_knobs.get(key, 0) == v:
                            continue
                        cand_knobs[key] = v
                    if cand_variant in ("umma_1cta", "umma_2cta") and not prune(cand_variant, cand_knobs, case.M, case.N, case.K):
                        continue
                    if cand_knobs.get(10) == 2 and not P.peak_multicast_available():
                        continue
                    ok, tc, ti = better((cand_variant, cand_knobs), best)
                    if ok:
                        best = (cand_variant, {k: x for k, x in cand_knobs.items() if x})
                        changed = True
            if not changed:
                break
        # final verdict against the built-in rules: four alternating pairs of longer measurements (under the power
        # cap two runs of the same kernel differ by a per cent or two, so single comparisons prove nothing); the
        # setting is kept when the median gain clears the threshold and no pair shows a loss
        if best != ("auto", {}):
            pairs = [(timed(best[0], best[1], 3 * seconds), timed("auto", {}, 3 * seconds)) for _ in range(4)]
            gains = sorted(a / b for b, a in pairs)
            tb, ta_ = float(np.median([b for b, _ in pairs])), float(np.median([a for _, a in pairs]))
            keep = 0.5 * (gains[1] + gains[2]) > min_gain and gains[0] > 1.0
        else:
            tb = ta_ = timed("auto", {}, 2 * seconds)
            keep = False
        tf_best, tf_auto = case.flops / (tb * 1e-3) / 1e12, case.flops / (ta_ * 1e-3) / 1e12
        log.append({"workload": case.name, "best": [best[0], {str(k): v for k, v in best[1].items()}],
                    "tflops": tf_best, "default_tflops": tf_auto, "kept": keep})
        print(json.dumps(log[-1]), file=sys.stderr, flush=True)
        if keep:
            entries.append(entry_for(case, best[0], best[1], tf_best, tf_auto))
        for k in range(NUM_KEYS):
            P.peak_set_tuning(k, 0)
        del sets
        torch.cuda.empty_cache()
    table = {"format": 1, "device": torch.cuda.get_device_name(0),
             "when": datetime.datetime.now(datetime.timezone.utc).strftime("%Y-%m-%dT%H:%M:%SZ"),
             "how": f"python -m paper_2512_19018_b200.tune --sweep --seconds {seconds}: coordinate descent per shape "
                    f"class, an entry only where the best setting beats the built-in rules by more than "
                    f"{(min_gain - 1) * 100:.1f} %; every other class stays on the built-in rules",
             "classes_tuned": [l["workload"] for l in log], "entries": entries}
    with open(out_path, "w") as f:
        json.dump(table, f, indent=1)
        f.write("\n")
    return table, log


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--sweep", action="store_true", help="tune every benchmark shape class and write the table")
    ap.add_argument("--out", default=None, help="where --sweep writes the table (default: beside the library)")
    ap.add_argument("--only", default="", help="--sweep: comma-separated workload names")
    ap.add_argument("--dtype", default="bf16_bf16", choices=sorted(DTYPES))
    ap.add_argument("--layout", default="NN", choices=["NN", "NT", "TN", "TT"])
    ap.add_argument("-M", type=int, default=4096)
    ap.add_argument("-N", type=int, default=4096)
    ap.add_argument("-K", type=int, default=4096)
    ap.add_argument("--alpha", type=float, default=1.0)
    ap.add_argument("--beta", type=float, default=0.0)
    ap.add_argument("--seconds", type=float, default=0.2, help="timed work per candidate")
    ap.add_argument("--quick", action="store_true")
    args = ap.parse_args(argv)
    if args.sweep:
        import os
        out = args.out or os.path.join(os.path.dirname(os.path.abspath(__file__)), "tuned_sm100.json")
        table, log = sweep(out, args.seconds if args.seconds != 0.2 else 0.15, [n for n in args.only.split(",") if n])
        print(json.dumps({"written": out, "entries": len(table["entries"]), "classes": len(log)}))
        return table

    import numpy as np
    import torch

    from . import binding as P
    from . import workloads as W

    dtype = DTYPES[args.dtype]
    ta, tb = args.layout[0] == "T", args.layout[1] == "T"
    case = W.GemmCase("tune", dtype, ta, tb, args.M, args.N, args.K, args.alpha, args.beta, "uniform")
    A_h, B_h, C_h = W.make_inputs(case, need_c0=True)

    def up(a, t):
        if t == "f32":
            return torch.from_numpy(a).cuda()
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.float16 if t == "f16" else torch.bfloat16)

    per_set = A_h.nbytes + B_h.nbytes + C_h.nbytes
    nsets = int(max(2, min(8, 4e8 // per_set + 1)))
    sets = [(up(A_h, case.in_type), up(B_h, case.in_type), up(C_h, case.out_type)) for _ in range(nsets)]
    variants = {"umma_1cta": P.PEAK_VARIANT_UMMA_1CTA, "umma_2cta": P.PEAK_VARIANT_UMMA_2CTA,
                "sgemm": P.PEAK_VARIANT_SGEMM, "auto": P.PEAK_VARIANT_AUTO}
    space = SPACE_F32 if case.in_type == "f32" else SPACE_16BIT

    def call(variant, i):
        A, B, C = sets[i % nsets]
        return P.peak_gemm_variant(variants[variant], dtype, ta, tb, case.M, case.N, case.K, case.alpha, A, case.lda,
                                   B, case.ldb, case.beta, C, case.ldc, check=False)

    def timed(variant, knobs):
        for k in range(NUM_KEYS):
            P.peak_set_tuning(k, knobs.get(k, 0))
        rc = call(variant, 0)
        if rc != P.PEAK_OK:
            return None
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(3):
            call(variant, i)
        e1.record()
        torch.cuda.synchronize()
        per = max(e0.elapsed_time(e1) / 3, 1e-3)
        steps = int(max(5, min(20000, args.seconds * 1e3 / per)))
        e0.record()
        for i in range(steps):
            call(variant, i)
        e1.record()
        torch.cuda.synchronize()
        if P.peak_check()[0] != P.PEAK_OK:
            return None
        return e0.elapsed_time(e1) / steps

    results = []
    timed("auto", {})                     # untimed pass: clocks and caches settle before the first measurement
    base = timed("auto", {})
    results.append(("auto", {}, base))
    for variant, knobs in candidates(space, args.quick):
        if not prune(variant, knobs, case.M, case.N, case.K):
            continue
        if variant.startswith("umma") and knobs.get(10) == 2 and not P.peak_multicast_available():
            continue
        ms = timed(variant, knobs)
        if ms is not None:
            results.append((variant, knobs, ms))
    again = timed("auto", {})             # the library's own choice once more, after all candidates
    if base is not None and again is not None:
        base = min(base, again)
        results[0] = ("auto", {}, base)
    for k in range(NUM_KEYS):
        P.peak_set_tuning(k, 0)
    results.sort(key=lambda r: r[2])
    best = results[0]
    out = {"shape": [case.M, case.N, case.K], "dtype": args.dtype, "layout": args.layout,
           "candidates_timed": len(results),
           "auto_ms": base, "auto_tflops": case.flops / (base * 1e-3) / 1e12 if base else None,
           "best": {"variant": best[0], "knobs": {str(k): v for k, v in best[1].items()}, "ms": best[2],
                    "tflops": case.flops / (best[2] * 1e-3) / 1e12},
           "top5": [{"variant": v, "knobs": {str(k): x for k, x in kn.items()}, "ms": ms} for v, kn, ms in results[:5]]}
    print(json.dumps(out))
    return out


if __name__ == "__main__":
    main()
    sys.exit(0)
