"""Randomised differential test: seeded random shapes, type pairs, layouts, pitches (TMA-friendly and not),
alpha/beta, kernel families and tuning knobs, each compared with the CPU oracle under the usual bounds (and
the guard bands of tests/parity.py).  Small sizes, so that the oracle keeps up; the point is the cross
product of code paths (ragged edges x k-splits x epilogue paths x warp groups x tile widths x plug-in)."""
import numpy as np
import pytest

from paper_2512_19018_b200 import binding as P
from paper_2512_19018_b200 import workloads as W
from tests import parity as R

pytestmark = pytest.mark.gpu

DTYPES = [W.PEAK_F16_F32, W.PEAK_BF16_BF16, W.PEAK_F16_F16, W.PEAK_BF16_F32, W.PEAK_F32_F32, W.PEAK_E4M3_BF16,
          W.PEAK_E4M3_F32, W.PEAK_E5M2_BF16, W.PEAK_E5M2_F32]


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_cases_against_the_oracle(seed):
    rng = np.random.default_rng(seed)
    done = 0
    try:
        for n in range(400):
            dt = DTYPES[rng.integers(len(DTYPES))]
            ta, tb = int(rng.integers(2)), int(rng.integers(2))
            big = rng.random() < 0.15
            M = int(rng.integers(1, 1400 if big else 420))
            N = int(rng.integers(1, 1400 if big else 420))
            K = int(rng.integers(1, 2200 if big else 600))
            in8 = W.IN_TYPE[dt] in ("e4m3", "e5m2")
            unit = 16 if in8 else (4 if dt == W.PEAK_F32_F32 else 8)
            if rng.random() < 0.75:      # pitches the copy engine accepts
                pa, pb = (-(M if ta else K)) % unit, (-(K if tb else N)) % unit
                if rng.random() < 0.3:
                    pa, pb = pa + unit, pb + 2 * unit
                pc = int(rng.choice([0, 0, 8, 3])) if rng.random() < 0.5 else (-N) % 8
            else:
                pa, pb, pc = int(rng.integers(0, 5)), int(rng.integers(0, 5)), int(rng.integers(0, 5))
            alpha = float(rng.choice([1.0, 0.5, -1.0, 2.0]))
            beta = float(rng.choice([0.0, 0.0, 1.0, 2.0, -0.5]))
            dist = str(rng.choice(["uniform", "smallint", "uniform"]))
            c = W.GemmCase(f"r{seed}_{n}", dt, bool(ta), bool(tb), M, N, K, alpha, beta, dist, pad_a=pa, pad_b=pb,
                           pad_c=pc, case=1000 * seed + n)
            knobs = {P.PEAK_TUNE_TILE_N: int(rng.choice([0, 0, 128, 256, 512, 192, 384])),
                     P.PEAK_TUNE_EPILOGUE: int(rng.choice([0, 0, 1, 2, 3])),
                     P.PEAK_TUNE_EPILOGUE_WARPS: int(rng.choice([0, 1, 2])),
                     P.PEAK_TUNE_SPLIT_K: int(rng.choice([0, 0, 0, 1, 2, 3])),
                     P.PEAK_TUNE_MULTICAST: int(rng.choice([0, 0, 1, 2])),
                     P.PEAK_TUNE_RASTER_GROUP: int(rng.choice([0, 0, 1, 3])),
                     P.PEAK_TUNE_TAIL_SPLIT: int(rng.choice([0, 0, 2])),
                     P.PEAK_TUNE_BALANCED_GRID: int(rng.choice([0, 1])),
                     P.PEAK_TUNE_K_ORDER: int(rng.choice([0, 1, 2])),
                     P.PEAK_TUNE_SWAP_AB: int(rng.choice([0, 0, 1, 2])),
                     P.PEAK_TUNE_SGEMM_TRANSPOSE: int(rng.choice([0, 1, 2])),
                     P.PEAK_TUNE_SHORT_A: int(rng.choice([0, 0, 1])),
                     P.PEAK_TUNE_CLUSTER_K: int(rng.choice([0, 0, 1, 2, 3, 4]))}
            for k, v in knobs.items():
                P.peak_set_tuning(k, v)
            variant = int(rng.choice([P.PEAK_VARIANT_AUTO, P.PEAK_VARIANT_AUTO, P.PEAK_VARIANT_UMMA_1CTA,
                                      P.PEAK_VARIANT_UMMA_2CTA, P.PEAK_VARIANT_FALLBACK]))
            dc = R.DeviceCase(c)
            try:
                dc.run(variant)
            except P.PeakError as e:
                if e.status == P.PEAK_ERR_UNSUPPORTED and variant != P.PEAK_VARIANT_AUTO:
                    continue             # a forced family that cannot run this problem says so; nothing was written
                raise
            R.check_full(dc, what=f"{c} knobs={knobs} variant={variant}")
            done += 1
    finally:
        for k in range(P.PEAK_TUNE_COUNT):
            P.peak_set_tuning(k, 0)
    assert done > 250


def test_random_multi_wave_cases_sampled():
    """The same idea at sizes of several tiles per CTA (ragged in every dimension, beta != 0 in half of the
    cases, back-to-back launches), compared with the oracle on a sampled grid that touches every tile."""
    rng = np.random.default_rng(21)
    types = [W.PEAK_F16_F32, W.PEAK_BF16_BF16, W.PEAK_F16_F16, W.PEAK_BF16_F32, W.PEAK_E4M3_BF16, W.PEAK_E5M2_F32]
    P.peak_set_tuning(P.PEAK_TUNE_WAIT_MS, 200)       # a lost hand-over shows up quickly instead of after seconds
    try:
        for n in range(80):
            dt = types[rng.integers(len(types))]
            in8 = W.IN_TYPE[dt] in ("e4m3", "e5m2")
            ta, tb = int(rng.integers(2)), int(rng.integers(2))
            M = int(rng.integers(1, 40)) * 128 + int(rng.choice([0, 0, 8, 56]))
            N = int(rng.integers(1, 40)) * 128 + int(rng.choice([0, 0, 8, 72]))
            K = int(rng.integers(1, 40)) * 64 + int(rng.choice([0, 0, 16, 40]))
            unit = 16 if in8 else 8
            c = W.GemmCase(f"m{n}", dt, bool(ta), bool(tb), M, N, K, float(rng.choice([1.0, 0.5])),
                           float(rng.choice([0.0, 0.0, 1.0, 2.0])), "uniform", pad_a=(-(M if ta else K)) % unit,
                           pad_b=(-(K if tb else N)) % unit, pad_c=int(rng.choice([0, 0, 8])), case=5000 + n)
            knobs = {P.PEAK_TUNE_TILE_N: int(rng.choice([0, 0, 0, 256, 512])),
                     P.PEAK_TUNE_EPILOGUE: int(rng.choice([0, 0, 0, 1, 3])),
                     P.PEAK_TUNE_EPILOGUE_WARPS: int(rng.choice([0, 0, 1, 2])),
                     P.PEAK_TUNE_MULTICAST: int(rng.choice([0, 0, 1, 2])),
                     P.PEAK_TUNE_RASTER_GROUP: int(rng.choice([0, 0, 2, 16])),
                     P.PEAK_TUNE_BALANCED_GRID: int(rng.choice([0, 1])),
                     P.PEAK_TUNE_K_ORDER: int(rng.choice([0, 1, 2])),
                     P.PEAK_TUNE_DEPENDENT_LAUNCH: int(rng.choice([0, 0, 1]))}
            for k, v in knobs.items():
                P.peak_set_tuning(k, v)
            dc = R.DeviceCase(c)
            for _ in range(2):
                dc.reset_c()
                dc.run(P.PEAK_VARIANT_AUTO)
            R.check_sampled(dc, tile_m=128, tile_n=128, budget_macs=2e7, what=f"{c} knobs={knobs}")
    finally:
        for k in range(P.PEAK_TUNE_COUNT):
            P.peak_set_tuning(k, 0)
