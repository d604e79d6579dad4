"""The dispatcher's own choices over a few hundred seeded random problems -- skinny, few-tile, one-wave, multi-wave,
long-K, short-K with large outputs; every tensor-core type pair, layout, ragged sizes, alpha / beta -- checked over the WHOLE output against the
fp64 cross-check kernel (itself pinned to the oracle on small cases in test_gpu_parity.py) with the per-element bound
of tests/parity.py.  Complements the hand-picked shapes of the other files: whatever kernel, tile width, k-split or
cluster shape the rules pick for a shape nobody thought of must still be right."""
import numpy as np
import pytest
import torch

from paper_2512_19018_b200 import binding as P
from paper_2512_19018_b200 import workloads as W
from tests import parity as R
from tests.test_gpu_full_configs import whole_matrix_check

pytestmark = pytest.mark.gpu

TYPES = [W.PEAK_BF16_BF16, W.PEAK_F16_F32, W.PEAK_F16_F16, W.PEAK_BF16_F32, W.PEAK_E4M3_BF16, W.PEAK_E5M2_F32, W.PEAK_F32_F32]


def draw(rng, cls):
    if cls == 0:     # skinny
        return int(rng.integers(1, 130)), int(rng.integers(64, 15000)), int(rng.integers(64, 9000))
    if cls == 1:     # a few row blocks, long K
        return int(rng.integers(129, 1100)), int(rng.integers(256, 5000)), int(rng.integers(512, 6000))
    if cls == 2:     # one or two waves
        return int(rng.integers(256, 2600)), int(rng.integers(256, 2600)), int(rng.integers(64, 3000))
    if cls == 3:     # tiny outputs, very long K
        return int(rng.integers(1, 600)), int(rng.integers(1, 600)), int(rng.integers(1, 20000))
    if cls == 4:     # several waves
        return int(rng.integers(1000, 4200)), int(rng.integers(1000, 4200)), int(rng.integers(1000, 4200))
    if cls == 5:     # very wide, few rows
        return int(rng.integers(1, 300)), int(rng.integers(2000, 30000)), int(rng.integers(1000, 5000))
    # several waves of tiles with few k-blocks: the epilogue bounds the launch
    return int(rng.integers(1500, 6000)), int(rng.integers(1500, 6000)), int(rng.integers(8, 700))


@pytest.mark.parametrize("seed", [5, 6])
def test_dispatcher_choices_whole_matrix(seed):
    rng = np.random.default_rng(seed)
    kernels = set()
    done = 0
    worst = 0.0
    while done < 160:
        dt = TYPES[int(rng.integers(len(TYPES)))]
        M, N, K = draw(rng, int(rng.integers(7)))
        if dt == W.PEAK_F32_F32:
            M, N, K = min(M, 1500), min(N, 3000), min(K, 3000)      # the CUDA-core path is 20 times slower
        if 2.0 * M * N * K > 1.2e12:
            continue
        ta, tb = int(rng.integers(2)), int(rng.integers(2))
        unit = 16 if W.IN_TYPE[dt] in ("e4m3", "e5m2") else (4 if dt == W.PEAK_F32_F32 else 8)
        pa, pb = (-(M if ta else K)) % unit, (-(K if tb else N)) % unit
        c = W.GemmCase(f"d{seed}_{done}", dt, bool(ta), bool(tb), M, N, K, float(rng.choice([1.0, 0.5, -1.0, 2.0])),
                       float(rng.choice([0.0, 0.0, 1.0, -0.5])), "uniform", pad_a=pa, pad_b=pb,
                       pad_c=int(rng.choice([0, 0, 8, 3])), case=1000 * seed + done)
        dc = R.DeviceCase(c)
        dc.run(P.PEAK_VARIANT_AUTO)
        kernels.add(P.peak_last_kernel().split(" grid")[0].split(" (")[0])
        w = whole_matrix_check(dc, max_flops=2e12)
        assert w is not None
        worst = max(worst, w)
        done += 1
        del dc
        if done % 40 == 0:
            torch.cuda.empty_cache()
    print(f"seed {seed}: {done} problems, {len(kernels)} different kernels, worst error / bound {worst:.3f}")
    assert len(kernels) >= 12            # the draw reaches the kernel families it is meant to reach
