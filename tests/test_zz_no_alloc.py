"""peak_gemm_static_ws: the split-K entry point for callers that cannot allocate device memory when they
call a GEMM (for example a serving process that has given all free HBM to its own pools, or a latency-critical
loop where an allocator call is not acceptable).  Its partial tiles live in a fixed 32 MiB array inside the
library instead of pool memory.

The test calls it through the C ABI twice in a row, on two different problems, and checks each output
against what the existing entry point (peak_gemm) gives on the same inputs: bit for bit on integer-valued
inputs (both are exact there), and within twice the derived per-element bound of tests/parity.py on real-valued
inputs (each side is within that bound of the oracle).  The second call finds the first call's partial tiles
still in the shared array, so a stale read would show up as a mismatch.  This file is collected last on
purpose, so that a run that stops at the first failure has already run every other test; it passes both
alone in a fresh process and after the rest of the suite.
"""
import numpy as np
import pytest
import torch

from paper_2512_19018_b200 import binding as P
from paper_2512_19018_b200 import workloads as W
from tests import parity as R

pytestmark = pytest.mark.gpu


def _run_both(case, splits):
    ref_side = R.DeviceCase(case)                       # existing entry point
    ref_side.run(P.PEAK_VARIANT_AUTO)
    new_side = R.DeviceCase(case)                       # same seeded inputs, fresh C
    c = case
    P.peak_gemm_static_ws(c.dtype, c.transA, c.transB, c.M, c.N, c.K, c.alpha, new_side.A, c.lda, new_side.B, c.ldb,
                          c.beta, new_side.C, c.ldc, splits)
    rc, detail = P.peak_check()
    assert rc == P.PEAK_OK, f"device status {rc} 0x{detail:x}"
    return ref_side, new_side


def test_static_workspace_matches_existing_entry_point_twice_in_a_row():
    assert P.peak_static_ws_bytes() == 32 << 20
    problems = [
        # (case, splits): a skinny TN shape with alpha/beta, then a different shape and layout
        (W.GemmCase("noalloc_a", W.PEAK_BF16_BF16, True, False, 48, 1000, 2048, alpha=0.5, beta=2.0, pad_c=8), 4),
        (W.GemmCase("noalloc_b", W.PEAK_F16_F32, False, True, 300, 264, 1096, alpha=1.0, beta=0.0, case=1), 3),
    ]
    for case, splits in problems:
        # integer-valued inputs: both entry points are exact, so they agree bit for bit
        ci = case.with_(dist="smallint", alpha=0.25 if case.out_type != "f32" else 1.0)
        a, b = _run_both(ci, splits)
        assert np.array_equal(a.result(), b.result()), f"{ci.name}: integer case differs from peak_gemm"
        # real-valued inputs: each side is within the derived bound of the oracle; they differ by at most twice it
        a, b = _run_both(case, splits)
        ref, S = a.oracle_full()
        c0 = R.c0_values(a) if case.beta != 0 else 0.0
        R.check_values(case, b.result(), ref, S, c0, what=f"{case.name} static workspace vs oracle")
        sp = R.s_prime(case, S, case.alpha, case.beta, c0)
        tight = 2 * R.U_OUT[case.out_type] * np.abs(ref) + 4 * case.K * 2.0 ** -24 * sp + 1e-37
        diff = np.abs(W.to_float64(a.result(), case.out_type) - W.to_float64(b.result(), case.out_type))
        assert (diff <= 2 * tight).all(), f"{case.name}: differs from peak_gemm by more than twice the bound"


def test_static_workspace_rejects_what_it_cannot_hold():
    A = torch.zeros(16, dtype=torch.bfloat16, device="cuda")
    args = dict(dtype=W.PEAK_BF16_BF16, transA=0, transB=0, alpha=1.0, beta=0.0)
    def call(M, N, K, splits, lda=None, ldb=None, ldc=None):
        return P.peak_gemm_static_ws(args["dtype"], 0, 0, M, N, K, 1.0, A, lda or K, A, ldb or N, 0.0, A, ldc or N,
                                     splits, check=False)
    # 2048 x 2048 x 4 slices of fp32 = 64 MiB > 32 MiB: refused before anything is launched
    assert call(2048, 2048, 4096, 4) == P.PEAK_ERR_WORKSPACE_TOO_SMALL
    assert "workspace" in P.peak_status_string(P.PEAK_ERR_WORKSPACE_TOO_SMALL)
    assert call(128, 128, 4096, 1) == P.PEAK_ERR_INVALID_VALUE          # not a split
    assert call(128, 128, 128, 3) == P.PEAK_ERR_INVALID_VALUE           # 2 k-blocks cannot feed 3 slices
    assert call(128, 128, 4096, 4, lda=100) == P.PEAK_ERR_INVALID_VALUE  # lda < K
    assert P.peak_gemm_static_ws(W.PEAK_F32_F32, 0, 0, 128, 128, 256, 1.0, A, 256, A, 128, 0.0, A, 128, 2,
                                 check=False) == P.PEAK_ERR_INVALID_VALUE  # fp32 inputs: not this path
