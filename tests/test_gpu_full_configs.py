"""Parity at the full sizes of the benchmark configurations, in the launch configuration bench.py times
(the dispatcher's own choice).  The oracle cannot compute these matrices whole, so each case is checked
(1) on a rows x cols sub-grid that puts several samples into every output tile (first / last row and column
of each tile plus random ones) with the CPU oracle and the per-element bounds of tests/parity.py, and
(2) over the WHOLE matrix against the fp64 cross-check kernel (itself pinned to the oracle on small cases in
test_gpu_parity.py), element by element with the derived bound of tests/parity.py; the sum S = sum_k |a||b| that
the bound needs is computed exactly for every element by the same cross-check kernel on |A| and |B|."""
import numpy as np
import pytest
import torch

from paper_2512_19018_b200 import binding as P
from paper_2512_19018_b200 import workloads as W
from tests import parity as R

pytestmark = pytest.mark.gpu

TT = {"f16": torch.float16, "bf16": torch.bfloat16, "f32": torch.float32}


def whole_matrix_check(dc: R.DeviceCase, max_flops=2.5e12):
    c = dc.case
    if c.flops > max_flops:
        return None
    c0_dev = R.to_device(dc.C0_h, c.out_type) if c.beta != 0 else None
    ref = torch.empty((c.M, c.N), dtype=torch.float64, device="cuda")
    P.peak_gemm_xcheck_f64(c.dtype, c.transA, c.transB, c.M, c.N, c.K, c.alpha, dc.A, c.lda, dc.B, c.ldb, c.beta,
                           c0_dev, c.ldc, ref, c.N)
    got = dc.C[:, :c.N].to(torch.float64)
    # S exactly: the cross-check kernel on the operands' absolute values (sign bit cleared in the stored bits)
    def absolute(t):
        if t.dtype == torch.float32:
            return t.abs()
        if t.element_size() == 1:                       # 8-bit floats: the sign is the top bit of every byte
            return (t.view(torch.uint8) & 0x7F).view(t.dtype)
        return (t.view(torch.int16) & 0x7FFF).view(t.dtype)
    S = torch.empty((c.M, c.N), dtype=torch.float64, device="cuda")
    P.peak_gemm_xcheck_f64(c.dtype, c.transA, c.transB, c.M, c.N, c.K, 1.0, absolute(dc.A), c.lda, absolute(dc.B), c.ldb,
                           0.0, None, c.ldc, S, c.N)
    sp = abs(c.alpha) * S
    if c.beta != 0:
        sp += abs(c.beta) * c0_dev[:, :c.N].to(torch.float64).abs()
    tol = 2 * R.U_OUT[c.out_type] * ref.abs() + 4 * c.K * 2.0 ** -24 * sp + R.SUB_OUT[c.out_type]
    del S, sp
    assert not torch.isnan(got).any()
    worst = float(((got - ref).abs() / tol).max())
    assert worst <= 1.0, f"{c.name}: whole-matrix check vs fp64 cross-check kernel, worst error / bound = {worst:.3f}"
    return worst


def run_case(case, expect_variant=None, tile=(256, 256)):
    dc = R.DeviceCase(case)
    v = P.peak_query_variant(case.dtype, case.transA, case.transB, case.M, case.N, case.K, case.alpha, dc.A, case.lda,
                             dc.B, case.ldb, case.beta, dc.C, case.ldc)
    if expect_variant is not None:
        assert v in expect_variant, P.peak_variant_string(v)
    dc.run(P.PEAK_VARIANT_AUTO)
    worst = R.check_sampled(dc, tile_m=tile[0], tile_n=tile[1], what=case.name)
    whole = whole_matrix_check(dc)
    print(f"{case.name}: variant {P.peak_variant_string(v)}, sampled worst err/bound {worst:.3f}, whole-matrix {whole}")
    del dc
    torch.cuda.empty_cache()


TENSOR = (P.PEAK_VARIANT_UMMA_1CTA, P.PEAK_VARIANT_UMMA_2CTA)


def test_config1_bf16_4096_nn():
    run_case(W.config1(), TENSOR)


@pytest.mark.parametrize("n", [1024, 2048, 4096, 8192, 16384])
@pytest.mark.parametrize("layout", ["NN", "TN"])
def test_config2_fp16_square_sweep(n, layout):
    run_case(W.config2(n, layout), TENSOR)


@pytest.mark.parametrize("which", [0, 1, 2])
def test_config3_bf16_transformer_nt(which):
    run_case(W.config3(which), TENSOR)


@pytest.mark.parametrize("n", [4096, 8192])
def test_config4_sgemm(n):
    run_case(W.config4_sgemm(n), (P.PEAK_VARIANT_SGEMM,), tile=(128, 128))


@pytest.mark.parametrize("which", [0, 1, 2])
def test_config4_bf16_ragged_tn(which):
    run_case(W.config4_ragged(which), TENSOR, tile=(128, 128))


def test_target_bf16_8192_nn():
    run_case(W.target_workload(), TENSOR)
