"""Fused epilogue tail (bias + activation) of peak_gemm_fused, on every kernel family, against the oracle
(oracle.gemm followed by oracle.bias_act).  Tolerance: the activation is Lipschitz with constant L (1 for
identity / ReLU, below 1.13 for GELU), so an error e in the pre-activation value costs at most L*e; on top
come the fp32 evaluation of bias add and erff (a few ulp of the pre-activation value) and the one output
rounding:   |C - ref| <= L * (4 K 2^-24 S' + 2^-22 |bias|) + 2^-21 |pre| + 2 u_out |ref| + tiny."""
import numpy as np
import pytest
import torch

import oracle
from paper_2512_19018_b200 import binding as P
from paper_2512_19018_b200 import workloads as W
from tests import parity as R

pytestmark = pytest.mark.gpu
LIP = {P.PEAK_ACT_NONE: 1.0, P.PEAK_ACT_RELU: 1.0, P.PEAK_ACT_GELU: 1.13}


@pytest.fixture
def reset_tuning():
    yield
    for key in range(P.PEAK_TUNE_COUNT):
        P.peak_set_tuning(key, 0)


def run_fused(case, variant, bias_h, act):
    dc = R.DeviceCase(case)
    bias_d = None if bias_h is None else torch.from_numpy(bias_h).cuda()
    P.peak_gemm_fused(case.dtype, case.transA, case.transB, case.M, case.N, case.K, case.alpha, dc.A, case.lda, dc.B,
                      case.ldb, case.beta, dc.C, case.ldc, bias_d, act, variant=variant)
    rc, detail = P.peak_check()
    assert rc == P.PEAK_OK, hex(detail)
    return dc


def check_fused(dc, bias_h, act, what):
    c = dc.case
    pre, S = dc.oracle_full()
    ref = oracle.bias_act(pre, bias_h, act)
    prebias = pre + (0 if bias_h is None else bias_h[None, :].astype(np.float64))
    c0 = R.c0_values(dc) if c.beta != 0 else 0.0
    sp = R.s_prime(c, S, c.alpha, c.beta, c0)
    tol = LIP[act] * (4 * max(c.K, 1) * 2.0 ** -24 * sp + 2.0 ** -22 * (0 if bias_h is None else np.abs(bias_h)[None, :])) \
        + 2.0 ** -21 * np.abs(prebias) + 2 * R.U_OUT[c.out_type] * np.abs(ref) + R.SUB_OUT[c.out_type]
    got = W.to_float64(dc.result(), c.out_type)
    err = np.abs(got - ref)
    assert not np.isnan(got).any(), what
    bad = err > tol
    if bad.any():
        k = np.unravel_index(np.argmax(err - tol), err.shape)
        raise AssertionError(f"{what}: {bad.sum()} beyond the bound; worst at {k}: got {got[k]} ref {ref[k]} "
                             f"err {err[k]:.3e} tol {tol[k]:.3e}")


VARIANTS_16 = [P.PEAK_VARIANT_FALLBACK, P.PEAK_VARIANT_UMMA_1CTA, P.PEAK_VARIANT_UMMA_2CTA, P.PEAK_VARIANT_AUTO]


@pytest.mark.parametrize("variant", VARIANTS_16)
@pytest.mark.parametrize("act", [P.PEAK_ACT_NONE, P.PEAK_ACT_RELU, P.PEAK_ACT_GELU])
def test_fused_tail_16bit(variant, act):
    rng = np.random.default_rng(7)
    for idx, (dtype, ta, tb, M, N, K, a, b) in enumerate([(W.PEAK_BF16_BF16, 0, 1, 300, 520, 264, 1.0, 0.0),
                                                          (W.PEAK_F16_F32, 1, 0, 264, 257, 320, 0.5, 2.0),
                                                          (W.PEAK_BF16_F32, 0, 0, 128, 72, 136, -1.0, 1.0)]):
        pa, pb = (-(M if ta else K)) % 8, (-(K if tb else N)) % 8
        c = W.GemmCase(f"fused{idx}", dtype, bool(ta), bool(tb), M, N, K, a, b, "uniform", pad_a=pa, pad_b=pb, pad_c=idx,
                       case=idx)
        bias = (rng.standard_normal(N) * 2).astype(np.float32) if idx != 2 else None
        dc = run_fused(c, variant, bias, act)
        check_fused(dc, bias, act, f"{c.name} act={act} variant={P.peak_variant_string(variant)}")


@pytest.mark.parametrize("act", [P.PEAK_ACT_RELU, P.PEAK_ACT_GELU])
def test_fused_tail_code_paths(act, reset_tuning):
    """The same tail through split-K (reduce kernel), 512-wide tiles, the multicast plug-in and direct stores."""
    rng = np.random.default_rng(8)
    c = W.GemmCase("fused_paths", W.PEAK_BF16_BF16, False, True, 768, 1024, 1024, 1.0, 1.0, "uniform")
    bias = rng.standard_normal(c.N).astype(np.float32)
    settings = [{P.PEAK_TUNE_SPLIT_K: 4}, {P.PEAK_TUNE_TILE_N: 512}, {P.PEAK_TUNE_EPILOGUE: 1}, {P.PEAK_TUNE_TILE_N: 128}]
    if P.peak_multicast_available():
        settings.append({P.PEAK_TUNE_MULTICAST: 2})
    for knobs in settings:
        for key in range(P.PEAK_TUNE_COUNT):
            P.peak_set_tuning(key, knobs.get(key, 0))
        dc = run_fused(c, P.PEAK_VARIANT_UMMA_2CTA, bias, act)
        check_fused(dc, bias, act, f"knobs {knobs} act={act}")


@pytest.mark.parametrize("ta,tb", [(0, 0), (0, 1), (1, 0), (1, 1)])
def test_fused_tail_sgemm(ta, tb):
    rng = np.random.default_rng(9)
    c = W.GemmCase("fused_sgemm", W.PEAK_F32_F32, bool(ta), bool(tb), 256, 384, 528, 0.5, 2.0, "uniform")
    bias = rng.standard_normal(c.N).astype(np.float32)
    for act in (P.PEAK_ACT_RELU, P.PEAK_ACT_GELU):
        dc = run_fused(c, P.PEAK_VARIANT_SGEMM, bias, act)
        check_fused(dc, bias, act, f"sgemm {c.layout} act={act}")


def test_fused_tail_exact_with_integers():
    """Integer A, B, C0 and bias with ReLU: every value is an exactly representable integer, so the output
    must equal the oracle's correctly rounded result bit for bit on every tensor-core variant."""
    rng = np.random.default_rng(10)
    for variant in (P.PEAK_VARIANT_UMMA_1CTA, P.PEAK_VARIANT_UMMA_2CTA, P.PEAK_VARIANT_FALLBACK):
        c = W.GemmCase("fused_int", W.PEAK_BF16_F32, False, False, 512, 512, 256, 1.0, -1.0, "smallint")
        bias = rng.integers(-64, 65, c.N).astype(np.float32)
        dc = run_fused(c, variant, bias, P.PEAK_ACT_RELU)
        pre, _ = dc.oracle_full()
        want = oracle.round_to(oracle.F32, oracle.bias_act(pre, bias, oracle.ACT_RELU))
        assert np.array_equal(dc.result().view(np.uint32), want)


def test_fused_quick_returns():
    """K == 0 or alpha == 0: the result is act(beta*C + bias); with no bias, no activation and beta == 1
    nothing is touched."""
    c = W.GemmCase("fused_qr", W.PEAK_F16_F32, False, False, 96, 80, 64, 1.0, 0.5, "uniform")
    rng = np.random.default_rng(11)
    bias = rng.standard_normal(c.N).astype(np.float32)
    dc = R.DeviceCase(c)
    c0 = R.c0_values(dc)
    bias_d = torch.from_numpy(bias).cuda()
    P.peak_gemm_fused(c.dtype, 0, 0, c.M, c.N, 0, 1.0, None, c.lda, None, c.ldb, 0.5, dc.C, c.ldc, bias_d, P.PEAK_ACT_RELU)
    torch.cuda.synchronize()
    want = np.maximum((np.float32(0.5) * c0.astype(np.float32) + bias[None, :]), 0).astype(np.float32)
    assert np.array_equal(dc.result(), want)
    rc = P.peak_gemm_fused(c.dtype, 0, 0, c.M, c.N, c.K, 1.0, dc.A, c.lda, dc.B, c.ldb, 0.0, dc.C, c.ldc, None, 9,
                           check=False)
    assert rc == P.PEAK_ERR_INVALID_VALUE
