"""Fused epilogue tail (bias + activation, and the residual operand of peak_gemm_fused_residual), on every
kernel family, against the oracle (oracle.gemm followed by oracle.bias_act and oracle.residual_add).  Tolerance: the activation is Lipschitz with constant L (1 for
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


def make_residual(case, rng, pad=0, dist="normal"):
    """A residual matrix in the output's storage type: (stored bits on the host, pitch)."""
    ldr = case.N + pad
    vals = rng.standard_normal((case.M, ldr)).astype(np.float32) if dist == "normal" else \
        rng.integers(-8, 9, (case.M, ldr)).astype(np.float32)
    return W.encode(vals, case.out_type), ldr


def run_fused(case, variant, bias_h, act, res=None):
    dc = R.DeviceCase(case)
    bias_d = None if bias_h is None else torch.from_numpy(bias_h).cuda()
    if res is None:
        P.peak_gemm_fused(case.dtype, case.transA, case.transB, case.M, case.N, case.K, case.alpha, dc.A, case.lda, dc.B,
                          case.ldb, case.beta, dc.C, case.ldc, bias_d, act, variant=variant)
    else:
        r_h, ldr = res
        dc.R_d = R.to_device(r_h, case.out_type)
        P.peak_gemm_fused_residual(case.dtype, case.transA, case.transB, case.M, case.N, case.K, case.alpha, dc.A,
                                   case.lda, dc.B, case.ldb, case.beta, dc.C, case.ldc, bias_d, act, dc.R_d, ldr,
                                   variant=variant)
    rc, detail = P.peak_check()
    assert rc == P.PEAK_OK, hex(detail)
    return dc


def check_fused(dc, bias_h, act, what, res=None):
    c = dc.case
    pre, S = dc.oracle_full()
    ref = oracle.bias_act(pre, bias_h, act)
    r_abs = 0.0
    if res is not None:
        ref = oracle.residual_add(ref, res[0], R.OT[c.out_type], res[1])
        r_abs = np.abs(W.to_float64(res[0][:, :c.N], c.out_type))
    prebias = pre + (0 if bias_h is None else bias_h[None, :].astype(np.float64))
    c0 = R.c0_values(dc) if c.beta != 0 else 0.0
    sp = R.s_prime(c, S, c.alpha, c.beta, c0)
    tol = LIP[act] * (4 * max(c.K, 1) * 2.0 ** -24 * sp + 2.0 ** -22 * (0 if bias_h is None else np.abs(bias_h)[None, :])) \
        + 2.0 ** -21 * np.abs(prebias) + 2 * R.U_OUT[c.out_type] * np.abs(ref) + R.SUB_OUT[c.out_type] \
        + 2.0 ** -23 * (r_abs + np.abs(ref))          # the one fp32 addition of the residual
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


# ------------------------------------------------------------------ residual operand
@pytest.mark.parametrize("variant", VARIANTS_16)
@pytest.mark.parametrize("act", [P.PEAK_ACT_NONE, P.PEAK_ACT_GELU])
def test_residual_16bit_every_family(variant, act):
    """C = act(alpha*A*B + beta*C + bias) + R on the portable kernel and the tensor-core kernels: aligned and
    unaligned R, with and without beta and bias, ragged shapes, all output types."""
    rng = np.random.default_rng(17)
    for idx, (dtype, ta, tb, M, N, K, a, b, rpad) in enumerate([(W.PEAK_BF16_BF16, 0, 1, 300, 520, 264, 1.0, 0.0, 0),
                                                                (W.PEAK_F16_F32, 1, 0, 264, 257, 320, 0.5, 2.0, 3),
                                                                (W.PEAK_F16_F16, 0, 0, 128, 72, 136, -1.0, 1.0, 8),
                                                                (W.PEAK_BF16_F32, 1, 1, 520, 768, 200, 1.0, 0.0, 4)]):
        pa, pb = (-(M if ta else K)) % 8, (-(K if tb else N)) % 8
        c = W.GemmCase(f"res{idx}", dtype, bool(ta), bool(tb), M, N, K, a, b, "uniform", pad_a=pa, pad_b=pb,
                       pad_c=(0 if idx != 1 else 1), case=idx)
        bias = (rng.standard_normal(N) * 2).astype(np.float32) if idx % 2 == 0 else None
        res = make_residual(c, rng, rpad)
        dc = run_fused(c, variant, bias, act, res)
        check_fused(dc, bias, act, f"{c.name} act={act} variant={P.peak_variant_string(variant)}", res)


def test_residual_code_paths(reset_tuning):
    """Residual through split-K (reduce kernel), 512-wide tiles, 128-wide tiles, direct stores, two epilogue
    groups and the multicast plug-in; integer inputs, so the result must be exact."""
    rng = np.random.default_rng(18)
    c = W.GemmCase("res_paths", W.PEAK_BF16_F32, False, True, 768, 1024, 1024, 1.0, 1.0, "smallint")
    bias = rng.integers(-16, 17, c.N).astype(np.float32)
    res = make_residual(c, rng, 0, dist="int")
    settings = [{}, {P.PEAK_TUNE_SPLIT_K: 4}, {P.PEAK_TUNE_TILE_N: 512}, {P.PEAK_TUNE_EPILOGUE: 1}, {P.PEAK_TUNE_TILE_N: 128},
                {P.PEAK_TUNE_EPILOGUE_WARPS: 2}, {P.PEAK_TUNE_EPILOGUE: 3}]
    if P.peak_multicast_available():
        settings += [{P.PEAK_TUNE_MULTICAST: 2}, {P.PEAK_TUNE_MULTICAST: 2, P.PEAK_TUNE_TILE_N: 512}]
    for knobs in settings:
        for key in range(P.PEAK_TUNE_COUNT):
            P.peak_set_tuning(key, knobs.get(key, 0))
        for variant in (P.PEAK_VARIANT_UMMA_2CTA, P.PEAK_VARIANT_UMMA_1CTA):
            dc = run_fused(c, variant, bias, P.PEAK_ACT_RELU, res)
            pre, _ = dc.oracle_full()
            want = oracle.round_to(oracle.F32, oracle.residual_add(oracle.bias_act(pre, bias, oracle.ACT_RELU), res[0],
                                                                   oracle.F32, res[1]))
            assert np.array_equal(dc.result().view(np.uint32), want), f"knobs {knobs} variant {variant}"


@pytest.mark.parametrize("ta,tb", [(0, 0), (0, 1), (1, 0), (1, 1)])
def test_residual_sgemm(ta, tb, reset_tuning):
    rng = np.random.default_rng(19)
    for copy in (0, 1, 2, 3):
        P.peak_set_tuning(P.PEAK_TUNE_SGEMM_COPY, copy)
        c = W.GemmCase("res_sgemm", W.PEAK_F32_F32, bool(ta), bool(tb), 256, 384, 528, 0.5, 2.0, "uniform")
        bias = rng.standard_normal(c.N).astype(np.float32)
        res = make_residual(c, rng, 4)
        dc = run_fused(c, P.PEAK_VARIANT_SGEMM, bias, P.PEAK_ACT_GELU, res)
        check_fused(dc, bias, P.PEAK_ACT_GELU, f"sgemm {c.layout} copy={copy}", res)
    P.peak_set_tuning(P.PEAK_TUNE_SGEMM_COPY, 0)
    c = W.GemmCase("res_sgemm_ragged", W.PEAK_F32_F32, bool(ta), bool(tb), 200, 331, 100, 1.0, 0.0, "uniform",
                   pad_a=(-(200 if ta else 100)) % 4, pad_b=(-(100 if tb else 331)) % 4)
    res = make_residual(c, rng, 1)                    # unaligned residual rows
    dc = run_fused(c, P.PEAK_VARIANT_AUTO, None, P.PEAK_ACT_NONE, res)
    check_fused(dc, None, P.PEAK_ACT_NONE, f"sgemm ragged {c.layout}", res)


def test_residual_quick_returns_and_arguments():
    """alpha == 0: C = act(beta*C + bias) + R through the scaling kernel; a pitch below N is refused."""
    c = W.GemmCase("res_qr", W.PEAK_BF16_BF16, False, False, 96, 80, 64, 0.0, 0.5, "uniform")
    rng = np.random.default_rng(20)
    bias = rng.standard_normal(c.N).astype(np.float32)
    res = make_residual(c, rng, 2)
    dc = run_fused(c, P.PEAK_VARIANT_AUTO, bias, P.PEAK_ACT_RELU, res)
    c0 = R.c0_values(dc)
    pre = 0.5 * c0
    want = oracle.residual_add(oracle.bias_act(pre, bias, oracle.ACT_RELU), res[0], oracle.BF16, res[1])
    got = W.to_float64(dc.result(), "bf16")
    assert np.all(np.abs(got - want) <= 2.0 ** -8 * np.abs(want) + 1e-6)
    rc = P.peak_gemm_fused_residual(c.dtype, 0, 0, c.M, c.N, c.K, 1.0, dc.A, c.lda, dc.B, c.ldb, 0.0, dc.C, c.ldc, None,
                                    0, dc.R_d, c.N - 1, check=False)
    assert rc == P.PEAK_ERR_INVALID_VALUE
