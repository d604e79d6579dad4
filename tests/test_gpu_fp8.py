"""GPU parity for 8-bit floating-point inputs (E4M3 / E5M2 operands, bf16 or fp32 output) against the CPU
oracle, whose decoders are written from the bit layout and pinned separately.  The tensor-core path takes all
four layouts (a K-major operand as one 128-byte swizzle row of K per matrix row, an MN-major one through the
major bit of the instruction descriptor); pitches that are not multiples of 16 bytes run on the portable
kernel."""
import numpy as np
import pytest

import oracle
from paper_2512_19018_b200 import binding as P
from paper_2512_19018_b200 import workloads as W
from tests import parity as R

pytestmark = pytest.mark.gpu

PAIRS_8 = [W.PEAK_E4M3_BF16, W.PEAK_E4M3_F32, W.PEAK_E5M2_BF16, W.PEAK_E5M2_F32]
LAYOUTS = [(0, 0), (0, 1), (1, 0), (1, 1)]
UMMA = [P.PEAK_VARIANT_UMMA_1CTA, P.PEAK_VARIANT_UMMA_2CTA]


def mk(dtype, ta, tb, M, N, K, **kw):
    return W.GemmCase(f"q{dtype}_{ta}{tb}_{M}x{N}x{K}", dtype, bool(ta), bool(tb), M, N, K, **kw)


def pad16(n):
    return (-n) % 16


def k_major(dtype, M, N, K, **kw):
    """A row-major M x K, B stored N x K (transB), pitches padded to 16 bytes as the TMA path needs."""
    return mk(dtype, 0, 1, M, N, K, pad_a=pad16(K), pad_b=pad16(K), **kw)


def any_layout(dtype, ta, tb, M, N, K, **kw):
    """Any layout with the pitches padded to 16 bytes, as the TMA path needs."""
    a_cols = M if ta else K
    b_cols = K if tb else N
    return mk(dtype, ta, tb, M, N, K, pad_a=pad16(a_cols), pad_b=pad16(b_cols), **kw)


@pytest.fixture
def reset_tuning():
    yield
    for key in range(P.PEAK_TUNE_COUNT):
        P.peak_set_tuning(key, 0)


def assert_bits_equal(c, dc, what):
    ref, _ = dc.oracle_full()
    want = oracle.round_to(R.OT[c.out_type], ref)
    got = dc.result()
    if c.out_type == "f32":
        got = got.view(np.uint32)
    if not np.array_equal(got, want):
        bad = np.argwhere(got != want)
        raise AssertionError(f"{what}: {len(bad)} of {got.size} wrong, first at {bad[0]}")


@pytest.mark.parametrize("dtype", PAIRS_8)
@pytest.mark.parametrize("ta,tb", LAYOUTS)
def test_fallback_fp8_any_layout_any_pitch(dtype, ta, tb):
    for (M, N, K, a, b) in [(1, 1, 1, 1.0, 0.0), (67, 130, 45, 0.5, 2.0), (128, 64, 200, -1.0, 1.0)]:
        c = mk(dtype, ta, tb, M, N, K, alpha=a, beta=b, pad_a=1, pad_b=3, pad_c=5, case=M)
        dc = R.DeviceCase(c)
        dc.run(P.PEAK_VARIANT_FALLBACK)
        R.check_full(dc)


def test_every_fp8_bit_pattern_decodes_as_the_oracle_does():
    """A = all 256 bit patterns minus the NaNs / infinities (one per row, K = 1), B = [1]: C = decode(A)."""
    for dtype, t in [(W.PEAK_E4M3_F32, "e4m3"), (W.PEAK_E5M2_F32, "e5m2")]:
        bits = np.arange(256, dtype=np.uint8)
        vals = oracle.decode(R.OT[t], bits)
        keep = np.isfinite(vals)
        a = np.zeros((256, 16), dtype=np.uint8)
        a[:, 0] = np.where(keep, bits, 0)
        one = W.encode(np.ones((1, 1), np.float32), t)
        b = np.zeros((16, 16), dtype=np.uint8)
        b[0, 0] = one[0, 0]
        import torch
        A, B = torch.from_numpy(a).cuda(), torch.from_numpy(b).cuda()
        for variant in [P.PEAK_VARIANT_FALLBACK] + UMMA:
            C = torch.full((256, 16), float("nan"), dtype=torch.float32, device="cuda")
            # K = 16 with zero padding so that the TMA pitch rule holds; B is N x K (transB)
            P.peak_gemm_variant(variant, dtype, 0, 1, 256, 16, 16, 1.0, A, 16, B, 16, 0.0, C, 16, None)
            rc, _ = P.peak_check(None)
            assert rc == P.PEAK_OK
            got = C.cpu().numpy()[:, 0].astype(np.float64)
            want = np.where(keep, vals, 0.0)
            assert np.array_equal(got, want), f"{t} {P.peak_variant_string(variant)}"
            assert (C.cpu().numpy()[:, 1:] == 0).all()


@pytest.mark.parametrize("variant", UMMA)
@pytest.mark.parametrize("dtype", PAIRS_8)
def test_umma_fp8_exact_small_integers(variant, dtype):
    """Entries in [-4, 4] are exact in both 8-bit formats; every partial sum is an integer below 2^24, so the
    result must equal the oracle's correctly rounded value bit for bit.  K spans one, several and a ragged
    number of 128-element k-blocks."""
    for (M, N, K) in [(128, 256, 128), (256, 512, 384), (384, 256, 512), (200, 328, 208), (130, 72, 48)]:
        c = k_major(dtype, M, N, K, dist="smallint", case=K)
        if c.out_type != "f32":
            c = c.with_(alpha=0.125)
        dc = R.DeviceCase(c)
        dc.run(variant)
        assert_bits_equal(c, dc, f"{c.name} {P.peak_variant_string(variant)}")


@pytest.mark.parametrize("variant", UMMA + [P.PEAK_VARIANT_AUTO])
@pytest.mark.parametrize("dtype", PAIRS_8)
def test_umma_fp8_ragged_alpha_beta(variant, dtype):
    for (M, N, K, a, b, dist) in [(300, 520, 1000, 1.0, 0.0, "uniform"), (129, 257, 4100, 0.5, 2.0, "uniform"),
                                  (512, 768, 2048, -1.0, 1.0, "transformer"), (64, 1000, 336, 2.0, 0.0, "normal_rsqrtk")]:
        c = k_major(dtype, M, N, K, alpha=a, beta=b, dist=dist, pad_c=pad16(N) + 8, case=K)
        dc = R.DeviceCase(c)
        dc.run(variant)
        R.check_full(dc, what=f"{c.name} {P.peak_variant_string(variant)}")


@pytest.mark.parametrize("variant", UMMA)
@pytest.mark.parametrize("dtype", [W.PEAK_E4M3_F32, W.PEAK_E5M2_BF16])
@pytest.mark.parametrize("ta,tb", LAYOUTS)
def test_umma_fp8_every_layout_exact_small_integers(variant, dtype, ta, tb):
    """All four layouts on the tensor cores: small integers, so that a wrong box, k-step or leading-dimension
    offset of an MN-major 8-bit operand (a dropped, repeated or misplaced k-row or column) changes the exact
    result.  Sizes cover one tile, several tiles and k-blocks, and ragged M, N and K."""
    for (M, N, K) in [(128, 256, 128), (256, 512, 384), (384, 256, 512), (200, 328, 208), (130, 72, 48),
                      (1000, 1100, 1300)]:
        c = any_layout(dtype, ta, tb, M, N, K, dist="smallint", case=K + 3 * ta + 5 * tb)
        if c.out_type != "f32":
            c = c.with_(alpha=0.125)
        dc = R.DeviceCase(c)
        dc.run(variant)
        assert_bits_equal(c, dc, f"{c.name} {c.layout} {P.peak_variant_string(variant)}")


@pytest.mark.parametrize("dtype", PAIRS_8)
@pytest.mark.parametrize("ta,tb", [(0, 0), (1, 0), (1, 1)])
def test_umma_fp8_mn_major_real_values(dtype, ta, tb, reset_tuning):
    """Real-valued inputs, alpha / beta, several tile widths and a k-split on the layouts with an MN-major
    operand; the dispatcher must pick a tensor-core kernel for them."""
    for tile_n, split in [(0, 0), (128, 0), (256, 3), (512, 0)]:
        P.peak_set_tuning(P.PEAK_TUNE_TILE_N, tile_n)
        P.peak_set_tuning(P.PEAK_TUNE_SPLIT_K, split)
        c = any_layout(dtype, ta, tb, 520, 1032, 3000 + 8, dist="uniform", alpha=0.75, beta=0.5, pad_c=8,
                       case=tile_n + split)
        for variant in UMMA + [P.PEAK_VARIANT_AUTO]:
            dc = R.DeviceCase(c)
            v = P.peak_query_variant(c.dtype, c.transA, c.transB, c.M, c.N, c.K, c.alpha, dc.A, c.lda, dc.B, c.ldb,
                                     c.beta, dc.C, c.ldc)
            assert v in UMMA, f"{c.layout}: dispatcher chose {P.peak_variant_string(v)}"
            dc.run(variant)
            assert "umma_gemm_kernel" in P.peak_last_kernel() or "umma_clusterk_kernel" in P.peak_last_kernel()
            R.check_full(dc, what=f"{c.name} {c.layout} bn{tile_n} split{split} {P.peak_variant_string(variant)}")


def test_fp8_every_bit_pattern_every_layout():
    """All finite bit patterns of both formats as A (one per row) against B = e_0, in every layout, on the
    tensor cores: the MN-major paths decode exactly as the oracle does."""
    import torch
    for dtype, t in [(W.PEAK_E4M3_F32, "e4m3"), (W.PEAK_E5M2_F32, "e5m2")]:
        bits = np.arange(256, dtype=np.uint8)
        vals = oracle.decode(R.OT[t], bits)
        keep = np.isfinite(vals)
        a = np.zeros((256, 32), dtype=np.uint8)          # op(A): 256 x 32, column 5 carries the patterns
        a[:, 5] = np.where(keep, bits, 0)
        one = W.encode(np.ones((1, 1), np.float32), t)[0, 0]
        b = np.zeros((32, 48), dtype=np.uint8)           # op(B): 32 x 48 with B[5, 7] = 1
        b[5, 7] = one
        want = np.where(keep, vals, 0.0)
        for ta, tb in LAYOUTS:
            As = np.ascontiguousarray(a.T if ta else a)
            Bs = np.ascontiguousarray(b.T if tb else b)
            A, B = torch.from_numpy(As).cuda(), torch.from_numpy(Bs).cuda()
            for variant in UMMA:
                C = torch.full((256, 48), float("nan"), dtype=torch.float32, device="cuda")
                P.peak_gemm_variant(variant, dtype, ta, tb, 256, 48, 32, 1.0, A, As.shape[1], B, Bs.shape[1], 0.0, C,
                                    48, None)
                rc, _ = P.peak_check(None)
                assert rc == P.PEAK_OK
                got = C.cpu().numpy().astype(np.float64)
                assert np.array_equal(got[:, 7], want), f"{t} {ta}{tb} {P.peak_variant_string(variant)}"
                got[:, 7] = 0
                assert (got == 0).all()


def test_fp8_unaligned_pitch_still_runs_on_the_portable_kernel():
    c = mk(W.PEAK_E4M3_BF16, 1, 0, 256, 256, 256, pad_a=3)
    dc = R.DeviceCase(c)
    with pytest.raises(P.PeakError):
        dc.run(P.PEAK_VARIANT_UMMA_2CTA)
    dc.run(P.PEAK_VARIANT_AUTO)
    assert "fallback" in P.peak_last_kernel()
    R.check_full(dc)


@pytest.mark.parametrize("dtype", [W.PEAK_E4M3_BF16, W.PEAK_E5M2_F32])
@pytest.mark.parametrize("tile_n,split", [(128, 0), (256, 3), (512, 0), (256, 0)])
def test_umma_fp8_tiles_and_split_k(dtype, tile_n, split, reset_tuning):
    P.peak_set_tuning(P.PEAK_TUNE_TILE_N, tile_n)
    P.peak_set_tuning(P.PEAK_TUNE_SPLIT_K, split)
    c = k_major(dtype, 512, 1024, 3000 + 8, dist="uniform", alpha=0.75, beta=0.5, case=tile_n + split)
    for variant in UMMA:
        dc = R.DeviceCase(c)
        dc.run(variant)
        R.check_full(dc, what=f"{c.name} bn{tile_n} split{split} {P.peak_variant_string(variant)}")


@pytest.mark.parametrize("dtype,ta,tb", [(W.PEAK_E4M3_BF16, 0, 1), (W.PEAK_E4M3_F32, 0, 1), (W.PEAK_E4M3_BF16, 0, 0),
                                         (W.PEAK_E5M2_BF16, 1, 0), (W.PEAK_E4M3_BF16, 1, 1)])
def test_fp8_full_size_sampled(dtype, ta, tb):
    """8192^3 in the launch configuration the benchmark times, on a sampled sub-grid."""
    c = any_layout(dtype, ta, tb, 8192, 8192, 8192, dist="uniform")
    dc = R.DeviceCase(c)
    dc.run(P.PEAK_VARIANT_AUTO)
    R.check_sampled(dc, tile_m=256, tile_n=256, budget_macs=6e8)


def test_fp8_strided_batched_one_launch():
    """8-bit inputs through the batched entry point: one persistent launch (3-D tensor maps, byte elements)."""
    from tests.test_gpu_batched import Batch
    for dtype in (W.PEAK_E4M3_BF16, W.PEAK_E5M2_F32):
        n0 = P.peak_kernel_launches()
        c = k_major(dtype, 264, 328, 400, alpha=0.25, beta=-1.0, dist="smallint", pad_c=0)
        b = Batch(c, batch=4, gap=16)
        b.run()
        assert P.peak_kernel_launches() - n0 == 1
        b.check(exact=True, what=f"fp8 batch {dtype}")
        b = Batch(k_major(dtype, 136, 200, 272, alpha=0.5, beta=2.0, dist="uniform"), batch=3, gap=32)
        b.run()
        b.check(what=f"fp8 batch real {dtype}")


@pytest.mark.parametrize("act", [P.PEAK_ACT_NONE, P.PEAK_ACT_RELU, P.PEAK_ACT_GELU])
def test_fp8_fused_bias_activation(act):
    from tests.test_gpu_fused import run_fused, check_fused
    rng = np.random.default_rng(11)
    for variant in [P.PEAK_VARIANT_FALLBACK] + UMMA:
        c = k_major(W.PEAK_E4M3_BF16, 300, 520, 400, alpha=0.5, beta=1.0, dist="uniform", case=act)
        bias = (rng.standard_normal(c.N) * 2).astype(np.float32)
        dc = run_fused(c, variant, bias, act)
        check_fused(dc, bias, act, f"fp8 fused act={act} {P.peak_variant_string(variant)}")


@pytest.mark.parametrize("dtype", [W.PEAK_E4M3_BF16, W.PEAK_E5M2_F32])
def test_fp8_multicast_plugin(dtype, reset_tuning):
    """8-bit inputs through the single-GPU multicast plug-in (forced on): integers bit for bit and identical
    to the plain kernel, reals within the bounds."""
    if not P.peak_multicast_available():
        pytest.skip("libpeak_gemm_mc.so is not present (multi-GPU runs leave it out)")
    for idx, (M, N, K) in enumerate([(512, 256, 128), (1024, 512, 896), (700, 328, 272), (1536, 1280, 2048)]):
        ci = k_major(dtype, M, N, K, dist="smallint", alpha=0.125, beta=-1.0, pad_c=8, case=idx)
        outs = []
        for mode in (2, 1):
            P.peak_set_tuning(P.PEAK_TUNE_MULTICAST, mode)
            dc = R.DeviceCase(ci)
            n0 = P.peak_kernel_launches()
            dc.run(P.PEAK_VARIANT_UMMA_2CTA)
            outs.append(dc.result().copy())
            if mode == 2:
                assert_bits_equal(ci, dc, f"{ci.name} multicast")
        assert np.array_equal(outs[0], outs[1])
        P.peak_set_tuning(P.PEAK_TUNE_MULTICAST, 2)
        cr = k_major(dtype, M, N, K, alpha=0.5, beta=2.0, dist="uniform", case=idx)
        dr = R.DeviceCase(cr)
        dr.run(P.PEAK_VARIANT_UMMA_2CTA)
        R.check_full(dr, what=f"{cr.name} multicast")
