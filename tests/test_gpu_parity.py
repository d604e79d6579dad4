"""GPU parity: every kernel family, called through the C ABI, against the CPU oracle on the same seeded
inputs -- element by element, at sizes that span several tiles, several k-blocks and ragged tails."""
import numpy as np
import pytest
import torch

import oracle
from paper_2512_19018_b200 import binding as P
from paper_2512_19018_b200 import workloads as W
from tests import parity as R

pytestmark = pytest.mark.gpu

LAYOUTS = [(0, 0), (0, 1), (1, 0), (1, 1)]
PAIRS_16 = [W.PEAK_F16_F32, W.PEAK_BF16_BF16, W.PEAK_F16_F16, W.PEAK_BF16_F32]
UMMA = [P.PEAK_VARIANT_UMMA_1CTA, P.PEAK_VARIANT_UMMA_2CTA]


def mk(dtype, ta, tb, M, N, K, **kw):
    return W.GemmCase(f"t{dtype}_{ta}{tb}_{M}x{N}x{K}", dtype, bool(ta), bool(tb), M, N, K, **kw)


# ------------------------------------------------------------------ fallback and cross-check kernels
@pytest.mark.parametrize("dtype", PAIRS_16 + [W.PEAK_F32_F32])
@pytest.mark.parametrize("ta,tb", LAYOUTS)
def test_fallback_any_layout_any_pitch(dtype, ta, tb):
    for (M, N, K, a, b) in [(1, 1, 1, 1.0, 0.0), (67, 130, 45, 0.5, 2.0), (128, 64, 200, -1.0, 1.0), (5, 300, 17, 2.0, 0.0)]:
        c = mk(dtype, ta, tb, M, N, K, alpha=a, beta=b, pad_a=1, pad_b=3, pad_c=5, case=M)
        dc = R.DeviceCase(c)
        dc.run(P.PEAK_VARIANT_FALLBACK)
        R.check_full(dc)


def test_config0_fp16_512_every_family():
    c = W.config0()
    for v in [P.PEAK_VARIANT_FALLBACK] + UMMA + [P.PEAK_VARIANT_AUTO]:
        dc = R.DeviceCase(c)
        dc.run(v)
        R.check_full(dc, what=f"config0/{P.peak_variant_string(v)}")


@pytest.mark.parametrize("dtype", [W.PEAK_BF16_BF16, W.PEAK_F32_F32, W.PEAK_F16_F32])
@pytest.mark.parametrize("ta,tb", LAYOUTS)
def test_xcheck_f64_matches_oracle(dtype, ta, tb):
    c = mk(dtype, ta, tb, 70, 90, 150, alpha=0.5, beta=2.0, pad_a=2, pad_b=2, pad_c=2)
    dc = R.DeviceCase(c)
    out = torch.full((c.M, c.N + 3), float("nan"), dtype=torch.float64, device="cuda")
    P.peak_gemm_xcheck_f64(c.dtype, c.transA, c.transB, c.M, c.N, c.K, c.alpha, dc.A, c.lda, dc.B, c.ldb, c.beta,
                           dc.C, c.ldc, out, c.N + 3)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    ref, S = dc.oracle_full()
    assert np.isnan(got[:, c.N:]).all()
    sp = R.s_prime(c, S, c.alpha, c.beta, R.c0_values(dc))
    assert (np.abs(got[:, :c.N] - ref) <= 4 * c.K * 2.0 ** -53 * sp).all()      # fp64 sum, fma vs mul+add
    assert np.array_equal(dc.result(), dc.C0_h[:, :c.N])                           # C0 is not written


# ------------------------------------------------------------------ tensor-core path: exactness
@pytest.mark.parametrize("variant", UMMA)
@pytest.mark.parametrize("dtype", [W.PEAK_F16_F32, W.PEAK_BF16_BF16, W.PEAK_BF16_F32, W.PEAK_F16_F16])
@pytest.mark.parametrize("ta,tb", LAYOUTS)
def test_umma_exact_small_integers(variant, dtype, ta, tb):
    """Entries in [-4, 4], K <= 512: every partial sum is an integer below 2^24, so any fp32 summation order
    is exact and the output must equal the oracle's correctly rounded value bit for bit.  A dropped or
    repeated k-block, a wrong swizzle or a wrong descriptor stride cannot pass."""
    for (M, N, K) in [(128, 256, 64), (256, 512, 192), (384, 256, 512), (200, 328, 136)]:
        c = mk(dtype, ta, tb, M, N, K, dist="smallint", case=K)
        if c.out_type != "f32":
            c = c.with_(alpha=0.125)     # keep |C| <= 16*512/8 within the exactly representable integers / eighths
        dc = R.DeviceCase(c)
        dc.run(variant)
        ref, _ = dc.oracle_full()
        want = oracle.round_to(R.OT[c.out_type], ref)
        got = dc.result()
        if c.out_type == "f32":
            got = got.view(np.uint32)
        if not np.array_equal(got, want):
            bad = np.argwhere(got != want)
            raise AssertionError(f"{c.name} {P.peak_variant_string(variant)}: {len(bad)} of {got.size} wrong, "
                                 f"first at {bad[0]}, rows {np.unique(bad[:, 0])[:8]}, cols {np.unique(bad[:, 1])[:8]}")


@pytest.mark.parametrize("variant", UMMA)
def test_umma_identity_and_rank1(variant):
    n = 256
    rng = np.random.default_rng(5)
    X = W.encode(rng.standard_normal((n, n)).astype(np.float32), "bf16")
    eye = W.encode(np.eye(n, dtype=np.float32), "bf16")
    A, B = R.to_device(eye, "bf16"), R.to_device(X, "bf16")
    C = torch.zeros((n, n), dtype=torch.bfloat16, device="cuda")
    P.peak_gemm_variant(variant, W.PEAK_BF16_BF16, 0, 0, n, n, n, 1.0, A, n, B, n, 0.0, C, n)
    assert P.peak_check()[0] == P.PEAK_OK
    assert np.array_equal(R.to_host(C, "bf16"), X)          # I * X == X exactly
    P.peak_gemm_variant(variant, W.PEAK_BF16_BF16, 0, 0, n, n, n, 1.0, B, n, A, n, 0.0, C, n)
    assert P.peak_check()[0] == P.PEAK_OK
    assert np.array_equal(R.to_host(C, "bf16"), X)          # X * I == X exactly


# ------------------------------------------------------------------ tensor-core path: tolerance parity
RAGGED = [(1, 8, 8), (7, 16, 24), (127, 255, 63), (129, 257, 65), (128, 256, 64), (300, 520, 200), (17, 1000, 72),
          (513, 24, 1032)]


@pytest.mark.parametrize("variant", UMMA)
@pytest.mark.parametrize("dtype", [W.PEAK_F16_F32, W.PEAK_BF16_BF16])
@pytest.mark.parametrize("ta,tb", LAYOUTS)
def test_umma_ragged_shapes_alpha_beta(variant, dtype, ta, tb):
    for idx, (M, N, K) in enumerate(RAGGED):
        # pitches must stay multiples of 8 elements for TMA: pad so that they are
        a_cols = M if ta else K
        b_cols = K if tb else N
        alpha, beta = [(1.0, 0.0), (0.5, 2.0), (-1.0, 1.0)][idx % 3]
        c = mk(dtype, ta, tb, M, N, K, alpha=alpha, beta=beta, pad_a=(-a_cols) % 8 + 8, pad_b=(-b_cols) % 8,
               pad_c=idx % 4, case=idx)
        dc = R.DeviceCase(c)
        dc.run(variant)
        R.check_full(dc, what=f"{c.name}/{P.peak_variant_string(variant)}")


@pytest.mark.parametrize("variant", UMMA)
def test_umma_run_to_run_bit_identical(variant):
    c = mk(W.PEAK_BF16_BF16, 0, 1, 640, 768, 1024, dist="normal_rsqrtk")
    dc = R.DeviceCase(c)
    outs = []
    for _ in range(3):
        dc.reset_c()
        dc.run(variant)
        outs.append(dc.result().copy())
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[0], outs[2])
    R.check_full(dc)


@pytest.mark.parametrize("variant", UMMA + [P.PEAK_VARIANT_FALLBACK])
def test_alpha_beta_invariants_on_gpu(variant):
    c = mk(W.PEAK_BF16_BF16, 0, 0, 256, 256, 128, beta=1.0)
    dc = R.DeviceCase(c)
    c0 = dc.C0_h[:, :c.N].copy()
    dc.run(variant, alpha=0.0, beta=1.0)                    # C unchanged, bit for bit
    assert np.array_equal(dc.result(), c0)
    dc.run(variant, alpha=0.0, beta=0.0)                    # zeros
    assert not dc.result().any()
    nan_case = R.DeviceCase(c.with_(beta=0.0), c_init="poison")
    nan_case.run(variant)                                   # beta == 0: NaN in C does not propagate
    R.check_full(nan_case)
    r1 = nan_case.result().copy()
    nan_case.reset_c()
    nan_case.run(variant, alpha=4.0)                        # power-of-two scaling is exact
    assert np.array_equal(W.to_float64(nan_case.result(), "bf16"), 4.0 * W.to_float64(r1, "bf16"))


def test_quick_returns_on_gpu():
    c = mk(W.PEAK_F16_F32, 0, 0, 96, 80, 64, beta=0.5)
    dc = R.DeviceCase(c)
    before = dc.result().copy()
    P.peak_gemm(c.dtype, 0, 0, 0, c.N, c.K, 1.0, dc.A, c.lda, dc.B, c.ldb, 0.5, dc.C, c.ldc)       # M == 0
    P.peak_gemm(c.dtype, 0, 0, c.M, 0, c.K, 1.0, dc.A, c.lda, dc.B, c.ldb, 0.5, dc.C, c.ldc)       # N == 0
    torch.cuda.synchronize()
    assert np.array_equal(dc.result(), before)
    P.peak_gemm(c.dtype, 0, 0, c.M, c.N, 0, 1.0, None, c.lda, None, c.ldb, 0.5, dc.C, c.ldc)        # K == 0
    torch.cuda.synchronize()
    assert np.array_equal(dc.result(), (0.5 * before).astype(np.float32))
    nanA = torch.full_like(dc.A, float("nan"))
    P.peak_gemm(c.dtype, 0, 0, c.M, c.N, c.K, 0.0, nanA, c.lda, nanA, c.ldb, 2.0, dc.C, c.ldc)      # alpha == 0
    torch.cuda.synchronize()
    assert np.array_equal(dc.result(), before)               # 2 * (0.5 * before); A and B were not read


# ------------------------------------------------------------------ SGEMM
@pytest.mark.parametrize("ta,tb", LAYOUTS)
def test_sgemm_parity(ta, tb):
    for (M, N, K, a, b) in [(128, 128, 16, 1.0, 0.0), (256, 384, 160, 0.5, 2.0), (384, 128, 1024, -1.0, 1.0)]:
        c = mk(W.PEAK_F32_F32, ta, tb, M, N, K, alpha=a, beta=b, pad_a=4, pad_b=8, pad_c=4, case=K)
        dc = R.DeviceCase(c)
        dc.run(P.PEAK_VARIANT_SGEMM)
        R.check_full(dc)
    ci = mk(W.PEAK_F32_F32, ta, tb, 256, 256, 512, dist="smallint")
    dc = R.DeviceCase(ci)
    dc.run(P.PEAK_VARIANT_SGEMM)
    ref, _ = dc.oracle_full()
    assert np.array_equal(dc.result().view(np.uint32), oracle.round_to(oracle.F32, ref))


@pytest.mark.parametrize("ta,tb", LAYOUTS)
def test_sgemm_ragged_shapes_run_the_fast_kernel(ta, tb, reset_tuning):
    """Shapes that are not made of whole tiles (ragged M, N, a K tail, one-row and one-column problems) run on the
    TMA-fed SGEMM kernel, whose copies zero-fill the edges: exact on integers, within the fp32 bounds on reals,
    guard bands and pitch padding untouched."""
    shapes = [(1000, 1000, 1000), (129, 257, 33), (1, 300, 50), (300, 1, 7), (131, 131, 16), (500, 300, 250)]
    for idx, (M, N, K) in enumerate(shapes):
        pa, pb = (-(M if ta else K)) % 4, (-(K if tb else N)) % 4        # the copy engine wants 16-byte pitches
        for pc in (0, 3):                                                # aligned and unaligned rows of C
            ci = mk(W.PEAK_F32_F32, ta, tb, M, N, K, dist="smallint", alpha=2.0, beta=-1.0, pad_a=pa, pad_b=pb,
                    pad_c=pc, case=idx)
            dc = R.DeviceCase(ci)
            dc.run(P.PEAK_VARIANT_SGEMM)
            assert "sgemm_tma_kernel" in P.peak_last_kernel()
            ref, _ = dc.oracle_full()
            assert np.array_equal(dc.result().view(np.uint32), oracle.round_to(oracle.F32, ref)), f"{ci}"
        cr = mk(W.PEAK_F32_F32, ta, tb, M, N, K, alpha=0.5, beta=2.0, pad_a=pa + 4, pad_b=pb, pad_c=1, case=idx)
        dr = R.DeviceCase(cr)
        dr.run(P.PEAK_VARIANT_AUTO)
        assert "sgemm_tma_kernel" in P.peak_last_kernel()
        R.check_full(dr)


@pytest.mark.parametrize("copy", [1, 2, 3])
@pytest.mark.parametrize("fma", [1, 2])
def test_sgemm_kernel_variants_agree_with_oracle(copy, fma, reset_tuning):
    """Register-staged vs asynchronous-copy tile loads, scalar vs two-wide FMA: every combination exact on
    integer inputs and within the fp32 bounds on real inputs, for all four layouts."""
    P.peak_set_tuning(P.PEAK_TUNE_SGEMM_COPY, copy)
    P.peak_set_tuning(P.PEAK_TUNE_SGEMM_FMA, fma)
    for ta, tb in LAYOUTS:
        ci = mk(W.PEAK_F32_F32, ta, tb, 384, 256, 528, dist="smallint", alpha=2.0, beta=-1.0, pad_a=4, pad_b=4, pad_c=4)
        dc = R.DeviceCase(ci)
        dc.run(P.PEAK_VARIANT_SGEMM)
        ref, _ = dc.oracle_full()
        assert np.array_equal(dc.result().view(np.uint32), oracle.round_to(oracle.F32, ref))
        cr = mk(W.PEAK_F32_F32, ta, tb, 256, 384, 1040, alpha=0.5, beta=2.0)
        dr = R.DeviceCase(cr)
        dr.run(P.PEAK_VARIANT_SGEMM)
        R.check_full(dr)


def test_sgemm_unsupported_shape_is_reported_not_faulted():
    c = mk(W.PEAK_F32_F32, 0, 0, 100, 128, 16, pad_a=1)      # a pitch the copy engine cannot take, not whole tiles
    dc = R.DeviceCase(c)
    rc = P.peak_gemm_variant(P.PEAK_VARIANT_SGEMM, c.dtype, 0, 0, c.M, c.N, c.K, 1.0, dc.A, c.lda, dc.B, c.ldb, 0.0,
                             dc.C, c.ldc, check=False)
    assert rc == P.PEAK_ERR_UNSUPPORTED
    rc = P.peak_gemm_variant(P.PEAK_VARIANT_UMMA_1CTA, c.dtype, 0, 0, c.M, c.N, c.K, 1.0, dc.A, c.lda, dc.B, c.ldb,
                             0.0, dc.C, c.ldc, check=False)
    assert rc == P.PEAK_ERR_UNSUPPORTED
    dc.run(P.PEAK_VARIANT_AUTO)                              # the dispatcher falls back
    R.check_full(dc)


def test_host_buffer_entry_point():
    c = mk(W.PEAK_BF16_BF16, 1, 0, 300, 264, 200, alpha=0.5, beta=2.0, pad_a=4, pad_c=8)
    A, B, C0 = W.make_inputs(c)
    C = C0.copy()
    P.peak_gemm_host(c.dtype, c.transA, c.transB, c.M, c.N, c.K, c.alpha, A, c.lda, B, c.ldb, c.beta, C, c.ldc)
    ref, S = oracle.gemm(oracle.BF16, oracle.BF16, 1, 0, c.M, c.N, c.K, c.alpha, A, c.lda, B, c.ldb, c.beta, C0, c.ldc)
    R.check_values(c, C[:, :c.N], ref, S, W.to_float64(C0[:, :c.N], "bf16"), what="host entry point")
    assert np.array_equal(C[:, c.N:], C0[:, c.N:])           # pitch padding survives the round trip
    P.peak_release_staging()


@pytest.mark.parametrize("ta,tb", LAYOUTS)
def test_host_buffer_entry_point_pipelined_panels(ta, tb):
    """From 1024 rows on the host entry point works in row panels (copy in / multiply / copy out overlap):
    ragged panel sizes, both storage orders of A, old C needed or not, pitch padding kept."""
    for (M, N, K, beta, pad_c) in [(1500, 328, 264, 2.0, 8), (4100, 136, 200, 0.0, 0), (1030, 520, 72, 0.0, 8)]:
        c = mk(W.PEAK_BF16_BF16, ta, tb, M, N, K, alpha=0.5, beta=beta, pad_a=(-(M if ta else K)) % 8,
               pad_b=(-(K if tb else N)) % 8, pad_c=pad_c, case=M)
        A, B, C0 = W.make_inputs(c, need_c0=True)
        C = C0.copy()
        n0 = P.peak_kernel_launches()
        P.peak_gemm_host(c.dtype, c.transA, c.transB, c.M, c.N, c.K, c.alpha, A, c.lda, B, c.ldb, c.beta, C, c.ldc)
        assert P.peak_kernel_launches() - n0 >= 2                 # more than one panel
        ref, S = oracle.gemm(oracle.BF16, oracle.BF16, ta, tb, c.M, c.N, c.K, c.alpha, A, c.lda, B, c.ldb, c.beta,
                             C0 if beta != 0 else None, c.ldc)
        c0 = W.to_float64(C0[:, :c.N], "bf16") if beta != 0 else 0.0
        R.check_values(c, C[:, :c.N], ref, S, c0, what=f"host panels {M}x{N}x{K} {ta}{tb}")
        if pad_c:
            assert np.array_equal(C[:, c.N:], C0[:, c.N:])
    P.peak_release_staging()


def test_launch_counter_moves():
    n0 = P.peak_kernel_launches()
    dc = R.DeviceCase(W.config0())
    dc.run()
    assert P.peak_kernel_launches() == n0 + 1


# ------------------------------------------------------------------ tuning knobs never change results
@pytest.fixture
def reset_tuning():
    yield
    for key in range(P.PEAK_TUNE_COUNT):
        P.peak_set_tuning(key, 0)


@pytest.mark.parametrize("variant", UMMA)
@pytest.mark.parametrize("tile_n", [128, 256])
@pytest.mark.parametrize("epilogue", [1, 2, 3])
def test_umma_tile_width_epilogue_and_split_k(variant, tile_n, epilogue, reset_tuning):
    """Tile width, epilogue store path and k-split are performance knobs: with integer inputs every
    combination must give the oracle's correctly rounded result bit for bit (which also shows that a split
    neither drops nor repeats a k-block), and with real inputs the tolerance checks must hold."""
    P.peak_set_tuning(P.PEAK_TUNE_TILE_N, tile_n)
    P.peak_set_tuning(P.PEAK_TUNE_EPILOGUE, epilogue)
    for split in (1, 2, 3, 5):
        P.peak_set_tuning(P.PEAK_TUNE_SPLIT_K, split)
        for idx, (dtype, ta, tb, M, N, K) in enumerate([(W.PEAK_BF16_BF16, 1, 0, 200, 328, 456),
                                                       (W.PEAK_F16_F32, 0, 1, 300, 136, 520),
                                                       (W.PEAK_BF16_F32, 0, 0, 16, 520, 640),
                                                       (W.PEAK_F16_F16, 1, 1, 264, 256, 320)]):
            ci = mk(dtype, ta, tb, M, N, K, dist="smallint", alpha=0.125, beta=-2.0, case=idx)
            dc = R.DeviceCase(ci)
            dc.run(variant)
            ref, _ = dc.oracle_full()
            want = oracle.round_to(R.OT[ci.out_type], ref)
            got = dc.result()
            got = got.view(np.uint32) if ci.out_type == "f32" else got
            assert np.array_equal(got, want), f"{ci.name} tile_n={tile_n} epilogue={epilogue} split={split}"
            cr = mk(dtype, ta, tb, M, N, K, alpha=0.5, beta=2.0, pad_c=8, case=idx)
            dr = R.DeviceCase(cr)
            dr.run(variant)
            R.check_full(dr, what=f"{cr.name} tile_n={tile_n} epilogue={epilogue} split={split}")


@pytest.mark.parametrize("variant", UMMA)
@pytest.mark.parametrize("tail", [1, 2])
def test_umma_last_wave_split(variant, tail, reset_tuning):
    """More tiles than SMs with a partly filled last wave: with the tail split forced on, the tiles of that
    wave are computed as k-slices and reduced by the second kernel; forced off, they are computed whole.
    Integer inputs (K = 1024, entries in [-4, 4]) make both exact: sampled elements of every tile must equal
    the oracle's correctly rounded value bit for bit, and the two settings must agree on the whole matrix."""
    P.peak_set_tuning(P.PEAK_TUNE_TAIL_SPLIT, tail)
    outs = []
    for (dtype, ta, tb, M, N) in [(W.PEAK_BF16_BF16, 0, 1, 2560, 2304), (W.PEAK_F16_F32, 1, 0, 3000, 3336)]:
        c = mk(dtype, ta, tb, M, N, 1024, dist="smallint", alpha=0.125, beta=-1.0, pad_c=8)
        dc = R.DeviceCase(c)
        dc.run(variant)
        rows, cols = R.sample_grid(c, 128, 128, budget_macs=6e8)
        ref, _ = dc.oracle_sub(rows, cols)
        want = oracle.round_to(R.OT[c.out_type], ref)
        got = dc.result()[np.ix_(rows, cols)]
        got = got.view(np.uint32) if c.out_type == "f32" else got
        assert np.array_equal(got, want), f"{c.name} tail={tail}"
        outs.append(dc.result().copy())
    key = ("tail_outs", variant)
    prev = _TAIL_CACHE.get(key)
    if prev is not None:
        assert all(np.array_equal(a, b) for a, b in zip(prev, outs)), "tail split on / off disagree"
    _TAIL_CACHE[key] = outs


_TAIL_CACHE = {}


@pytest.mark.parametrize("dtype", [W.PEAK_BF16_BF16, W.PEAK_F16_F32])
@pytest.mark.parametrize("ta,tb", LAYOUTS)
def test_umma_512_wide_tiles(dtype, ta, tb, reset_tuning):
    """256 x 512 pair tiles computed as two 256-column halves over both accumulator slots: exact on integer
    inputs (several tiles per CTA pair so that the half-by-half hand-over between epilogue and main loop is
    exercised), bounds on real inputs with alpha/beta and ragged edges."""
    P.peak_set_tuning(P.PEAK_TUNE_TILE_N, 512)
    for idx, (M, N, K) in enumerate([(256, 512, 64), (512, 1024, 320), (300, 700, 200), (8192, 6144, 128)]):
        pa, pb = (-(M if ta else K)) % 8, (-(K if tb else N)) % 8
        ci = mk(dtype, ta, tb, M, N, K, dist="smallint", alpha=0.125, beta=-1.0, case=idx, pad_a=pa, pad_b=pb, pad_c=8)
        dc = R.DeviceCase(ci)
        dc.run(P.PEAK_VARIANT_UMMA_2CTA)
        if M * N * K <= 2e9:
            ref, _ = dc.oracle_full()
            got = dc.result()
        else:                       # 192 tiles over 74 CTA pairs: check a sub-grid that samples every tile
            rows, cols = R.sample_grid(ci, 256, 256, budget_macs=4e8)
            ref, _ = dc.oracle_sub(rows, cols)
            got = dc.result()[np.ix_(rows, cols)]
        want = oracle.round_to(R.OT[ci.out_type], ref)
        got = got.view(np.uint32) if ci.out_type == "f32" else got
        assert np.array_equal(got, want), f"{ci.name}: 512-wide tiles differ from the oracle"
        if M * N * K <= 2e9:
            cr = mk(dtype, ta, tb, M, N, K, alpha=0.5, beta=2.0, case=idx, pad_a=pa, pad_b=pb)
            dr = R.DeviceCase(cr)
            dr.run(P.PEAK_VARIANT_UMMA_2CTA)
            R.check_full(dr, what=f"{cr.name} 512-wide")


def test_auto_dispatch_skinny_shapes(reset_tuning):
    """Shapes with few output tiles (the dispatcher may split K): results against the oracle, run twice
    for bit-identical output (the split reduction is in a fixed order)."""
    for (M, N, K) in [(16, 1024, 4096), (128, 1792, 2048), (40, 264, 8192)]:
        c = mk(W.PEAK_BF16_BF16, 1, 0, M, N, K, alpha=0.5, beta=2.0, case=M)
        dc = R.DeviceCase(c)
        dc.run()
        first = dc.result().copy()
        R.check_full(dc)
        dc.reset_c()
        dc.run()
        assert np.array_equal(first, dc.result())


@pytest.mark.parametrize("variant", UMMA)
def test_bounded_wait_reports_timeout_and_context_survives(variant, reset_tuning):
    """Failure detection without a GPU fault: a test hook makes one CTA leave a pipeline stage unfilled (a
    barrier that nothing completes).  The waits downstream give up after their budget (set to 20 ms here),
    the kernel unwinds and frees its tensor memory, peak_check() reports PEAK_ERR_TIMEOUT once, and the next
    call on the same context computes correct results."""
    c = mk(W.PEAK_BF16_BF16, 0, 1, 512, 512, 256)
    dc = R.DeviceCase(c)
    P.peak_set_tuning(P.PEAK_TUNE_WAIT_MS, 20)
    P.peak_set_tuning(P.PEAK_TUNE_INJECT_STALL, 1)
    P.peak_gemm_variant(variant, c.dtype, c.transA, c.transB, c.M, c.N, c.K, 1.0, dc.A, c.lda, dc.B, c.ldb, 0.0, dc.C,
                        c.ldc)
    rc, detail = P.peak_check()
    assert rc == P.PEAK_ERR_TIMEOUT and (detail & 0x80000000)
    assert P.peak_check()[0] == P.PEAK_OK                      # the status word was cleared
    P.peak_set_tuning(P.PEAK_TUNE_INJECT_STALL, 0)
    P.peak_set_tuning(P.PEAK_TUNE_WAIT_MS, 0)
    dc.reset_c()
    dc.run(variant)                                            # same context, same buffers: correct again
    R.check_full(dc)


@pytest.mark.parametrize("tile_n", [256, 512])
@pytest.mark.parametrize("dtype", [W.PEAK_BF16_BF16, W.PEAK_F16_F32])
@pytest.mark.parametrize("ta,tb", LAYOUTS)
def test_multicast_plugin_matches_oracle(dtype, ta, tb, tile_n, reset_tuning):
    """The optional cluster-multicast plug-in (four-CTA clusters sharing B tiles), forced on: exact on integer
    inputs for every layout, within the bounds on real inputs with alpha/beta and ragged edges, and identical
    to the plain kernel's output bit for bit on the integer cases."""
    if not P.peak_multicast_available():
        pytest.skip("libpeak_gemm_mc.so is not present (multi-GPU runs leave it out)")
    P.peak_set_tuning(P.PEAK_TUNE_TILE_N, tile_n)      # 512 x 256 or 512 x 512 super-tiles
    for idx, (M, N, K) in enumerate([(512, 256, 64), (1024, 512, 448), (700, 328, 264), (1536, 1280, 1024)]):
        pa, pb = (-(M if ta else K)) % 8, (-(K if tb else N)) % 8     # TMA needs pitches that are multiples of 8
        ci = mk(dtype, ta, tb, M, N, K, dist="smallint", alpha=0.125, beta=-1.0, case=idx, pad_a=pa, pad_b=pb, pad_c=8)
        outs = []
        for mode in (2, 1):
            P.peak_set_tuning(P.PEAK_TUNE_MULTICAST, mode)
            dc = R.DeviceCase(ci)
            dc.run(P.PEAK_VARIANT_UMMA_2CTA)
            outs.append(dc.result().copy())
            if mode == 2:
                ref, _ = dc.oracle_full()
                want = oracle.round_to(R.OT[ci.out_type], ref)
                got = outs[0].view(np.uint32) if ci.out_type == "f32" else outs[0]
                assert np.array_equal(got, want), f"{ci.name}: multicast result differs from the oracle"
        assert np.array_equal(outs[0], outs[1]), f"{ci.name}: multicast and plain kernels disagree"
        P.peak_set_tuning(P.PEAK_TUNE_MULTICAST, 2)
        cr = mk(dtype, ta, tb, M, N, K, alpha=0.5, beta=2.0, case=idx, pad_a=pa, pad_b=pb)
        dr = R.DeviceCase(cr)
        dr.run(P.PEAK_VARIANT_UMMA_2CTA)
        R.check_full(dr, what=f"{cr.name} multicast")


def test_set_tuning_rejects_bad_arguments():
    with pytest.raises(P.PeakError):
        P.peak_set_tuning(99, 1)
    with pytest.raises(P.PeakError):
        P.peak_set_tuning(P.PEAK_TUNE_TILE_N, -1)


def test_tuner_runs_and_restores_defaults():
    from paper_2512_19018_b200 import tune
    out = tune.main(["--dtype", "bf16_bf16", "--layout", "NT", "-M", "512", "-N", "512", "-K", "512", "--seconds",
                     "0.002", "--quick"])
    assert out["candidates_timed"] >= 4 and out["best"]["ms"] <= out["auto_ms"] * 1.5
    # the tuner leaves the library at its defaults
    c = mk(W.PEAK_BF16_BF16, 0, 1, 512, 512, 512)
    dc = R.DeviceCase(c)
    dc.run()
    R.check_full(dc)


def test_cuda_graph_capture_and_replay():
    """Calls that need no workspace allocate nothing and can be captured into a CUDA graph; replays recompute
    C from whatever A and B then hold."""
    c = mk(W.PEAK_BF16_BF16, 0, 0, 768, 512, 384)
    dc = R.DeviceCase(c)
    stream = torch.cuda.Stream()
    dc.run(stream=None)                                        # warm-up outside the capture (first-use set-up)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            P.peak_gemm(c.dtype, c.transA, c.transB, c.M, c.N, c.K, c.alpha, dc.A, c.lda, dc.B, c.ldb, c.beta, dc.C,
                        c.ldc, stream)
    dc.reset_c_in_place = None
    dc.C.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert P.peak_check()[0] == P.PEAK_OK
    R.check_full(dc)
    dc.A.mul_(2.0)                                             # new operand values, same buffers
    dc.A_h = R.to_host(dc.A, c.in_type)
    graph.replay()
    torch.cuda.synchronize()
    R.check_full(dc)


@pytest.mark.parametrize("variant", [P.PEAK_VARIANT_FALLBACK] + UMMA)
@pytest.mark.parametrize("dtype,tiny,big", [(W.PEAK_F16_F32, 2.0 ** -24, 2.0 ** 12), (W.PEAK_BF16_F32, 2.0 ** -133, 2.0 ** 120)])
def test_subnormal_inputs_are_honoured(variant, dtype, tiny, big):
    """A holds subnormal values of the input format (small integer multiples of its smallest subnormal), B
    large powers of two: every product and every partial sum is exactly representable in fp32, so the
    result must equal the oracle bit for bit.  A path that flushed subnormal inputs to zero would return 0."""
    M, N, K = 128, 128, 64
    rng = np.random.default_rng(5)
    a = rng.integers(-7, 8, size=(M, K)).astype(np.float64) * tiny
    b = rng.integers(-2, 3, size=(K, N)).astype(np.float64) * big
    t = W.IN_TYPE[dtype]
    A_h = oracle.round_to(R.OT[t], a)
    B_h = oracle.round_to(R.OT[t], b)
    assert np.array_equal(oracle.decode(R.OT[t], A_h), a) and np.array_equal(oracle.decode(R.OT[t], B_h), b)
    A, B = R.to_device(A_h, t), R.to_device(B_h, t)
    C = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    P.peak_gemm_variant(variant, dtype, 0, 0, M, N, K, 1.0, A, K, B, N, 0.0, C, N)
    rc, _ = P.peak_check()
    assert rc == P.PEAK_OK
    ref, _ = oracle.gemm(R.OT[t], oracle.F32, 0, 0, M, N, K, 1.0, A_h, K, B_h, N, 0.0, None, N)
    want = oracle.round_to(oracle.F32, ref)
    assert np.abs(ref).max() > 0
    got = C.cpu().numpy().view(np.uint32)
    assert np.array_equal(got, want), f"{(got != want).sum()} of {got.size} differ"


@pytest.mark.parametrize("variant", [P.PEAK_VARIANT_FALLBACK] + UMMA)
@pytest.mark.parametrize("dtype", [W.PEAK_F16_F16, W.PEAK_BF16_BF16, W.PEAK_F16_F32])
def test_inf_nan_propagate_and_outputs_overflow_to_inf(variant, dtype):
    """IEEE propagation through the sum (an infinity in A makes its row of C infinite, NaN where it meets a
    zero of B; a NaN poisons its row) and no saturation when the rounded output overflows."""
    M, N, K = 128, 256, 64
    c = mk(dtype, 0, 0, M, N, K, dist="smallint", case=77)
    A_h, B_h, _ = W.make_inputs(c)
    t = c.in_type
    inf_bits = {"f16": 0x7C00, "bf16": 0x7F80}[t]
    A_h[3, 5] = inf_bits                       # +inf in row 3
    A_h[9, 0] = W.NAN_BITS[t]                  # NaN in row 9
    A, B = R.to_device(A_h, t), R.to_device(B_h, t)
    Cd = R.to_device(W.poison_c(c), c.out_type)
    P.peak_gemm_variant(variant, dtype, 0, 0, M, N, K, 1.0, A, c.lda, B, c.ldb, 0.0, Cd, c.ldc)
    assert P.peak_check()[0] == P.PEAK_OK
    got = W.to_float64(R.to_host(Cd, c.out_type), c.out_type)[:, :N]
    ref, _ = oracle.gemm(R.OT[t], R.OT[c.out_type], 0, 0, M, N, K, 1.0, A_h, c.lda, B_h, c.ldb, 0.0, None, c.ldc)
    assert np.isnan(ref[9]).all() and np.isinf(ref[3]).any() and np.isnan(ref[3]).any()
    assert np.array_equal(np.isnan(got), np.isnan(ref))
    assert np.array_equal(np.isposinf(got), np.isposinf(ref)) and np.array_equal(np.isneginf(got), np.isneginf(ref))
    fin = np.isfinite(ref)
    assert np.array_equal(got[fin], ref[fin])                      # small integers elsewhere: exact
    if c.out_type != "f32":
        # alpha pushes finite sums beyond the largest finite 16-bit value: +-inf, not the largest finite number
        big = 3.0e38 if c.out_type == "bf16" else 6.0e4
        Cd = R.to_device(W.poison_c(c), c.out_type)
        A2_h, B2_h, _ = W.make_inputs(c)
        P.peak_gemm_variant(variant, dtype, 0, 0, M, N, K, big, R.to_device(A2_h, t), c.lda, R.to_device(B2_h, t), c.ldb,
                            0.0, Cd, c.ldc)
        assert P.peak_check()[0] == P.PEAK_OK
        got = W.to_float64(R.to_host(Cd, c.out_type), c.out_type)[:, :N]
        ref, _ = oracle.gemm(R.OT[t], R.OT[c.out_type], 0, 0, M, N, K, float(np.float32(big)), A2_h, c.lda, B2_h, c.ldb,
                             0.0, None, c.ldc)
        want = W.to_float64(oracle.round_to(R.OT[c.out_type], ref), c.out_type)
        assert np.isinf(want).any() and np.array_equal(np.isinf(got), np.isinf(want))
        assert np.array_equal(np.sign(got[np.isinf(got)]), np.sign(want[np.isinf(want)]))


@pytest.mark.parametrize("variant", UMMA)
@pytest.mark.parametrize("warps", [1, 2])
@pytest.mark.parametrize("tile_n", [128, 256])
def test_umma_epilogue_warp_groups(variant, warps, tile_n, reset_tuning):
    """One or two groups of epilogue warps on one-slot tiles: same bits (integers), same tolerance (reals),
    for every output type, with ragged edges, alpha/beta, a k-split and both store paths."""
    P.peak_set_tuning(P.PEAK_TUNE_EPILOGUE_WARPS, warps)
    P.peak_set_tuning(P.PEAK_TUNE_TILE_N, tile_n)
    for dtype in PAIRS_16:
        for (ta, tb, M, N, K, split) in [(0, 0, 384, 520, 200, 0), (1, 1, 200, 328, 264, 2), (0, 1, 130, 257, 136, 0)]:
            P.peak_set_tuning(P.PEAK_TUNE_SPLIT_K, split)
            pa, pb = (-(M if ta else K)) % 8, (-(K if tb else N)) % 8
            ci = mk(dtype, ta, tb, M, N, K, dist="smallint", alpha=0.25, beta=-1.0, pad_a=pa, pad_b=pb, case=tile_n + warps)
            di = R.DeviceCase(ci)
            di.run(variant)
            ref, _ = di.oracle_full()
            want = oracle.round_to(R.OT[ci.out_type], ref)
            got = di.result()
            if ci.out_type == "f32":
                got = got.view(np.uint32)
            assert np.array_equal(got, want), f"{ci.name} warps={warps} tile_n={tile_n} split={split}"
            cr = ci.with_(dist="uniform", alpha=0.5, beta=2.0)
            dr = R.DeviceCase(cr)
            dr.run(variant)
            R.check_full(dr, what=f"{cr.name} warps={warps} tile_n={tile_n} split={split}")


def test_two_host_threads_two_streams():
    """Distinct streams from distinct host threads at the same time (the binding releases the GIL inside the
    library): different shapes and kernel families, a k-split among them; every result must match the oracle."""
    import threading
    jobs = [mk(W.PEAK_BF16_BF16, 0, 0, 520, 776, 264, alpha=0.5, beta=2.0, case=1),
            mk(W.PEAK_F16_F32, 1, 0, 96, 1032, 1544, alpha=1.0, beta=1.0, pad_a=0, case=2),      # k-split path
            mk(W.PEAK_F32_F32, 0, 0, 256, 256, 128, alpha=-1.0, beta=0.5, case=3),               # SGEMM
            mk(W.PEAK_BF16_F32, 0, 1, 1000, 264, 520, alpha=2.0, beta=0.0, case=4)]
    cases = [R.DeviceCase(c) for c in jobs]
    errors = []

    def worker(idx):
        try:
            st = torch.cuda.Stream()
            for rep in range(20):
                for k in range(idx, len(cases), 2):
                    dc = cases[k]
                    dc.reset_c()
                    st.wait_stream(torch.cuda.current_stream())     # the upload of C ran on the default stream
                    c = dc.case
                    P.peak_gemm(c.dtype, c.transA, c.transB, c.M, c.N, c.K, c.alpha, dc.A, c.lda, dc.B, c.ldb, c.beta,
                                dc.C, c.ldc, st)
                    rc, detail = P.peak_check(st)
                    assert rc == P.PEAK_OK, hex(detail)
                    if rep == 19:
                        R.check_full(dc, what=f"thread {idx} {c.name}")
        except Exception as exc:                                     # reported by the main thread
            errors.append(exc)

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors[0]


@pytest.mark.parametrize("dtype", [W.PEAK_F16_F32, W.PEAK_BF16_BF16])
@pytest.mark.parametrize("knobs", [{"tile": 512, "warps": 0, "mc": 1}, {"tile": 256, "warps": 2, "mc": 1},
                                   {"tile": 512, "warps": 0, "mc": 2}, {"tile": 256, "warps": 2, "mc": 2}])
def test_old_c_by_tma_with_a_group_that_has_no_columns(dtype, knobs, reset_tuning):
    """beta != 0 on kernels with two groups of epilogue warps, several tiles per CTA, and a last tile column so
    narrow that the second group's columns lie beyond N: that group must request nothing (a request without
    its wait left a barrier armed and the next tile's wait ran out)."""
    if knobs["mc"] == 2 and not P.peak_multicast_available():
        pytest.skip("libpeak_gemm_mc.so is not present")
    P.peak_set_tuning(P.PEAK_TUNE_TILE_N, knobs["tile"])
    P.peak_set_tuning(P.PEAK_TUNE_EPILOGUE_WARPS, knobs["warps"])
    P.peak_set_tuning(P.PEAK_TUNE_MULTICAST, knobs["mc"])
    P.peak_set_tuning(P.PEAK_TUNE_WAIT_MS, 50)
    for (M, N, K) in [(3840, 2056, 192), (4480, 1544, 128), (2944, 4992, 128)]:
        c = mk(dtype, 0, 1, M, N, K, alpha=0.5, beta=2.0, case=N)
        dc = R.DeviceCase(c)
        dc.run(P.PEAK_VARIANT_UMMA_2CTA)
        R.check_sampled(dc, tile_m=128, tile_n=128, budget_macs=2e7, what=f"{c.name} {knobs}")


def test_cuda_graph_with_k_split_and_several_calls():
    """A captured sequence: a k-split problem (pooled workspace allocated and freed inside the capture, reduce
    kernel launched as a programmatic dependent), a beta != 0 problem, a wide-tile problem and the three forms of
    the one-tile-per-CTA kernel (cluster launches), replayed twice."""
    cases = [mk(W.PEAK_BF16_BF16, 1, 0, 16, 1024, 2048, alpha=0.5, beta=2.0, case=1),        # split-K
             mk(W.PEAK_F16_F32, 0, 1, 520, 776, 264, alpha=1.0, beta=1.0, case=2),
             mk(W.PEAK_BF16_BF16, 0, 0, 512, 1024, 4096, case=3),
             # the one-tile-per-CTA kernel: four k-slices on a cluster, two k-slices, whole tiles
             mk(W.PEAK_BF16_BF16, 1, 0, 16, 4096, 4096, alpha=0.5, beta=2.0, case=4),
             mk(W.PEAK_BF16_F32, 0, 1, 128, 6400, 3200, alpha=1.0, beta=1.0, case=5),
             mk(W.PEAK_F16_F16, 0, 0, 256, 2560, 512, alpha=2.0, beta=0.0, case=6)]
    dcs = [R.DeviceCase(c) for c in cases]
    stream = torch.cuda.Stream()
    names = []
    for dc in dcs:
        dc.run(stream=None)                                    # first-use set-up outside the capture
        names.append(P.peak_last_kernel())
    assert "umma_clusterk_kernel<128, __nv_bfloat16, 4, 0>" in names[3], names[3]
    assert "umma_clusterk_kernel<128, float, 2, 0>" in names[4], names[4]
    assert "umma_clusterk_kernel<128, __half, 1, 0>" in names[5], names[5]
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            for dc in dcs:
                c = dc.case
                P.peak_gemm(c.dtype, c.transA, c.transB, c.M, c.N, c.K, c.alpha, dc.A, c.lda, dc.B, c.ldb, c.beta,
                            dc.C, c.ldc, stream)
    for rep in range(2):
        for dc in dcs:                                          # restore C0 in place (the graph holds the pointers)
            dc.Cfull.copy_(R.to_device(dc.Cfull_h, dc.case.out_type))
        graph.replay()
        torch.cuda.synchronize()
        assert P.peak_check()[0] == P.PEAK_OK
        for dc in dcs:
            R.check_full(dc, what=f"graph replay {rep} {dc.case.name}")


@pytest.mark.parametrize("variant", UMMA)
def test_alternating_k_order_is_exact_and_repeatable(variant, reset_tuning):
    """Every other tile of a CTA walks its k-blocks downwards (PEAK_TUNE_K_ORDER = 2): on integer inputs the
    result is still exact, whatever the tile width, k-split or layout, on problems of several tiles per CTA with a
    ragged K tail; and two runs give identical bits."""
    P.peak_set_tuning(P.PEAK_TUNE_K_ORDER, 2)
    for idx, (ta, tb, M, N, K, bn, split) in enumerate([(0, 0, 2304, 3328, 1000, 0, 0), (1, 0, 2048, 4096, 712, 128, 0),
                                                        (0, 1, 3072, 2560, 1544, 512, 0), (1, 1, 1024, 1536, 2056, 256, 3)]):
        P.peak_set_tuning(P.PEAK_TUNE_TILE_N, bn)
        P.peak_set_tuning(P.PEAK_TUNE_SPLIT_K, split)
        c = mk(W.PEAK_BF16_F32, ta, tb, M, N, K, dist="smallint", alpha=1.0, beta=-1.0, case=idx)
        dc = R.DeviceCase(c)
        dc.run(variant)
        first = dc.result().copy()
        ref, _ = dc.oracle_sub(*R.sample_grid(c, 128, 128, 3e8))
        rows, cols = R.sample_grid(c, 128, 128, 3e8)
        assert np.array_equal(first[np.ix_(rows, cols)].view(np.uint32), oracle.round_to(oracle.F32, ref)), f"{c}"
        dc.reset_c()
        dc.run(variant)
        assert np.array_equal(dc.result(), first)


# ------------------------------------------------------------------ k-slices on the CTAs of a cluster
@pytest.mark.parametrize("ta,tb", LAYOUTS)
def test_cluster_k_slices_exact(ta, tb, reset_tuning):
    """Every tile split 2 or 4 ways on single-CTA tiles runs as one launch: the slices on the CTAs of a cluster,
    added through distributed shared memory in slice order.  Exact on integers for ragged M, N, K (several tile
    rows, last slice shorter, slices narrower than a store chunk), every output type, 8-bit inputs, alpha / beta,
    TMA and direct stores; the workspace path (PEAK_TUNE_CLUSTER_K = 1) gives the same bits."""
    shapes = [(16, 4096, 1024), (1, 128, 512), (100, 1000, 2056), (128, 264, 1100), (300, 520, 1544), (130, 77, 4100)]
    for idx, (M, N, K) in enumerate(shapes):
        for dtype in (W.PEAK_BF16_BF16, W.PEAK_F16_F32, W.PEAK_F16_F16, W.PEAK_E4M3_BF16, W.PEAK_E5M2_F32):
            in8 = dtype in (W.PEAK_E4M3_BF16, W.PEAK_E5M2_F32)
            unit = 16 if in8 else 8
            pa, pb = (-(M if ta else K)) % unit, (-(K if tb else N)) % unit
            c = mk(dtype, ta, tb, M, N, K, dist="smallint", alpha=0.5 if dtype != W.PEAK_F16_F32 else 2.0,
                   beta=[0.0, 1.0, -2.0][idx % 3], pad_a=pa, pad_b=pb, pad_c=[0, 8, 3][idx % 3], case=idx)
            kblocks = (K + (127 if in8 else 63)) // (128 if in8 else 64)
            for bn in (128, 256):
                for split in (2, 4):
                    per = (kblocks + split - 1) // split
                    if per * (split - 1) >= kblocks:
                        continue                                  # a slice would be empty: the library refuses
                    P.peak_set_tuning(P.PEAK_TUNE_TILE_N, bn)
                    P.peak_set_tuning(P.PEAK_TUNE_SPLIT_K, split)
                    outs = []
                    for mode in (0, 1):
                        P.peak_set_tuning(P.PEAK_TUNE_CLUSTER_K, mode)
                        dc = R.DeviceCase(c)
                        dc.run(P.PEAK_VARIANT_UMMA_1CTA)
                        name = P.peak_last_kernel()
                        assert ("umma_clusterk_kernel<%d," % bn in name) == (mode == 0), name
                        ref, _ = dc.oracle_full()
                        want = oracle.round_to(R.OT[c.out_type], ref)
                        got = dc.result()
                        got = got.view(np.uint32) if c.out_type == "f32" else got
                        assert np.array_equal(got, want), f"{c} bn={bn} split={split} cluster_k={mode}"
                        outs.append(got.copy())
                    assert np.array_equal(outs[0], outs[1])


def test_cluster_k_real_values_fused_tail_and_selection(reset_tuning):
    """Real-valued inputs through the cluster-split kernel with bias, GELU and a residual, run twice (bitwise
    repeatable); and the dispatcher's own choice: a skinny problem whose 128-wide tiles fill a quarter of the SMs
    runs four slices per tile in one launch."""
    from tests.test_gpu_fused import run_fused, check_fused, make_residual
    rng = np.random.default_rng(41)
    for idx, (ta, tb, M, N, K, a, b) in enumerate([(1, 0, 16, 4096, 4096, 0.5, 2.0), (0, 1, 128, 1100, 2056, 1.0, 0.0),
                                                   (0, 0, 200, 512, 1000, -1.0, 1.0), (1, 1, 5, 300, 1096, 2.0, 0.0)]):
        pa, pb = (-(M if ta else K)) % 8, (-(K if tb else N)) % 8
        c = W.GemmCase(f"ck{idx}", W.PEAK_BF16_BF16 if idx % 2 == 0 else W.PEAK_F16_F32, bool(ta), bool(tb), M, N, K, a, b,
                       "uniform", pad_a=pa, pad_b=pb, pad_c=idx, case=idx)
        for bn, split in ((128, 4), (256, 2)):
            P.peak_set_tuning(P.PEAK_TUNE_TILE_N, bn)
            P.peak_set_tuning(P.PEAK_TUNE_SPLIT_K, split)
            dc = R.DeviceCase(c)
            dc.run(P.PEAK_VARIANT_UMMA_1CTA)
            assert "umma_clusterk_kernel" in P.peak_last_kernel()
            R.check_full(dc, what=f"{c} bn={bn} split={split}")
            first = dc.result().copy()
            dc.reset_c()
            dc.run(P.PEAK_VARIANT_UMMA_1CTA)
            assert np.array_equal(first, dc.result())
            bias = (rng.standard_normal(N) * 2).astype(np.float32)
            res = make_residual(c, rng, idx)
            dcf = run_fused(c, P.PEAK_VARIANT_UMMA_1CTA, bias, P.PEAK_ACT_GELU, res)
            assert "umma_clusterk_kernel" in P.peak_last_kernel()
            check_fused(dcf, bias, P.PEAK_ACT_GELU, f"cluster-k fused {c} bn={bn} split={split}", res)
    for k in range(P.PEAK_TUNE_COUNT):
        P.peak_set_tuning(k, 0)
    c = W.config4_ragged(1)
    dc = R.DeviceCase(c)
    dc.run(P.PEAK_VARIANT_AUTO)
    assert "umma_clusterk_kernel<128, __nv_bfloat16, 4, 0>" in P.peak_last_kernel(), P.peak_last_kernel()
    R.check_full(dc, what=c.name)
    P.peak_set_tuning(P.PEAK_TUNE_CLUSTER_K, 1)
    dc = R.DeviceCase(c)
    dc.run(P.PEAK_VARIANT_AUTO)
    assert "umma_gemm_kernel<1," in P.peak_last_kernel()
    R.check_full(dc, what=c.name)
    # fewer tiles than an eighth of the SMs: four slices in a cluster from 16 to 160 k-blocks (exact on integers,
    # ragged edges included), the workspace split beyond
    P.peak_set_tuning(P.PEAK_TUNE_CLUSTER_K, 0)
    for idx, (ta, tb, M, N, K, four) in enumerate([(0, 1, 256, 512, 4096, True), (0, 0, 250, 300, 1032, True),
                                                   (1, 1, 16, 1000, 10240, True), (0, 1, 128, 256, 16384, False)]):
        pa, pb = (-(M if ta else K)) % 8, (-(K if tb else N)) % 8
        c = mk(W.PEAK_BF16_BF16 if idx % 2 == 0 else W.PEAK_F16_F32, ta, tb, M, N, K, dist="smallint", alpha=0.5,
               beta=[0.0, 1.0][idx % 2], pad_a=pa, pad_b=pb, pad_c=idx, case=idx)
        dc = R.DeviceCase(c)
        dc.run(P.PEAK_VARIANT_AUTO)
        name = P.peak_last_kernel()
        assert ("umma_clusterk_kernel<128," in name and ", 4, 0>" in name) == four, name
        R.check_full(dc, what=f"few tiles {c}")


def test_short_k_epilogue_bound_exact_and_selected(reset_tuning):
    """Problems of more than a wave whose tiles have few k-blocks are bounded by the epilogue: up to four k-blocks
    (eight with beta != 0) they take single-CTA 128 x 256 tiles with eight epilogue warps; pair tiles forced onto
    them take the 512-wide tile up to four k-blocks and eight epilogue warps up to eight.  beta = 0 runs the
    plain-store loop (ragged last chunk of a row, odd chunk counts, rows beyond M), beta != 0 and the fused tail the
    general one; exact on integers for 16-bit and 8-bit inputs and for a 32-bit output, bitwise repeatable."""
    A, P2 = P.PEAK_VARIANT_AUTO, P.PEAK_VARIANT_UMMA_2CTA
    cases = [(0, 1, 2304, 2560, 64, W.PEAK_BF16_BF16, 0.0, A, "<1, 256,"), (0, 0, 2300, 2504, 200, W.PEAK_BF16_BF16, 0.0, A, "0, 0, 1, 0>"),
             (1, 0, 2304, 2568, 256, W.PEAK_F16_F32, 0.0, A, "<1, 256,"), (1, 1, 2200, 2560, 136, W.PEAK_BF16_BF16, -1.0, A, "<1, 256,"),
             (0, 1, 2304, 2560, 512, W.PEAK_E4M3_BF16, 0.0, A, "<1, 256,"), (0, 0, 2304, 2600, 448, W.PEAK_F16_F16, 2.0, A, "<1, 256,"),
             (0, 1, 2304, 2560, 64, W.PEAK_BF16_BF16, 0.0, P2, "<2, 512,"), (0, 0, 2300, 2504, 200, W.PEAK_BF16_BF16, 0.0, P2, "<2, 512,"),
             (1, 0, 2304, 2568, 256, W.PEAK_F16_F32, 0.0, P2, "<2, 512,"), (0, 1, 2304, 2560, 512, W.PEAK_E4M3_BF16, 0.0, P2, "<2, 512,"),
             (0, 1, 2304, 2560, 448, W.PEAK_BF16_BF16, 0.0, A, "<2, 256, __nv_bfloat16, 0, 0, 0, 1, 0>"),
             (0, 0, 2304, 2600, 320, W.PEAK_F16_F16, 2.0, P2, "0, 0, 1, 0>")]
    for idx, (ta, tb, M, N, K, dtype, beta, variant, tag) in enumerate(cases):
        unit = 16 if dtype == W.PEAK_E4M3_BF16 else 8
        pa, pb = (-(M if ta else K)) % unit, (-(K if tb else N)) % unit
        c = mk(dtype, ta, tb, M, N, K, dist="smallint", alpha=0.5, beta=beta, pad_a=pa, pad_b=pb, pad_c=[0, 8][idx % 2], case=idx)
        dc = R.DeviceCase(c)
        dc.run(variant)
        assert "umma_gemm_kernel" in P.peak_last_kernel() and tag in P.peak_last_kernel(), P.peak_last_kernel()
        R.check_full(dc, what=f"short k {c}")
        first = dc.result().copy()
        dc.reset_c()
        dc.run(variant)
        assert np.array_equal(first, dc.result())
    # real values with bias and GELU through the general loop of the same kernels
    from tests.test_gpu_fused import run_fused, check_fused
    rng = np.random.default_rng(77)
    c = W.GemmCase("shortk_fused", W.PEAK_BF16_BF16, False, True, 2304, 2560, 192, 1.0, 0.0, "uniform", case=9)
    bias = (rng.standard_normal(c.N) * 2).astype(np.float32)
    dcf = run_fused(c, P.PEAK_VARIANT_AUTO, bias, P.PEAK_ACT_GELU, None)
    check_fused(dcf, bias, P.PEAK_ACT_GELU, "short k fused", None)


def test_one_tile_per_cta_kernel_two_issuers_exact(reset_tuning):
    """Whole 128-wide tiles that all run at once take the one-tile-per-CTA kernel without a cluster: two MMA
    issuers accumulate the even and the odd k-blocks separately and the epilogue adds them.  Exact on integers in
    every layout for one k-block (second accumulator never written), odd and even counts, ragged edges, every
    output type, beta != 0 with TMA and direct stores; real values within the bounds, bitwise repeatable; the
    persistent kernel (PEAK_TUNE_CLUSTER_K = 1) gives the same bits on integers."""
    shapes = [(128, 1024, 64), (100, 1000, 136), (300, 520, 1544), (128, 4100, 520), (512, 1280, 4096), (7, 130, 200)]
    for ta, tb in LAYOUTS:
        for idx, (M, N, K) in enumerate(shapes):
            for dtype in (W.PEAK_BF16_BF16, W.PEAK_F16_F32, W.PEAK_F16_F16, W.PEAK_E4M3_BF16):
                unit = 16 if dtype == W.PEAK_E4M3_BF16 else 8
                pa, pb = (-(M if ta else K)) % unit, (-(K if tb else N)) % unit
                c = mk(dtype, ta, tb, M, N, K, dist="smallint", alpha=0.5, beta=[0.0, 1.0, -2.0][idx % 3], pad_a=pa,
                       pad_b=pb, pad_c=[0, 8, 3][idx % 3], case=idx)
                P.peak_set_tuning(P.PEAK_TUNE_TILE_N, 128)
                P.peak_set_tuning(P.PEAK_TUNE_SPLIT_K, 1)
                outs = []
                for mode in (0, 1):
                    P.peak_set_tuning(P.PEAK_TUNE_CLUSTER_K, mode)
                    dc = R.DeviceCase(c)
                    dc.run(P.PEAK_VARIANT_UMMA_1CTA)
                    name = P.peak_last_kernel()
                    assert ("umma_clusterk_kernel<128," in name and ", 1, " in name) == (mode == 0), name
                    ref, _ = dc.oracle_full()
                    want = oracle.round_to(R.OT[c.out_type], ref)
                    got = dc.result()
                    got = got.view(np.uint32) if c.out_type == "f32" else got
                    assert np.array_equal(got, want), f"{c} cluster_k={mode}"
                    outs.append(got.copy())
                assert np.array_equal(outs[0], outs[1])
    for k in range(P.PEAK_TUNE_COUNT):
        P.peak_set_tuning(k, 0)
    c = mk(W.PEAK_BF16_BF16, 1, 0, 128, 14336, 1024, alpha=0.5, beta=2.0)
    dc = R.DeviceCase(c)
    dc.run(P.PEAK_VARIANT_AUTO)
    assert "umma_clusterk_kernel<128, __nv_bfloat16, 1, 0>" in P.peak_last_kernel(), P.peak_last_kernel()
    R.check_full(dc, what=f"{c}")
    first = dc.result().copy()
    dc.reset_c()
    dc.run(P.PEAK_VARIANT_AUTO)
    assert np.array_equal(first, dc.result())


@pytest.mark.parametrize("ta,tb", LAYOUTS)
def test_one_tile_per_pair_kernel_exact(ta, tb, reset_tuning):
    """Whole tiles of a one-wave problem with at least two 128-row blocks run as 256 x 128 CTA-pair tiles (the pair's
    leader issues cta_group::2 MMAs from two threads into two accumulators; each CTA stages its rows of A and its
    half of the B tile).  Exact on integers in every layout for ragged M (a pair whose second CTA has no rows), N,
    K, one k-block, odd counts, every output type, 8-bit inputs with B stored N x K, beta != 0, whole and in two
    k-slices (the two pairs of a four-CTA cluster exchange their partial sums); the same bits as single-CTA tiles;
    chosen by the dispatcher from 32 k-blocks on."""
    shapes = [(256, 1024, 64), (300, 1000, 136), (129, 520, 1544), (512, 4100, 520), (700, 1152, 2056)]
    for idx, (M, N, K) in enumerate(shapes):
        pair_tiles = ((M + 255) // 256) * ((N + 127) // 128)   # 8, 16, 5, 66 (too many four-CTA clusters at once), 27
        for dtype in (W.PEAK_BF16_BF16, W.PEAK_F16_F32, W.PEAK_F16_F16, W.PEAK_E4M3_BF16):
            in8 = dtype == W.PEAK_E4M3_BF16
            if in8 and not tb:
                continue
            unit = 16 if in8 else 8
            pa, pb = (-(M if ta else K)) % unit, (-(K if tb else N)) % unit
            c = mk(dtype, ta, tb, M, N, K, dist="smallint", alpha=0.5, beta=[0.0, 1.0, -2.0][idx % 3], pad_a=pa, pad_b=pb,
                   pad_c=[0, 8, 3][idx % 3], case=idx)
            outs = []
            kblocks = (K + (127 if in8 else 63)) // (128 if in8 else 64)
            for mode, split in ((4, 1), (3, 1), (4, 2), (3, 2)):
                if split == 2 and kblocks < 2:
                    continue
                P.peak_set_tuning(P.PEAK_TUNE_TILE_N, 128)
                P.peak_set_tuning(P.PEAK_TUNE_SPLIT_K, split)
                P.peak_set_tuning(P.PEAK_TUNE_CLUSTER_K, mode)
                dc = R.DeviceCase(c)
                dc.run(P.PEAK_VARIANT_UMMA_1CTA)
                name = P.peak_last_kernel()
                # (two k-slices of pair tiles -- the two pairs of a four-CTA cluster -- exist for 16-bit inputs)
                pair = mode == 4 and not (split == 2 and (in8 or pair_tiles > 40))
                assert f"umma_clusterk_kernel<128," in name and f", {split}, " in name and (", 2> " in name) == pair, name
                ref, _ = dc.oracle_full()
                want = oracle.round_to(R.OT[c.out_type], ref)
                got = dc.result()
                got = got.view(np.uint32) if c.out_type == "f32" else got
                assert np.array_equal(got, want), f"{c} cluster_k={mode} split={split}"
                outs.append(got.copy())
            assert all(np.array_equal(outs[0], o) for o in outs[1:])
    for k in range(P.PEAK_TUNE_COUNT):
        P.peak_set_tuning(k, 0)
    c = mk(W.PEAK_BF16_BF16, ta, tb, 512, 4096, 2048, alpha=0.5, beta=2.0)
    dc = R.DeviceCase(c)
    dc.run(P.PEAK_VARIANT_AUTO)
    assert "umma_clusterk_kernel<128, __nv_bfloat16, 1, 0, 2>" in P.peak_last_kernel(), P.peak_last_kernel()
    R.check_sampled(dc, tile_m=256, tile_n=128, what=f"{c}")
    first = dc.result().copy()
    dc.reset_c()
    dc.run(P.PEAK_VARIANT_AUTO)
    assert np.array_equal(first, dc.result())


@pytest.mark.parametrize("ta,tb", LAYOUTS)
def test_one_wave_of_256_wide_pair_tiles_exact(ta, tb, reset_tuning):
    """At most one 256 x 256 tile per CTA pair: the one-tile kernel's pair form with a 256-wide tile (one issuer, two
    producers per CTA, two groups of epilogue warps).  Exact on integers for ragged shapes, every output type,
    beta != 0, the fused tail; the same bits as the persistent kernel (PEAK_TUNE_CLUSTER_K = 3) and on 192-column
    tiles (B with k contiguous; chosen where they still make one wave); not used when the tiles need more than
    one wave."""
    from tests.test_gpu_fused import run_fused, check_fused, make_residual
    rng = np.random.default_rng(53)
    for idx, (M, N, K) in enumerate([(512, 768, 256), (700, 1000, 264), (130, 2000, 72), (1024, 1920, 1032)]):
        for dtype in (W.PEAK_BF16_BF16, W.PEAK_F16_F32, W.PEAK_F16_F16):
            pa, pb = (-(M if ta else K)) % 8, (-(K if tb else N)) % 8
            c = mk(dtype, ta, tb, M, N, K, dist="smallint", alpha=0.5, beta=[0.0, 1.0, -2.0][idx % 3], pad_a=pa, pad_b=pb,
                   pad_c=[0, 8, 3][idx % 3], case=idx)
            outs = []
            for mode in (0, 3):
                P.peak_set_tuning(P.PEAK_TUNE_CLUSTER_K, mode)
                P.peak_set_tuning(P.PEAK_TUNE_TILE_N, 256)
                P.peak_set_tuning(P.PEAK_TUNE_MULTICAST, 1)
                dc = R.DeviceCase(c)
                dc.run(P.PEAK_VARIANT_UMMA_2CTA)
                name = P.peak_last_kernel()
                assert ("umma_clusterk_kernel<256," in name and ", 2> " in name) == (mode == 0), name
                ref, _ = dc.oracle_full()
                want = oracle.round_to(R.OT[c.out_type], ref)
                got = dc.result()
                got = got.view(np.uint32) if c.out_type == "f32" else got
                assert np.array_equal(got, want), f"{c} cluster_k={mode}"
                outs.append(got.copy())
            if tb:   # B with k contiguous: the same kernel on 192-column tiles
                P.peak_set_tuning(P.PEAK_TUNE_CLUSTER_K, 0)
                P.peak_set_tuning(P.PEAK_TUNE_TILE_N, 192)
                dc = R.DeviceCase(c)
                dc.run(P.PEAK_VARIANT_UMMA_2CTA)
                name = P.peak_last_kernel()
                assert "umma_clusterk_kernel<256," in name and "width=192" in name, name
                got = dc.result()
                got = got.view(np.uint32) if c.out_type == "f32" else got
                assert np.array_equal(got, want), f"{c} width=192"
            assert np.array_equal(outs[0], outs[1])
    for k in range(P.PEAK_TUNE_COUNT):
        P.peak_set_tuning(k, 0)
    if tb:
        c = mk(W.PEAK_BF16_BF16, ta, tb, 768, 4096, 256, alpha=0.5, beta=2.0)      # 66 tiles of 192 against 48 of 256
        dc = R.DeviceCase(c)
        dc.run(P.PEAK_VARIANT_AUTO)
        assert "width=192" in P.peak_last_kernel(), P.peak_last_kernel()
        R.check_full(dc, what=f"{c}")
    c = W.GemmCase("one_wave_fused", W.PEAK_BF16_BF16, bool(ta), bool(tb), 520, 1100, 264, 0.5, 2.0, "uniform",
                   pad_a=(-(520 if ta else 264)) % 8, pad_b=(-(264 if tb else 1100)) % 8)
    bias = rng.standard_normal(c.N).astype(np.float32)
    res = make_residual(c, rng, 2)
    P.peak_set_tuning(P.PEAK_TUNE_TILE_N, 256)
    dc = run_fused(c, P.PEAK_VARIANT_UMMA_2CTA, bias, P.PEAK_ACT_GELU, res)
    assert "umma_clusterk_kernel<256," in P.peak_last_kernel(), P.peak_last_kernel()
    check_fused(dc, bias, P.PEAK_ACT_GELU, f"one wave of pair tiles, fused {c.layout}", res)
    big = mk(W.PEAK_BF16_BF16, ta, tb, 2560, 2304, 128, dist="smallint")     # 90 tiles: more than one per pair
    dc = R.DeviceCase(big)
    P.peak_set_tuning(P.PEAK_TUNE_MULTICAST, 1)
    dc.run(P.PEAK_VARIANT_UMMA_2CTA)
    assert "umma_gemm_kernel<2," in P.peak_last_kernel(), P.peak_last_kernel()


def test_cluster_k_bounded_wait_reports_timeout(reset_tuning):
    """The stalled-stage hook in the cluster-split kernel: the CTA whose stage never fills gives up after its
    budget, still reaches both cluster barriers (its peers wait there, not on a flag), the status word reports the
    timeout once and the context computes correctly afterwards."""
    c = mk(W.PEAK_BF16_BF16, 0, 1, 128, 512, 2048)
    dc = R.DeviceCase(c)
    P.peak_set_tuning(P.PEAK_TUNE_TILE_N, 128)
    P.peak_set_tuning(P.PEAK_TUNE_SPLIT_K, 4)
    P.peak_set_tuning(P.PEAK_TUNE_WAIT_MS, 20)
    P.peak_set_tuning(P.PEAK_TUNE_INJECT_STALL, 1)
    P.peak_gemm_variant(P.PEAK_VARIANT_UMMA_1CTA, c.dtype, c.transA, c.transB, c.M, c.N, c.K, 1.0, dc.A, c.lda, dc.B, c.ldb,
                        0.0, dc.C, c.ldc)
    assert "umma_clusterk_kernel" in P.peak_last_kernel()
    rc, detail = P.peak_check()
    assert rc == P.PEAK_ERR_TIMEOUT and (detail & 0x80000000)
    assert P.peak_check()[0] == P.PEAK_OK
    P.peak_set_tuning(P.PEAK_TUNE_INJECT_STALL, 0)
    P.peak_set_tuning(P.PEAK_TUNE_WAIT_MS, 0)
    dc.reset_c()
    dc.run(P.PEAK_VARIANT_UMMA_1CTA)
    assert "umma_clusterk_kernel" in P.peak_last_kernel()
    R.check_full(dc)
    # the same with whole 256 x 128 pair tiles: the leader's last stage never fills, both CTAs of the pair unwind
    c = mk(W.PEAK_BF16_BF16, 0, 1, 256, 512, 2048)
    dc = R.DeviceCase(c)
    P.peak_set_tuning(P.PEAK_TUNE_SPLIT_K, 1)
    P.peak_set_tuning(P.PEAK_TUNE_CLUSTER_K, 4)
    P.peak_set_tuning(P.PEAK_TUNE_WAIT_MS, 20)
    P.peak_set_tuning(P.PEAK_TUNE_INJECT_STALL, 1)
    P.peak_gemm_variant(P.PEAK_VARIANT_UMMA_1CTA, c.dtype, c.transA, c.transB, c.M, c.N, c.K, 1.0, dc.A, c.lda, dc.B, c.ldb,
                        0.0, dc.C, c.ldc)
    assert ", 2> " in P.peak_last_kernel(), P.peak_last_kernel()
    rc, detail = P.peak_check()
    assert rc == P.PEAK_ERR_TIMEOUT and (detail & 0x80000000)
    P.peak_set_tuning(P.PEAK_TUNE_INJECT_STALL, 0)
    P.peak_set_tuning(P.PEAK_TUNE_WAIT_MS, 0)
    dc.reset_c()
    dc.run(P.PEAK_VARIANT_UMMA_1CTA)
    assert ", 2> " in P.peak_last_kernel()
    R.check_full(dc)


@pytest.mark.parametrize("ta,tb", LAYOUTS)
def test_shared_operand_clusters_plugin_exact(ta, tb, reset_tuning):
    """The plug-in's single-CTA tiles in clusters of CM x CN tiles that share A / B tiles by multicast copies
    (PEAK_TUNE_SHARE = 100 w + 10 CM + CN): every cluster shape, exact on integers for ragged shapes (clusters
    that reach beyond the matrix), alpha / beta, 16-bit and fp32 output, and the same bits as the main library's
    own kernels."""
    if not P.peak_multicast_available():
        pytest.skip("libpeak_gemm_mc.so is not present (multi-GPU runs leave it out)")
    for idx, (M, N, K) in enumerate([(128, 1024, 512), (100, 1000, 264), (512, 512, 64), (300, 900, 1096)]):
        for dtype in (W.PEAK_BF16_BF16, W.PEAK_F16_F32):
            pa, pb = (-(M if ta else K)) % 8, (-(K if tb else N)) % 8
            c = mk(dtype, ta, tb, M, N, K, dist="smallint", alpha=0.5, beta=[1.0, 0.0][idx % 2], pad_a=pa, pad_b=pb,
                   pad_c=[0, 8][idx % 2], case=idx)
            want = None
            for mode in (1, 112, 114, 121, 122, 124, 141, 142, 212, 214, 221, 222):
                P.peak_set_tuning(P.PEAK_TUNE_SHARE, mode)
                dc = R.DeviceCase(c)
                dc.run(P.PEAK_VARIANT_AUTO)
                assert ("umma_share_kernel" in P.peak_last_kernel()) == (mode != 1), P.peak_last_kernel()
                got = dc.result()
                got = got.view(np.uint32) if c.out_type == "f32" else got
                if want is None:
                    ref, _ = dc.oracle_full()
                    want = oracle.round_to(R.OT[c.out_type], ref)
                assert np.array_equal(got, want), f"{c} share={mode}"


def test_shared_operand_clusters_bounded_wait(reset_tuning):
    """The stalled-stage hook in the shared-operand kernel: one CTA never sends its parts of the last stage, so
    its own and its peers' waits run out; every CTA still reaches the closing cluster barrier, the timeout is
    reported once and the context computes correctly afterwards."""
    if not P.peak_multicast_available():
        pytest.skip("libpeak_gemm_mc.so is not present (multi-GPU runs leave it out)")
    c = mk(W.PEAK_BF16_BF16, 0, 1, 256, 512, 1024)
    dc = R.DeviceCase(c)
    P.peak_set_tuning(P.PEAK_TUNE_SHARE, 122)
    P.peak_set_tuning(P.PEAK_TUNE_WAIT_MS, 20)
    P.peak_set_tuning(P.PEAK_TUNE_INJECT_STALL, 1)
    P.peak_gemm_variant(P.PEAK_VARIANT_AUTO, c.dtype, c.transA, c.transB, c.M, c.N, c.K, 1.0, dc.A, c.lda, dc.B, c.ldb,
                        0.0, dc.C, c.ldc)
    assert "umma_share_kernel" in P.peak_last_kernel()
    rc, detail = P.peak_check()
    assert rc == P.PEAK_ERR_TIMEOUT and (detail & 0x80000000)
    assert P.peak_check()[0] == P.PEAK_OK
    P.peak_set_tuning(P.PEAK_TUNE_INJECT_STALL, 0)
    P.peak_set_tuning(P.PEAK_TUNE_WAIT_MS, 0)
    dc.reset_c()
    dc.run(P.PEAK_VARIANT_AUTO)
    assert "umma_share_kernel" in P.peak_last_kernel()
    R.check_full(dc)


@pytest.mark.parametrize("ta,tb", [(0, 1), (1, 1)])
def test_narrower_pair_tiles_exact_and_selected(ta, tb, reset_tuning):
    """CTA-pair tiles of 192 / 384 columns on the 256- / 512-wide kernels (B with k contiguous): exact on integers
    for ragged shapes, alpha / beta (old C by TMA and by per-thread loads), fp32 and 16-bit outputs, 8-bit inputs, one
    and two groups of epilogue warps, the fused tail; the same bits as the full-width tiles; chosen by the dispatcher
    where one wave of 384-wide tiles replaces a poorly filled wave of 512-wide ones."""
    from tests.test_gpu_fused import run_fused, check_fused, make_residual
    rng = np.random.default_rng(47)
    for idx, (M, N, K) in enumerate([(512, 768, 256), (700, 1000, 264), (1024, 1920, 520), (300, 400, 72), (260, 2304, 136)]):
        for dtype in (W.PEAK_BF16_BF16, W.PEAK_F16_F32, W.PEAK_E4M3_BF16):
            unit = 16 if dtype == W.PEAK_E4M3_BF16 else 8
            pa, pb = (-(M if ta else K)) % unit, (-(K if tb else N)) % unit
            c = mk(dtype, ta, tb, M, N, K, dist="smallint", alpha=0.5, beta=[0.0, 1.0, -2.0][idx % 3], pad_a=pa, pad_b=pb,
                   pad_c=[0, 8, 3][idx % 3], case=idx)
            want = None
            for width in (0, 192, 384):
                for epi, warps in ((0, 0), (3, 1), (1, 2)):
                    P.peak_set_tuning(P.PEAK_TUNE_TILE_N, width)
                    P.peak_set_tuning(P.PEAK_TUNE_EPILOGUE, epi)
                    P.peak_set_tuning(P.PEAK_TUNE_EPILOGUE_WARPS, warps)
                    P.peak_set_tuning(P.PEAK_TUNE_MULTICAST, 1)
                    dc = R.DeviceCase(c)
                    dc.run(P.PEAK_VARIANT_UMMA_2CTA)
                    assert (f"width={width}" in P.peak_last_kernel()) == (width != 0), P.peak_last_kernel()
                    got = dc.result()
                    got = got.view(np.uint32) if c.out_type == "f32" else got
                    if want is None:
                        ref, _ = dc.oracle_full()
                        want = oracle.round_to(R.OT[c.out_type], ref)
                    assert np.array_equal(got, want), f"{c} width={width} epilogue={epi} warps={warps}"
    for k in range(P.PEAK_TUNE_COUNT):
        P.peak_set_tuning(k, 0)
    c = W.GemmCase("narrow_fused", W.PEAK_BF16_BF16, bool(ta), bool(tb), 520, 1100, 264, 0.5, 2.0, "uniform", pad_a=(-(520 if ta else 264)) % 8,
                   pad_b=0)
    bias = rng.standard_normal(c.N).astype(np.float32)
    res = make_residual(c, rng, 2)
    for width in (192, 384):
        P.peak_set_tuning(P.PEAK_TUNE_TILE_N, width)
        dc = run_fused(c, P.PEAK_VARIANT_UMMA_2CTA, bias, P.PEAK_ACT_GELU, res)
        assert f"width={width}" in P.peak_last_kernel()
        check_fused(dc, bias, P.PEAK_ACT_GELU, f"narrow tiles fused {c.layout} width={width}", res)
    P.peak_set_tuning(P.PEAK_TUNE_TILE_N, 0)
    big = mk(W.PEAK_BF16_BF16, ta, tb, 2560, 2560, 2560, pad_a=0, pad_b=0)
    dc = R.DeviceCase(big)
    dc.run(P.PEAK_VARIANT_AUTO)
    assert "width=384" in P.peak_last_kernel(), P.peak_last_kernel()
    R.check_sampled(dc, tile_m=256, tile_n=384, what="2560^3 on 384-wide tiles")
    P.peak_set_tuning(P.PEAK_TUNE_NARROW, 1)
    dc.reset_c()
    dc.run(P.PEAK_VARIANT_AUTO)
    assert "width=" not in P.peak_last_kernel()


# ------------------------------------------------------------------ exchanged operands (M <= 64)
@pytest.mark.parametrize("ta,tb", LAYOUTS)
def test_swapped_operands_exact_and_selected(ta, tb, reset_tuning):
    """With PEAK_TUNE_SWAP_AB = 2, problems with M <= 64 are computed as C^T = op(B)^T op(A)^T on single-CTA tiles
    with a 64-wide MMA N and written back transposed: exact on integers for ragged M, N, K, every output type,
    alpha / beta, with and without a k-split; without the knob the plain tiles run."""
    P.peak_set_tuning(P.PEAK_TUNE_SWAP_AB, 2)
    shapes = [(16, 4096, 1024), (1, 128, 64), (7, 1000, 200), (33, 520, 1544), (64, 257, 72), (48, 2048, 4100)]
    for idx, (M, N, K) in enumerate(shapes):
        for dtype in (W.PEAK_BF16_BF16, W.PEAK_F16_F32, W.PEAK_F16_F16):
            pa, pb = (-(M if ta else K)) % 8, (-(K if tb else N)) % 8
            c = mk(dtype, ta, tb, M, N, K, dist="smallint", alpha=0.5 if dtype != W.PEAK_F16_F32 else 2.0,
                   beta=[0.0, 1.0, -2.0][idx % 3], pad_a=pa, pad_b=pb, pad_c=idx % 2, case=idx)
            for split in (0, 1, 3):
                if split > max(1, (K + 63) // 64):
                    continue
                P.peak_set_tuning(P.PEAK_TUNE_SPLIT_K, split)
                dc = R.DeviceCase(c)
                dc.run(P.PEAK_VARIANT_AUTO)
                name = P.peak_last_kernel()
                assert "umma_gemm_kernel<1, 64," in name and ", 1> " in name, name
                ref, _ = dc.oracle_full()
                want = oracle.round_to(R.OT[c.out_type], ref)
                got = dc.result()
                got = got.view(np.uint32) if c.out_type == "f32" else got
                assert np.array_equal(got, want), f"{c} split={split}"
    P.peak_set_tuning(P.PEAK_TUNE_SPLIT_K, 0)
    P.peak_set_tuning(P.PEAK_TUNE_SWAP_AB, 0)
    c = mk(W.PEAK_BF16_BF16, ta, tb, 16, 1024, 512, dist="smallint", pad_a=(-(16 if ta else 512)) % 8)
    dc = R.DeviceCase(c)
    dc.run(P.PEAK_VARIANT_AUTO)
    assert ", 0> " in P.peak_last_kernel()


def test_swapped_operands_real_values_and_fused_tail(reset_tuning):
    """Real-valued inputs through the exchanged-operand kernel, with bias (one value per column of C, i.e. per
    accumulator row), GELU and a residual; whole tiles and k-slices."""
    from tests.test_gpu_fused import run_fused, check_fused, make_residual
    rng = np.random.default_rng(31)
    P.peak_set_tuning(P.PEAK_TUNE_SWAP_AB, 2)
    for idx, (ta, tb, M, N, K, a, b) in enumerate([(1, 0, 16, 4096, 4096, 0.5, 2.0), (0, 1, 40, 1100, 520, 1.0, 0.0),
                                                   (0, 0, 64, 512, 1000, -1.0, 1.0), (1, 1, 5, 300, 136, 2.0, 0.0)]):
        pa, pb = (-(M if ta else K)) % 8, (-(K if tb else N)) % 8
        c = W.GemmCase(f"swap{idx}", W.PEAK_BF16_BF16 if idx % 2 == 0 else W.PEAK_F16_F32, bool(ta), bool(tb), M, N, K, a, b,
                       "uniform", pad_a=pa, pad_b=pb, pad_c=idx, case=idx)
        dc = R.DeviceCase(c)
        dc.run(P.PEAK_VARIANT_AUTO)
        assert ", 1> " in P.peak_last_kernel()
        R.check_full(dc, what=f"{c}")
        bias = (rng.standard_normal(N) * 2).astype(np.float32)
        res = make_residual(c, rng, idx)
        for split in (0, 2):
            P.peak_set_tuning(P.PEAK_TUNE_SPLIT_K, split)
            dcf = run_fused(c, P.PEAK_VARIANT_AUTO, bias, P.PEAK_ACT_GELU, res)
            assert ", 1> " in P.peak_last_kernel()
            check_fused(dcf, bias, P.PEAK_ACT_GELU, f"swapped fused {c} split={split}", res)
        P.peak_set_tuning(P.PEAK_TUNE_SPLIT_K, 0)


@pytest.mark.parametrize("ta,tb", LAYOUTS)
def test_short_a_loads_exact(ta, tb, reset_tuning):
    """Problems with M < 128 on single-CTA tiles fetch only the rows of A that exist (rounded up to 8; whole
    64-row boxes when A is stored m-contiguous), so the rest of the A stage keeps whatever an earlier tile left
    there -- NaN patterns included -- and only accumulator rows that are never stored see it.  Exact on integers
    for M from 1 to 127 after a problem that filled every stage with NaNs, with and without a k-split and for
    8-bit inputs; PEAK_TUNE_SHORT_A = 1 (whole boxes) gives the same bits."""
    nan_case = mk(W.PEAK_BF16_BF16, ta, tb, 128, 148 * 256, 512, dist="smallint", case=77)
    dn = R.DeviceCase(nan_case)                  # one tile on every SM, shared memory left full of NaN patterns
    dn.A.view(torch.int16).fill_(0x7FC0)
    dn.B.view(torch.int16).fill_(0x7FC0)
    for idx, (M, N, K) in enumerate([(1, 4096, 1024), (8, 136, 72), (9, 1000, 520), (16, 4096, 4096), (63, 264, 200),
                                     (65, 520, 136), (100, 2048, 1032), (127, 384, 4100)]):
        for dtype in (W.PEAK_BF16_BF16, W.PEAK_F16_F32, W.PEAK_E4M3_BF16):
            unit = 16 if dtype == W.PEAK_E4M3_BF16 else 8
            pa, pb = (-(M if ta else K)) % unit, (-(K if tb else N)) % unit
            c = mk(dtype, ta, tb, M, N, K, dist="smallint", alpha=0.5, beta=[0.0, 1.0][idx % 2], pad_a=pa, pad_b=pb,
                   case=idx)
            results = []
            for mode in (0, 1):
                for split in (0, 1, 4):
                    if split > max(1, (K + 63) // 64):
                        continue
                    P.peak_set_tuning(P.PEAK_TUNE_SHORT_A, 1)
                    P.peak_set_tuning(P.PEAK_TUNE_SPLIT_K, 1)
                    dn.run(P.PEAK_VARIANT_UMMA_1CTA)
                    P.peak_set_tuning(P.PEAK_TUNE_SHORT_A, mode)
                    P.peak_set_tuning(P.PEAK_TUNE_SPLIT_K, split)
                    dc = R.DeviceCase(c)
                    dc.run(P.PEAK_VARIANT_UMMA_1CTA)
                    ref, _ = dc.oracle_full()
                    want = oracle.round_to(R.OT[c.out_type], ref)
                    got = dc.result()
                    got = got.view(np.uint32) if c.out_type == "f32" else got
                    assert np.array_equal(got, want), f"{c} short_a={mode} split={split}"
                    results.append(got.copy())
            assert all(np.array_equal(results[0], r) for r in results[1:])


@pytest.mark.parametrize("ta,tb", LAYOUTS)
def test_sgemm_transposing_prepass_and_wide_register_tile(ta, tb, reset_tuning):
    """SGEMM with a k-contiguous operand copied, transposed, into pool memory first (PEAK_TUNE_SGEMM_TRANSPOSE = 2:
    always) and the 8 x 16 register-tile kernel on dense tiles: exact on integers for ragged shapes and padded
    pitches in every layout, within the fp32 bounds on reals with alpha / beta / bias / residual; with the knob at
    1 the direct kernels run and give the same bits on integers."""
    from tests.test_gpu_fused import run_fused, check_fused, make_residual
    rng = np.random.default_rng(41)
    for idx, (M, N, K) in enumerate([(1000, 1000, 1000), (129, 257, 33), (1, 300, 50), (512, 384, 528), (333, 70, 2050)]):
        pa, pb = (-(M if ta else K)) % 4 + 4 * (idx % 2), (-(K if tb else N)) % 4
        ci = mk(W.PEAK_F32_F32, ta, tb, M, N, K, dist="smallint", alpha=2.0, beta=-1.0, pad_a=pa, pad_b=pb, pad_c=idx % 3,
                case=idx)
        outs = []
        for mode in (2, 1):
            P.peak_set_tuning(P.PEAK_TUNE_SGEMM_TRANSPOSE, mode)
            dc = R.DeviceCase(ci)
            dc.run(P.PEAK_VARIANT_SGEMM)
            if mode == 2:
                assert "sgemm_tma_kernel<0, 0, 2, 1>" in P.peak_last_kernel(), P.peak_last_kernel()
            ref, _ = dc.oracle_full()
            assert np.array_equal(dc.result().view(np.uint32), oracle.round_to(oracle.F32, ref)), f"{ci} mode {mode}"
            outs.append(dc.result().copy())
        assert np.array_equal(outs[0], outs[1])
    P.peak_set_tuning(P.PEAK_TUNE_SGEMM_TRANSPOSE, 2)
    c = W.GemmCase("sg_tr_fused", W.PEAK_F32_F32, bool(ta), bool(tb), 520, 392, 264, 0.5, 2.0, "uniform")
    bias = rng.standard_normal(c.N).astype(np.float32)
    res = make_residual(c, rng, 4)
    dc = run_fused(c, P.PEAK_VARIANT_AUTO, bias, P.PEAK_ACT_GELU, res)
    check_fused(dc, bias, P.PEAK_ACT_GELU, f"sgemm transposed {c.layout}", res)


@pytest.mark.parametrize("ta,tb", LAYOUTS)
def test_sgemm_k_slices_exact_and_selected(ta, tb, reset_tuning):
    """SGEMM problems with fewer tiles than two blocks per SM are cut along k: every block stores the raw sums of
    its slice, a second kernel (a programmatic dependent) adds the slices in order and applies alpha / beta, bias,
    activation and residual.  Exact on integers in every layout for ragged shapes, forced slice counts (the last
    slice shorter), padded pitches; chosen by the dispatcher for small grids and not for large ones; bitwise
    repeatable on reals."""
    from tests.test_gpu_fused import run_fused, check_fused, make_residual
    rng = np.random.default_rng(43)
    for idx, (M, N, K) in enumerate([(256, 256, 256), (129, 257, 1000), (1, 300, 530), (512, 384, 528), (100, 70, 4100)]):
        pa, pb = (-(M if ta else K)) % 4 + 4 * (idx % 2), (-(K if tb else N)) % 4
        ci = mk(W.PEAK_F32_F32, ta, tb, M, N, K, dist="smallint", alpha=2.0, beta=-1.0, pad_a=pa, pad_b=pb, pad_c=idx % 3,
                case=idx)
        outs = []
        for split in (0, 1, 2, 3, 7):
            P.peak_set_tuning(P.PEAK_TUNE_SPLIT_K, split)
            dc = R.DeviceCase(ci)
            dc.run(P.PEAK_VARIANT_SGEMM)
            name = P.peak_last_kernel()
            slices = int(name.split("slices=")[1])
            if split == 0:
                assert slices > 1, name                      # a handful of tiles: the dispatcher cuts along k
            elif split == 1:
                assert slices == 1, name
            else:
                assert 1 < slices <= split, name
            ref, _ = dc.oracle_full()
            assert np.array_equal(dc.result().view(np.uint32), oracle.round_to(oracle.F32, ref)), f"{ci} split {split}"
            outs.append(dc.result().copy())
        assert all(np.array_equal(outs[0], o) for o in outs[1:])
    P.peak_set_tuning(P.PEAK_TUNE_SPLIT_K, 0)
    c = W.GemmCase("sg_slices_fused", W.PEAK_F32_F32, bool(ta), bool(tb), 520, 392, 1064, 0.5, 2.0, "uniform")
    bias = rng.standard_normal(c.N).astype(np.float32)
    res = make_residual(c, rng, 4)
    dc = run_fused(c, P.PEAK_VARIANT_AUTO, bias, P.PEAK_ACT_GELU, res)
    assert "slices=" in P.peak_last_kernel() and not P.peak_last_kernel().endswith("slices=1"), P.peak_last_kernel()
    check_fused(dc, bias, P.PEAK_ACT_GELU, f"sgemm k-slices fused {c.layout}", res)
    first = dc.result().copy()
    dc2 = run_fused(c, P.PEAK_VARIANT_AUTO, bias, P.PEAK_ACT_GELU, res)
    assert np.array_equal(first, dc2.result())
    big = mk(W.PEAK_F32_F32, ta, tb, 2304, 2304, 64, dist="smallint")     # 324 tiles: whole tiles
    dc = R.DeviceCase(big)
    dc.run(P.PEAK_VARIANT_AUTO)
    assert P.peak_last_kernel().endswith("slices=1"), P.peak_last_kernel()


def test_sgemm_tma_paths_in_a_cuda_graph_and_on_two_streams(reset_tuning):
    """The TMA-fed SGEMM inside a captured graph -- a ragged problem, and one whose k-contiguous operands are first
    transposed into pool memory (allocated and freed inside the capture) -- replayed twice; then the same two
    problems from two host threads on two streams at once."""
    import threading
    P.peak_set_tuning(P.PEAK_TUNE_SGEMM_TRANSPOSE, 2)
    cases = [mk(W.PEAK_F32_F32, 0, 1, 520, 392, 264, alpha=0.5, beta=2.0, case=1),      # both operands transposed first
             mk(W.PEAK_F32_F32, 1, 0, 333, 260, 100, alpha=1.0, beta=0.0, pad_a=3, case=2)]
    dcs = [R.DeviceCase(c) for c in cases]
    for dc in dcs:
        dc.run(stream=None)                                    # first-use set-up outside the capture
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            for dc in dcs:
                c = dc.case
                P.peak_gemm(c.dtype, c.transA, c.transB, c.M, c.N, c.K, c.alpha, dc.A, c.lda, dc.B, c.ldb, c.beta,
                            dc.C, c.ldc, stream)
    for rep in range(2):
        for dc in dcs:
            dc.Cfull.copy_(R.to_device(dc.Cfull_h, dc.case.out_type))
        graph.replay()
        torch.cuda.synchronize()
        assert P.peak_check()[0] == P.PEAK_OK
        for dc in dcs:
            R.check_full(dc, what=f"sgemm graph replay {rep} {dc.case.name}")
    errors = []

    def worker(idx):
        try:
            st = torch.cuda.Stream()
            dc = dcs[idx]
            c = dc.case
            for rep in range(10):
                dc.reset_c()
                st.wait_stream(torch.cuda.current_stream())
                P.peak_gemm(c.dtype, c.transA, c.transB, c.M, c.N, c.K, c.alpha, dc.A, c.lda, dc.B, c.ldb, c.beta, dc.C,
                            c.ldc, st)
                rc, detail = P.peak_check(st)
                assert rc == P.PEAK_OK, hex(detail)
            R.check_full(dc, what=f"sgemm thread {idx}")
        except Exception as exc:
            errors.append(exc)

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors[0]
