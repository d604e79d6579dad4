"""Host-side checks that need no GPU: the library loads and exports what the header declares, arguments
are validated before any device call, the dispatcher's choices, the tile order, the input generators."""
import os
import re

import numpy as np
import pytest

from paper_2512_19018_b200 import binding as P
from paper_2512_19018_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2512_19018_b200 import build
    build.build()
    return P.load()


def test_exports_match_header(lib):
    text = open(os.path.join(ROOT, "include", "peak_gemm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = sorted(set(re.findall(r"\b(peak_[a-z0-9_]+)\s*\(", text)))
    assert declared == sorted(P.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in the header but not exported"
    assert P.peak_version() >= 100
    assert P.peak_status_string(P.PEAK_OK) == "ok"
    assert P.peak_variant_string(P.PEAK_VARIANT_UMMA_2CTA) == "umma_2cta"


def test_invalid_arguments_rejected_without_a_device(lib):
    A = B = C = 0x1000  # never dereferenced: validation comes first
    ok = dict(dtype=P.PEAK_BF16_BF16, transA=0, transB=0, M=64, N=64, K=64, alpha=1.0, A=A, lda=64, B=B, ldb=64,
              beta=0.0, C=C, ldc=64)
    def call(**kw):
        a = dict(ok, **kw)
        return P.peak_gemm(a["dtype"], a["transA"], a["transB"], a["M"], a["N"], a["K"], a["alpha"], a["A"], a["lda"],
                           a["B"], a["ldb"], a["beta"], a["C"], a["ldc"], None, check=False)
    assert call(dtype=9) == P.PEAK_ERR_INVALID_VALUE
    assert call(dtype=-1) == P.PEAK_ERR_INVALID_VALUE
    assert call(transA=2) == P.PEAK_ERR_INVALID_VALUE
    assert call(transB=-1) == P.PEAK_ERR_INVALID_VALUE
    assert call(M=-1) == P.PEAK_ERR_INVALID_VALUE
    assert call(lda=63) == P.PEAK_ERR_INVALID_VALUE
    assert call(ldb=63) == P.PEAK_ERR_INVALID_VALUE
    assert call(ldc=63) == P.PEAK_ERR_INVALID_VALUE
    assert call(transA=1, M=128, lda=64) == P.PEAK_ERR_INVALID_VALUE        # A stored K x M needs lda >= M
    assert call(transB=1, K=128, lda=128, ldb=64) == P.PEAK_ERR_INVALID_VALUE  # B stored N x K needs ldb >= K
    assert call(A=None) == P.PEAK_ERR_INVALID_VALUE
    assert call(C=None) == P.PEAK_ERR_INVALID_VALUE
    # nothing to do: returns OK without touching a device
    assert call(M=0) == P.PEAK_OK
    assert call(N=0) == P.PEAK_OK
    assert call(alpha=0.0, beta=1.0) == P.PEAK_OK
    assert call(K=0, beta=1.0, A=None, B=None) == P.PEAK_OK
    rc = P.peak_gemm_variant(99, P.PEAK_BF16_BF16, 0, 0, 64, 64, 64, 1.0, A, 64, B, 64, 0.0, C, 64, None, check=False)
    assert rc == P.PEAK_ERR_INVALID_VALUE


def test_no_silent_fallback_without_gpu(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    rc = P.peak_gemm(P.PEAK_BF16_BF16, 0, 0, 64, 64, 64, 1.0, 0x1000, 64, 0x1000, 64, 0.0, 0x1000, 64, None,
                     check=False)
    assert rc in (P.PEAK_ERR_CUDA, P.PEAK_ERR_ARCH)     # fails loudly: there is no CPU path
    with pytest.raises(P.PeakError):
        P.peak_gemm(P.PEAK_BF16_BF16, 0, 0, 64, 64, 64, 1.0, 0x1000, 64, 0x1000, 64, 0.0, 0x1000, 64, None)


def test_dispatch_choices(lib):
    q = P.peak_query_variant
    al = 0x10000  # a 16-byte aligned fake pointer
    assert q(P.PEAK_BF16_BF16, 0, 0, 4096, 4096, 4096, 1.0, al, 4096, al, 4096, 0.0, al, 4096) in (
        P.PEAK_VARIANT_UMMA_1CTA, P.PEAK_VARIANT_UMMA_2CTA)
    assert q(P.PEAK_F16_F32, 1, 0, 5000, 3000, 2500, 0.5, al, 5000, al, 3000, 2.0, al, 3000) in (
        P.PEAK_VARIANT_UMMA_1CTA, P.PEAK_VARIANT_UMMA_2CTA)
    # a pitch that is not a multiple of 16 bytes, or a misaligned base, cannot use TMA
    assert q(P.PEAK_BF16_BF16, 0, 0, 100, 100, 100, 1.0, al, 100, al, 100, 0.0, al, 100) == P.PEAK_VARIANT_FALLBACK
    assert q(P.PEAK_BF16_BF16, 0, 0, 128, 128, 128, 1.0, al + 2, 128, al, 128, 0.0, al, 128) == P.PEAK_VARIANT_FALLBACK
    assert q(P.PEAK_F32_F32, 0, 0, 4096, 4096, 4096, 1.0, al, 4096, al, 4096, 0.0, al, 4096) == P.PEAK_VARIANT_SGEMM
    assert q(P.PEAK_F32_F32, 0, 0, 100, 4096, 4096, 1.0, al, 4096, al, 4096, 0.0, al, 4096) == P.PEAK_VARIANT_SGEMM
    assert q(P.PEAK_F32_F32, 0, 0, 100, 4096, 4096, 1.0, al, 4098, al, 4096, 0.0, al, 4096) == P.PEAK_VARIANT_FALLBACK
    assert q(P.PEAK_F32_F32, 0, 0, 0, 4096, 4096, 1.0, al, 4096, al, 4096, 0.0, al, 4096) == P.PEAK_VARIANT_NONE
    assert q(P.PEAK_F32_F32, 0, 0, 64, 64, 0, 1.0, None, 1, None, 64, 0.5, al, 64) == P.PEAK_VARIANT_SCALE
    assert q(P.PEAK_F32_F32, 0, 0, 64, 64, 64, 0.0, al, 64, al, 64, 1.0, al, 64) == P.PEAK_VARIANT_NONE
    assert q(P.PEAK_F32_F32, 0, 0, 64, 64, 64, 0.0, al, 64, al, 64, 0.0, al, 64) == P.PEAK_VARIANT_SCALE
    assert q(9, 0, 0, 64, 64, 64, 1.0, al, 64, al, 64, 0.0, al, 64) == -P.PEAK_ERR_INVALID_VALUE
    # 8-bit float inputs: tensor cores for every layout, given 16-byte pitches
    for dt in (P.PEAK_E4M3_BF16, P.PEAK_E4M3_F32, P.PEAK_E5M2_BF16, P.PEAK_E5M2_F32):
        for ta, tb in [(0, 1), (0, 0), (1, 0), (1, 1)]:
            assert q(dt, ta, tb, 4096, 4096, 4096, 1.0, al, 4096, al, 4096, 0.0, al, 4096) == P.PEAK_VARIANT_UMMA_2CTA
        assert q(dt, 1, 0, 4096, 4096, 4096, 1.0, al, 4100, al, 4096, 0.0, al, 4096) == P.PEAK_VARIANT_FALLBACK
        assert q(dt, 0, 1, 4096, 4096, 1000, 1.0, al, 1000, al, 1000, 0.0, al, 4096) == P.PEAK_VARIANT_FALLBACK
        assert q(dt, 0, 1, 4096, 4096, 1000, 1.0, al, 1008, al, 1008, 0.0, al, 4096) == P.PEAK_VARIANT_UMMA_2CTA
    # few tiles: single-CTA tiles spread the problem over more SMs than 256-row pair tiles would
    assert q(P.PEAK_BF16_BF16, 0, 0, 1024, 1024, 1024, 1.0, al, 1024, al, 1024, 0.0, al, 1024) == P.PEAK_VARIANT_UMMA_1CTA
    assert q(P.PEAK_BF16_BF16, 0, 0, 1536, 1536, 1536, 1.0, al, 1536, al, 1536, 0.0, al, 1536) == P.PEAK_VARIANT_UMMA_1CTA
    assert q(P.PEAK_BF16_BF16, 0, 0, 2048, 2048, 2048, 1.0, al, 2048, al, 2048, 0.0, al, 2048) == P.PEAK_VARIANT_UMMA_2CTA
    assert q(P.PEAK_BF16_BF16, 0, 0, 128, 4096, 4096, 1.0, al, 4096, al, 4096, 0.0, al, 4096) == P.PEAK_VARIANT_UMMA_1CTA


@pytest.mark.parametrize("tiles_m,tiles_n,group", [(1, 1, 8), (64, 32, 16), (32, 32, 8), (20, 12, 16), (7, 5, 3),
                                                   (1, 16, 8), (40, 1, 16), (13, 9, 1), (5, 7, 100)])
def test_tile_order_is_a_bijection_and_grouped(lib, tiles_m, tiles_n, group):
    seen = set()
    prev_group = 0
    for t in range(tiles_m * tiles_n):
        tm, tn = P.peak_tile_coord(t, tiles_m, tiles_n, group)
        assert 0 <= tm < tiles_m and 0 <= tn < tiles_n
        seen.add((tm, tn))
        g = tm // group
        assert g >= prev_group          # groups of tile-rows are finished one after the other
        prev_group = g
    assert len(seen) == tiles_m * tiles_n
    # consecutive tiles inside a group walk down the rows first (they share the B panel)
    if tiles_m >= 2 and group >= 2:
        a, b = P.peak_tile_coord(0, tiles_m, tiles_n, group), P.peak_tile_coord(1, tiles_m, tiles_n, group)
        assert b == (a[0] + 1, a[1])
    with pytest.raises(P.PeakError):
        P.peak_tile_coord(tiles_m * tiles_n, tiles_m, tiles_n, group)


def test_workload_generators_are_seeded_and_shaped():
    c = W.config0()
    A1, B1, C1 = W.make_inputs(c)
    A2, B2, _ = W.make_inputs(c)
    assert C1 is None and np.array_equal(A1, A2) and np.array_equal(B1, B2)
    assert A1.shape == (512, 512) and A1.dtype == np.uint16
    a = W.to_float64(A1, "f16")
    assert a.min() >= -1.0 and a.max() <= 1.0 and abs(a.mean()) < 0.01
    r = W.config4_ragged(0)
    assert (r.layout, r.lda, r.ldb, r.ldc) == ("TN", 5000, 3000, 3000)
    assert r.a_shape == (2500, 5000) and r.b_shape == (2500, 3000)
    t = W.config3(1)
    assert t.layout == "NT" and t.b_shape == (14336, 4096) and t.beta == 1.0
    small = t.with_(M=64, N=48, K=32)
    A, B, C0 = W.make_inputs(small)
    assert B.shape == (48, 32) and C0.shape == (64, 48)
    assert abs(W.to_float64(B, "bf16").std() - 0.02) < 0.003
    p = W.GemmCase("pad", W.PEAK_F32_F32, False, False, 5, 6, 7, pad_a=2, pad_c=1, beta=1.0)
    A, B, C0 = W.make_inputs(p)
    assert A.shape == (5, 9) and np.isnan(A[:, 7:]).all() and C0.shape == (5, 7)
    assert W.config1().min_bytes() == 3 * 4096 * 4096 * 2


def test_tuner_enumerates_and_prunes():
    from paper_2512_19018_b200 import tune
    cands = [(v, k) for v, k in tune.candidates(tune.SPACE_16BIT) if tune.prune(v, k, 4096, 4096, 4096)]
    assert len(cands) > 20 and len(set((v, tuple(sorted(k.items()))) for v, k in cands)) == len(cands)
    for v, k in cands:
        assert not (v == "umma_1cta" and k.get(1) == 512)             # wide tiles need CTA pairs
        assert not (k.get(10) == 2 and k.get(1) == 128)                # the plug-in runs 256- and 512-wide tiles
        assert not (k.get(2, 1) > 1 and k.get(1) == 512)
    assert any(k.get(10) == 2 and k.get(1) == 512 for v, k in cands)  # ... so the 512-wide plug-in kernel is timed
    # a k-split cannot have more slices than k-blocks
    assert not tune.prune("umma_2cta", {1: 256, 2: 8, 3: 2, 10: 1, 0: 0}, 256, 256, 128)
    assert len(list(tune.candidates(tune.SPACE_F32, quick=True))) == 8


def test_per_device_once_bookkeeping():
    """Context set-up (a kernel's shared-memory attribute, occupancy queries) is remembered per device, so a
    second GPU used by the same process is set up as well; the library checks its own bookkeeping on the host."""
    assert P.peak_selftest_per_device_once() == 0


def test_last_kernel_is_text_and_needs_a_buffer():
    assert isinstance(P.peak_last_kernel(), str)
    assert P.load().peak_last_kernel(None, 16) == P.PEAK_ERR_INVALID_VALUE


def test_bench_traffic_is_read_from_the_profile_of_the_launched_kernel():
    """bench.py quotes DRAM traffic from the ncu summary under profiles/ only when that summary covers the kernel
    that was launched; a different kernel (or an unprofiled workload) gives null and a reason."""
    import bench
    t, src = bench.profile_traffic("bf16_8192_nn", "umma_gemm_kernel<2, 512, __nv_bfloat16, 0, 0, 0, 0> grid=148 items=512 splits=1")
    assert t is not None and 0.3e9 < t < 3e9 and "profiles/" in src
    t, src = bench.profile_traffic("bf16_8192_nn", "umma_gemm_kernel<2, 512, __nv_bfloat16, 0, 0, 0, 0, 0> grid=148")
    assert t is not None                                   # a trailing flag added later, left at 0: same kernel
    t, src = bench.profile_traffic("bf16_8192_nn", "umma_gemm_kernel<2, 512, __nv_bfloat16, 0, 0, 0, 0, 1> grid=148")
    assert t is None
    t, src = bench.profile_traffic("bf16_8192_nn", "umma_gemm_kernel<2, 256, __nv_bfloat16, 0, 0, 0, 0> grid=148")
    assert t is None and "differs" in src
    t, src = bench.profile_traffic("no_such_workload", "x_kernel<1>")
    assert t is None and "no ncu summary" in src
    # the two skinny benchmark shapes: the summary of the one-tile-per-CTA kernel, not the older one beside it
    t, src = bench.profile_traffic("bf16_128x14336x4096_tn", "umma_clusterk_kernel<128, __nv_bfloat16, 1, 0> grid=112 clusters=112")
    assert t is not None and 1.2e8 < t < 1.4e8 and "umma_clusterk" in src
    t, src = bench.profile_traffic("bf16_16x4096x4096_tn", "umma_clusterk_kernel<128, __nv_bfloat16, 4, 0> grid=128 clusters=32")
    assert t is not None and 3.3e7 < t < 3.6e7
    t, src = bench.profile_traffic("bf16_128x14336x4096_tn", "umma_clusterk_kernel<128, __nv_bfloat16, 1, 0, 2> grid=112")
    assert t is None                                        # the pair form is another kernel


def test_bench_rotation_rule():
    import bench
    table = bench.workloads_table()
    assert bench.rotation_sets(table["bf16_8192_nn"]) == 1 and "larger than L2" in bench.l2_note(table["bf16_8192_nn"])
    n = bench.rotation_sets(table["bf16_4096_nn"])
    assert n >= 4 and n * bench.set_bytes(table["bf16_4096_nn"]) > 3 * bench.L2_BYTES


def test_tuning_table_is_loaded_matched_and_overridable(tmp_path):
    """The persisted tuning table: a (fake) table changes the dispatcher's visible choice exactly for the
    problems its entry covers; knobs it may not set are dropped; emptying it restores the built-in rules;
    a file that cannot be read or understood leaves the current table alone."""
    import json
    al = 1 << 20
    q = lambda M, N, K, beta=0.0, dt=P.PEAK_BF16_BF16: P.peak_query_variant(dt, 0, 0, M, N, K, 1.0, al, K, al, N, beta, al, N)
    default_file = os.path.join(os.path.dirname(P.LIB_PATH), "tuned_sm100.json")
    try:
        assert P.peak_tuned_table_load(None) == 0 and P.peak_tuned_table_entries() == 0
        assert q(4096, 4096, 4096) == P.PEAK_VARIANT_UMMA_2CTA
        fake = {"format": 1, "note": "test", "entries": [
            {"in": "bf16", "out": "bf16", "layout": "NN", "beta": 0, "M": 4096, "N": 4096, "K": 4096,
             "variant": "umma_1cta", "knobs": {"1": 128, "0": 4, "8": 5, "9": 1}, "tflops": 1.0},
            {"in": "bf16", "out": "bf16", "layout": "NX?", "M": 1, "N": 1, "K": 1},          # malformed: skipped
            {"in": "f32", "out": "f32", "layout": "NN", "beta": 1, "M": 512, "N": 512, "K": 512, "knobs": {"7": 2}}]}
        path = tmp_path / "table.json"
        path.write_text(json.dumps(fake))
        assert P.peak_tuned_table_load(str(path)) == 2 and P.peak_tuned_table_entries() == 2
        assert q(4096, 4096, 4096) == P.PEAK_VARIANT_UMMA_1CTA           # the entry's family
        assert q(5000, 3000, 4096) == P.PEAK_VARIANT_UMMA_1CTA           # within sqrt(2) of the entry in every dimension
        assert q(8192, 8192, 8192) == P.PEAK_VARIANT_UMMA_2CTA           # outside: built-in rule
        assert q(4096, 4096, 4096, beta=1.0) == P.PEAK_VARIANT_UMMA_2CTA  # other beta class
        assert q(4096, 4096, 4096, dt=P.PEAK_BF16_F32) == P.PEAK_VARIANT_UMMA_2CTA
        v, knobs = P.peak_tuned_lookup(P.PEAK_BF16_BF16, 0, 0, 4096, 4096, 4096, 0.0)
        assert v == P.PEAK_VARIANT_UMMA_1CTA and knobs == {P.PEAK_TUNE_TILE_N: 128, P.PEAK_TUNE_RASTER_GROUP: 4}
        assert P.peak_tuned_lookup(P.PEAK_BF16_BF16, 0, 0, 4096, 4096, 16384, 0.0) is None
        v, knobs = P.peak_tuned_lookup(P.PEAK_F32_F32, 0, 0, 600, 400, 512, 2.0)
        assert v == 0 and knobs == {P.PEAK_TUNE_SGEMM_COPY: 2}
        bad = tmp_path / "bad.json"
        bad.write_text("{\"entries\": [1, 2")
        assert P.peak_tuned_table_load(str(bad)) == -1 and P.peak_tuned_table_entries() == 2
        assert P.peak_tuned_table_load(str(tmp_path / "missing.json")) == -2 and P.peak_tuned_table_entries() == 2
        assert P.peak_tuned_table_load("") == 0
        assert q(4096, 4096, 4096) == P.PEAK_VARIANT_UMMA_2CTA
    finally:
        P.peak_tuned_table_load(default_file if os.path.exists(default_file) else None)


def test_shipped_tuning_table_parses():
    """The table that ships with the package (written by the sweep) is understood by the library's reader."""
    import json
    path = os.path.join(os.path.dirname(P.LIB_PATH), "tuned_sm100.json")
    if not os.path.exists(path):
        pytest.skip("no tuned_sm100.json in the package")
    n = len(json.load(open(path))["entries"])
    assert P.peak_tuned_table_load(path) == n
