"""peak_gemm_strided_batched against the oracle applied matrix by matrix (the definition of a batched GEMM):
one-launch tensor-core path (tiles numbered across the batch, 3-D tensor maps), its split-K form, and the
launch-per-matrix path of the other kernel families, with gaps between the matrices, alpha/beta, exact
integer cases and the argument checks."""
import numpy as np
import pytest
import torch

import oracle
from paper_2512_19018_b200 import binding as P
from paper_2512_19018_b200 import workloads as W
from tests import parity as R

pytestmark = pytest.mark.gpu


@pytest.fixture
def reset_tuning():
    yield
    for key in range(P.PEAK_TUNE_COUNT):
        P.peak_set_tuning(key, 0)


class Batch:
    """`batch` seeded problems of one shape laid out with strides (and `gap` spare elements between matrices)."""

    def __init__(self, case, batch, gap=0, share_b=False):
        self.case, self.batch, self.share_b = case, batch, share_b
        self.cases = [case.with_(case=case.case + 101 * b) for b in range(batch)]
        ins = [W.make_inputs(c, need_c0=True) for c in self.cases]
        if share_b:
            ins = [(a, ins[0][1], c0) for a, _, c0 in ins]
        self.ins = ins
        self.sA = ins[0][0].size + gap
        self.sB = 0 if share_b else ins[0][1].size + gap
        self.sC = ins[0][2].size + gap
        def stack(k, stride, t, n):
            flat = np.full(max(stride, ins[0][k].size) * n, 0, dtype=ins[0][k].dtype)
            for b in range(n):
                flat[b * stride:b * stride + ins[b][k].size] = ins[b][k].ravel()
            return R.to_device(flat, t)
        self.A = stack(0, self.sA, case.in_type, batch)
        self.B = stack(1, self.sB, case.in_type, 1 if share_b else batch)
        self.C = stack(2, self.sC, case.out_type, batch)

    def run(self):
        c = self.case
        P.peak_gemm_strided_batched(c.dtype, c.transA, c.transB, c.M, c.N, c.K, c.alpha, self.A, c.lda, self.sA, self.B,
                                    c.ldb, self.sB, c.beta, self.C, c.ldc, self.sC, self.batch)
        rc, detail = P.peak_check()
        assert rc == P.PEAK_OK, hex(detail)

    def results(self):
        c = self.case
        flat = R.to_host(self.C, c.out_type)
        return [flat[b * self.sC:b * self.sC + c.M * c.ldc].reshape(c.M, c.ldc)[:, :c.N] for b in range(self.batch)]

    def check(self, exact=False, what=""):
        c = self.case
        for b, got in enumerate(self.results()):
            A, B, C0 = self.ins[b]
            ref, S = oracle.gemm(R.OT[c.in_type], R.OT[c.out_type], c.transA, c.transB, c.M, c.N, c.K, c.alpha, A, c.lda,
                                 B, c.ldb, c.beta, C0 if c.beta != 0 else None, c.ldc)
            if exact:
                want = oracle.round_to(R.OT[c.out_type], ref)
                g = got.view(np.uint32) if c.out_type == "f32" else got
                assert np.array_equal(g, want), f"{what} matrix {b}"
            else:
                c0 = W.to_float64(C0[:, :c.N], c.out_type) if c.beta != 0 else 0.0
                R.check_values(c, got, ref, S, c0, what=f"{what} matrix {b}")


def mk(dtype, ta, tb, M, N, K, **kw):
    pa, pb = (-(M if ta else K)) % 8, (-(K if tb else N)) % 8
    return W.GemmCase(f"b{dtype}_{ta}{tb}_{M}x{N}x{K}", dtype, bool(ta), bool(tb), M, N, K, pad_a=pa, pad_b=pb, **kw)


@pytest.mark.parametrize("dtype", [W.PEAK_BF16_BF16, W.PEAK_F16_F32])
@pytest.mark.parametrize("ta,tb", [(0, 0), (0, 1), (1, 0), (1, 1)])
def test_batched_tensor_core_one_launch(dtype, ta, tb):
    n0 = P.peak_kernel_launches()
    b = Batch(mk(dtype, ta, tb, 264, 328, 200, alpha=0.5, beta=2.0), batch=5, gap=8)
    b.run()
    assert P.peak_kernel_launches() - n0 == 1                  # the whole batch is one persistent-kernel launch
    b.check(what="batched real")
    bi = Batch(mk(dtype, ta, tb, 264, 328, 200, alpha=0.25, beta=-1.0, dist="smallint"), batch=5, gap=8)
    bi.run()
    bi.check(exact=True, what="batched integers")


def test_batched_many_small_and_split(reset_tuning):
    """Attention-like: many small problems (each a single tile) and a forced k-split across the batch."""
    b = Batch(mk(W.PEAK_BF16_BF16, 0, 1, 128, 128, 64, dist="smallint"), batch=48)
    b.run()
    b.check(exact=True, what="48 x (128,128,64)")
    P.peak_set_tuning(P.PEAK_TUNE_SPLIT_K, 3)
    b = Batch(mk(W.PEAK_BF16_F32, 1, 0, 96, 264, 704, alpha=1.0, beta=1.0, dist="smallint"), batch=3, gap=16)
    b.run()
    b.check(exact=True, what="batch with k-split")


def test_batched_short_k_tiles(reset_tuning):
    """Batches of more than a wave of tiles with at most four k-blocks (eight with beta != 0) take single-CTA
    128 x 256 tiles (the plain-store loop with beta = 0, the general one otherwise): exact on integers, ragged edges
    included."""
    for ta, tb, M, N, K, beta in [(0, 1, 1024, 1024, 128, 0.0), (0, 0, 1000, 1016, 200, 0.0), (1, 0, 1024, 1024, 64, 1.0),
                                  (0, 1, 256, 256, 128, 0.0), (1, 1, 520, 776, 448, -1.0)]:
        b = Batch(mk(W.PEAK_BF16_BF16, ta, tb, M, N, K, alpha=0.5, beta=beta, dist="smallint"), batch=5 if M > 520 else 96,
                  gap=8)
        b.run()
        # single-CTA 256-wide tiles of a batch, eight epilogue warps (the last template flag but one)
        assert "umma_gemm_kernel<1, 256," in P.peak_last_kernel() and ", 1, 0, 1, 0>" in P.peak_last_kernel(), P.peak_last_kernel()
        b.check(exact=True, what=f"short-k batch {M}x{N}x{K} beta={beta}")


def test_batched_other_kernel_families():
    # fp32 -> SGEMM, one launch per matrix
    b = Batch(W.GemmCase("bs", W.PEAK_F32_F32, False, False, 256, 128, 64, 0.5, 2.0, "uniform"), batch=3, gap=4)
    n0 = P.peak_kernel_launches()
    b.run()
    assert P.peak_kernel_launches() - n0 == 3
    b.check(what="sgemm batch")
    # pitches TMA cannot use -> fallback kernel per matrix
    b = Batch(W.GemmCase("bf", W.PEAK_BF16_BF16, False, False, 37, 53, 41, 1.0, 1.0, "uniform", pad_a=1), batch=4, gap=3)
    b.run()
    b.check(what="fallback batch")
    # one B for every matrix of the batch (strideB == 0)
    b = Batch(mk(W.PEAK_BF16_BF16, 0, 1, 256, 256, 128, dist="smallint"), batch=3, share_b=True)
    b.run()
    b.check(exact=True, what="shared B")


def test_batched_argument_checks():
    t = torch.zeros(1 << 16, dtype=torch.bfloat16, device="cuda")
    call = lambda **k: P.peak_gemm_strided_batched(W.PEAK_BF16_BF16, 0, 0, 64, 64, 64, 1.0, t, 64, k.get("sA", 4096), t, 64,
                                                   k.get("sB", 4096), 0.0, t, 64, k.get("sC", 4096), k.get("batch", 2),
                                                   check=False)
    assert call(batch=0) == P.PEAK_OK
    assert call(batch=-1) == P.PEAK_ERR_INVALID_VALUE
    assert call(sC=100) == P.PEAK_ERR_INVALID_VALUE            # C matrices would overlap
    assert call(sA=-8) == P.PEAK_ERR_INVALID_VALUE
    assert call(batch=1, sC=0) == P.PEAK_OK                    # a batch of one ignores the strides
    torch.cuda.synchronize()
