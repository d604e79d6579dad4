"""Helpers for the GPU parity tests: run one GEMM case through the C ABI and compare it with the oracle.

The tolerances are written out here:
  * 16-bit inputs (the stated bound): |C - ref| <= 1e-2 * S' + 1e-3 per element, where
    S' = |alpha| * sum_k |a_ik b_kj| + |beta| * |C0_ij|  (S' = S when alpha = 1, beta = 0);
  * fp32 inputs (the stated bound): ||C - ref||_F / ||ref||_F <= 1e-5;
  * a tighter self-check on every element, derived from the arithmetic: products of two 16-bit values are
    exact in fp32, so only the <= K fp32 accumulation roundings and the single output rounding contribute:
        |C - ref| <= 2 * u_out * |ref| + 4 * K * 2^-24 * S' + sub_out,
    u_out = 2^-8 (bf16), 2^-11 (fp16), 2^-24 (fp32); sub_out = half the spacing of the output format's
    subnormals (2^-25 for fp16), the rounding error of results too small for the relative bound;
  * 8-bit inputs: products of two 8-bit floats are exact in fp32 as well, so the same two bounds apply;
  * exact cases (small integers): the output bits equal the oracle's correctly rounded result.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2512_19018_b200 import binding as P
from paper_2512_19018_b200 import workloads as W

OT = {"f16": oracle.F16, "bf16": oracle.BF16, "f32": oracle.F32, "e4m3": oracle.E4M3, "e5m2": oracle.E5M2}
U_OUT = {"bf16": 2.0 ** -8, "f16": 2.0 ** -11, "f32": 2.0 ** -24}
# half the spacing of the output format's subnormals: the absolute rounding error where the relative bound
# u_out * |x| no longer holds (fp16 results below 2^-14 are common with cancelling sums and small K)
SUB_OUT = {"bf16": 2.0 ** -134, "f16": 2.0 ** -25, "f32": 2.0 ** -150}
TORCH_STORE = {"f16": torch.float16, "bf16": torch.bfloat16, "f32": torch.float32}
GUARD_ROWS = 3


def to_device(arr: np.ndarray, t: str) -> torch.Tensor:
    """Upload stored bits unchanged."""
    if t in ("f32", "e4m3", "e5m2"):     # float32 values / raw bytes
        return torch.from_numpy(arr).cuda()
    return torch.from_numpy(arr.view(np.int16)).cuda().view(TORCH_STORE[t])


def to_host(ten: torch.Tensor, t: str) -> np.ndarray:
    if t == "f32":
        return ten.cpu().numpy()
    return ten.view(torch.int16).cpu().numpy().view(np.uint16)


def guard_pattern(t: str):
    return np.float32(-77.25) if t == "f32" else np.uint16(0xC29A if t == "bf16" else 0xD4D4)


class DeviceCase:
    """Inputs of one case resident on the GPU, with guard rows above and below C."""

    def __init__(self, case: W.GemmCase, c_init: str = "auto"):
        self.case = case
        A, B, C0 = W.make_inputs(case)
        self.A_h, self.B_h = A, B
        if C0 is None:
            C0 = W.poison_c(case) if c_init in ("auto", "poison") else np.zeros((case.M, case.ldc), W.NP_STORE[case.out_type])
        self.C0_h = C0
        t = case.out_type
        full = np.empty((case.M + 2 * GUARD_ROWS, case.ldc), dtype=C0.dtype)
        full[:] = guard_pattern(t)
        full[GUARD_ROWS:GUARD_ROWS + case.M, :] = C0
        if case.ldc > case.N:
            full[GUARD_ROWS:GUARD_ROWS + case.M, case.N:] = guard_pattern(t)
        self.Cfull_h = full
        self.A = to_device(A, case.in_type)
        self.B = to_device(B, case.in_type)
        self.reset_c()

    def reset_c(self):
        self.Cfull = to_device(self.Cfull_h, self.case.out_type)
        self.C = self.Cfull[GUARD_ROWS:GUARD_ROWS + self.case.M]

    def run(self, variant=P.PEAK_VARIANT_AUTO, alpha=None, beta=None, stream=None):
        c = self.case
        alpha = c.alpha if alpha is None else alpha
        beta = c.beta if beta is None else beta
        P.peak_gemm_variant(variant, c.dtype, c.transA, c.transB, c.M, c.N, c.K, alpha, self.A, c.lda, self.B, c.ldb,
                            beta, self.C, c.ldc, stream)
        rc, detail = P.peak_check(stream)
        assert rc == P.PEAK_OK, f"peak_check: {P.peak_status_string(rc)} detail=0x{detail:08x}"

    def result(self) -> np.ndarray:
        """Stored bits of C (M x N) after checking that guards and pitch padding are untouched."""
        c = self.case
        full = to_host(self.Cfull, c.out_type)
        g = guard_pattern(c.out_type)
        assert (full[:GUARD_ROWS] == g).all() and (full[GUARD_ROWS + c.M:] == g).all(), "guard rows overwritten"
        if c.ldc > c.N:
            assert (full[GUARD_ROWS:GUARD_ROWS + c.M, c.N:] == g).all(), "pitch padding overwritten"
        return full[GUARD_ROWS:GUARD_ROWS + c.M, :c.N]

    # ---- oracle sides -------------------------------------------------------------------------
    def oracle_full(self, alpha=None, beta=None):
        c = self.case
        alpha = c.alpha if alpha is None else alpha
        beta = c.beta if beta is None else beta
        return oracle.gemm(OT[c.in_type], OT[c.out_type], c.transA, c.transB, c.M, c.N, c.K, alpha, self.A_h, c.lda,
                           self.B_h, c.ldb, beta, self.C0_h if beta != 0 else None, c.ldc)

    def oracle_sub(self, rows, cols, alpha=None, beta=None):
        c = self.case
        alpha = c.alpha if alpha is None else alpha
        beta = c.beta if beta is None else beta
        return oracle.gemm_submatrix(OT[c.in_type], OT[c.out_type], c.transA, c.transB, c.M, c.N, c.K, alpha,
                                     self.A_h, c.lda, self.B_h, c.ldb, beta, self.C0_h if beta != 0 else None, c.ldc,
                                     rows, cols)

    def oracle_points(self, si, sj, alpha=None, beta=None):
        c = self.case
        alpha = c.alpha if alpha is None else alpha
        beta = c.beta if beta is None else beta
        return oracle.gemm_points(OT[c.in_type], OT[c.out_type], c.transA, c.transB, c.M, c.N, c.K, alpha, self.A_h,
                                  c.lda, self.B_h, c.ldb, beta, self.C0_h if beta != 0 else None, c.ldc, si, sj)


def s_prime(case, S, alpha, beta, c0_vals):
    sp = abs(alpha) * S
    if beta != 0:
        sp = sp + abs(beta) * np.abs(c0_vals)
    return sp


def check_values(case: W.GemmCase, got_bits: np.ndarray, ref: np.ndarray, S: np.ndarray, c0_vals, alpha=None,
                 beta=None, what=""):
    """Apply the stated bound and the tighter self-check to every compared element."""
    alpha = case.alpha if alpha is None else alpha
    beta = case.beta if beta is None else beta
    got = W.to_float64(got_bits, case.out_type)
    assert not np.isnan(got).any(), f"{what}: NaN in the result"
    sp = s_prime(case, S, alpha, beta, c0_vals)
    err = np.abs(got - ref)
    tight = 2 * U_OUT[case.out_type] * np.abs(ref) + 4 * max(case.K, 1) * 2.0 ** -24 * sp + SUB_OUT[case.out_type]
    if case.in_type == "f32":
        num, den = np.sqrt((err ** 2).sum()), np.sqrt((ref ** 2).sum())
        assert num <= 1e-5 * den + 1e-30, f"{what}: relative Frobenius error {num / max(den, 1e-300):.3e} > 1e-5"
    else:
        stated = 1e-2 * sp + 1e-3
        bad = err > stated
        assert not bad.any(), f"{what}: {bad.sum()} elements beyond 1e-2*S+1e-3, worst {err.max():.3e}"
    bad = err > tight
    if bad.any():
        k = np.unravel_index(np.argmax(err - tight), err.shape)
        raise AssertionError(f"{what}: {bad.sum()} of {err.size} elements beyond the derived bound; worst at {k}: "
                             f"got {got[k]!r} ref {ref[k]!r} err {err[k]:.3e} tol {tight[k]:.3e}")
    return float((err / np.maximum(tight, 1e-300)).max())


def c0_values(dc: DeviceCase, rows=None, cols=None):
    c = dc.case
    v = W.to_float64(dc.C0_h[:, :c.N], c.out_type)
    if rows is not None:
        v = v[np.ix_(rows, cols)]
    return v


def check_full(dc: DeviceCase, alpha=None, beta=None, what=""):
    c = dc.case
    beta_ = c.beta if beta is None else beta
    ref, S = dc.oracle_full(alpha, beta)
    c0 = c0_values(dc) if beta_ != 0 else 0.0
    return check_values(c, dc.result(), ref, S, c0, alpha, beta, what or c.name)


def sample_grid(case: W.GemmCase, tile_m: int, tile_n: int, budget_macs: float = 1.2e9, seed: int = 0):
    """Rows and columns such that every tile_m x tile_n output tile holds several sampled elements:
    first / last row and column of every tile (clipped), plus random ones; sized to a MAC budget."""
    rng = np.random.default_rng(case.seed + seed)
    rows = set([0, case.M - 1])
    cols = set([0, case.N - 1])
    for t0 in range(0, case.M, tile_m):
        rows.update([t0, min(t0 + tile_m, case.M) - 1])
    for t0 in range(0, case.N, tile_n):
        cols.update([t0, min(t0 + tile_n, case.N) - 1])
    side = int(max(8, np.sqrt(budget_macs / max(case.K, 1))))
    def fill(s, n, want):
        want = min(want, n)
        while len(s) < want:
            s.update(rng.integers(0, n, size=want - len(s)).tolist())
        out = np.array(sorted(s), dtype=np.int64)
        if len(out) > want:   # too many tile edges: keep a random subset, but always the extremes
            keep = set([0, n - 1]) | set(rng.choice(out, size=want - 2, replace=False).tolist())
            out = np.array(sorted(keep), dtype=np.int64)
        return out
    return fill(rows, case.M, side), fill(cols, case.N, side)


def check_sampled(dc: DeviceCase, tile_m=128, tile_n=256, what="", budget_macs=1.2e9):
    c = dc.case
    rows, cols = sample_grid(c, tile_m, tile_n, budget_macs)
    ref, S = dc.oracle_sub(rows, cols)
    got = dc.result()[np.ix_(rows, cols)]
    c0 = c0_values(dc, rows, cols) if c.beta != 0 else 0.0
    worst = check_values(c, got, ref, S, c0, what=what or c.name)
    # scattered single elements off the grid (the listed-points entry point: one k-loop per element)
    rng = np.random.default_rng(c.seed + 4242)
    n_pts = int(min(512, max(16, 2e8 // max(c.K, 1))))
    si, sj = rng.integers(0, c.M, n_pts), rng.integers(0, c.N, n_pts)
    ref_p, S_p = dc.oracle_points(si, sj)
    c0_p = c0_values(dc)[si, sj] if c.beta != 0 else 0.0
    return max(worst, check_values(c, dc.result()[si, sj], ref_p, S_p, c0_p, what=(what or c.name) + " (points)"))
