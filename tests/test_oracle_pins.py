"""Pins for the CPU oracle: it is checked against things other than itself --
IEEE conversions done by numpy, closed forms, exact integer arithmetic,
invariants of the definition, a hand-worked example and numpy's float64 matmul.
None of these tests needs a GPU."""
import os

import numpy as np
import pytest

from paper_2512_19018_b200 import workloads as W

GOLD = os.path.join(os.path.dirname(__file__), "golden")
T = {"f16": 0, "bf16": 1, "f32": 2}


# ---------------------------------------------------------------- decoders
def test_decode_f16_exhaustive(oracle):
    bits = np.arange(65536, dtype=np.uint16)
    got = oracle.decode(oracle.F16, bits)
    want = bits.view(np.float16).astype(np.float64)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], want[~nan])
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(want[~nan]))


def test_decode_bf16_exhaustive(oracle):
    bits = np.arange(65536, dtype=np.uint16)
    got = oracle.decode(oracle.BF16, bits)
    with np.errstate(invalid="ignore"):
        want = (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], want[~nan])
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(want[~nan]))


def test_decode_f32_samples(oracle):
    rng = np.random.default_rng(1)
    bits = rng.integers(0, 2**32, size=40000, dtype=np.uint64).astype(np.uint32)
    special = np.array([0, 1, 0x007FFFFF, 0x00800000, 0x7F7FFFFF, 0x7F800000, 0xFF800000, 0x80000000, 0x7FC00000,
                        0x3F800000, 0xBF800000, 0x00000002, 0x80000001], dtype=np.uint32)
    bits = np.concatenate([bits, special])
    got = oracle.decode(oracle.F32, bits)
    with np.errstate(invalid="ignore"):
        want = bits.view(np.float32).astype(np.float64)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], want[~nan])


# ---------------------------------------------------------------- rounding
def _interesting_doubles(rng):
    x = np.concatenate([
        rng.standard_normal(20000),
        rng.standard_normal(20000) * 1e-6,
        rng.standard_normal(5000) * 1e-8,       # fp16 subnormal range
        rng.standard_normal(5000) * 1e5,        # fp16 overflow range
        rng.standard_normal(2000) * 1e-40,      # fp32 / bf16 subnormal range
        rng.standard_normal(2000) * 1e38 * 4,   # fp32 overflow range
        np.array([0.0, -0.0, np.inf, -np.inf, 65504.0, 65519.99, 65520.0, 2.0**-24, 2.0**-25, 1.5 * 2.0**-25,
                  2.0**-14, 2.0**-14 - 2.0**-25, 1.0 + 2.0**-11, 1.0 + 3 * 2.0**-11, 1.0 + 2.0**-8,
                  1.0 + 3 * 2.0**-8, 1.0 + 2.0**-24, 1.0 + 3 * 2.0**-24]),
    ])
    return x


def test_round_f16_matches_numpy(oracle):
    x = _interesting_doubles(np.random.default_rng(2))
    with np.errstate(over="ignore"):
        want = x.astype(np.float16).view(np.uint16)      # IEEE double -> half, one rounding
    got = oracle.round_to(oracle.F16, x)
    assert np.array_equal(got, want)


def test_round_f32_matches_numpy(oracle):
    x = _interesting_doubles(np.random.default_rng(3))
    with np.errstate(over="ignore"):
        want = x.astype(np.float32).view(np.uint32)
    got = oracle.round_to(oracle.F32, x)
    assert np.array_equal(got, want)


def test_round_bf16_ties_and_roundtrip(oracle):
    # every finite bf16 value survives a round trip
    bits = np.arange(65536, dtype=np.uint16)
    with np.errstate(invalid="ignore"):
        vals = (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    fin = np.isfinite(vals)
    assert np.array_equal(oracle.round_to(oracle.BF16, vals[fin]), bits[fin])
    # the midpoint of two neighbours goes to the one with an even pattern; a hair off goes to the nearer one
    pos = bits[(bits < 0x7F7F)]                       # positive finite, next one also finite
    lo = (pos.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    hi = ((pos + 1).astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    mid = 0.5 * (lo + hi)                             # exact in double
    even = np.where(pos % 2 == 0, pos, pos + 1).astype(np.uint16)
    assert np.array_equal(oracle.round_to(oracle.BF16, mid), even)
    assert np.array_equal(oracle.round_to(oracle.BF16, np.nextafter(mid, -np.inf)), pos)
    assert np.array_equal(oracle.round_to(oracle.BF16, np.nextafter(mid, np.inf)), (pos + 1).astype(np.uint16))
    assert np.array_equal(oracle.round_to(oracle.BF16, -mid), even | 0x8000)
    # overflow to infinity
    assert list(oracle.round_to(oracle.BF16, [3.5e38, -3.5e38])) == [0x7F80, 0xFF80]
    # float32 inputs: agrees with torch's float32 -> bfloat16 conversion
    x32 = (np.random.default_rng(4).standard_normal(50000) * 3).astype(np.float32)
    assert np.array_equal(oracle.round_to(oracle.BF16, x32.astype(np.float64)), W.encode(x32, "bf16"))


# ---------------------------------------------------------------- hand-worked example
def _golden():
    out = {}
    with open(os.path.join(GOLD, "gemm_2x3x2_hand.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            k, *v = line.split()
            out[k] = np.array([float(t) for t in v])
    return out


@pytest.mark.parametrize("t", ["f16", "bf16", "f32"])
def test_hand_worked_example(oracle, t):
    g = _golden()
    A, B, C0 = (W.encode(g[k].astype(np.float32), t) for k in ("A", "B", "C0"))
    tt = T[t]
    ref, S = oracle.gemm(tt, tt, 0, 0, 2, 2, 3, 1.0, A, 3, B, 2, 0.0, None, 2)
    assert np.array_equal(ref.ravel(), g["AB"])
    assert np.array_equal(S.ravel(), g["AB"])
    ref, _ = oracle.gemm(tt, tt, 0, 0, 2, 2, 3, 0.5, A, 3, B, 2, 2.0, C0, 2)
    assert np.array_equal(ref.ravel(), g["REF_ALPHA0.5_BETA2"])
    ref, _ = oracle.gemm(tt, tt, 1, 0, 2, 2, 3, 1.0, A, 2, B, 2, 0.0, None, 2)       # A stored 3x2
    assert np.array_equal(ref.ravel(), g["AtB"])
    ref, _ = oracle.gemm(tt, tt, 0, 1, 2, 2, 3, 1.0, A, 3, B, 3, 0.0, None, 2)       # B stored 2x3
    assert np.array_equal(ref.ravel(), g["ABt"])
    si, sj = np.array([0, 0, 1, 1]), np.array([0, 1, 0, 1])
    ref, S = oracle.gemm_points(tt, tt, 0, 1, 2, 2, 3, 1.0, A, 3, B, 3, 0.0, None, 2, si, sj)
    assert np.array_equal(ref, g["ABt"]) and np.array_equal(S, g["ABt"])


# ---------------------------------------------------------------- closed forms
def _case(t, ta, tb, M, N, K, dist="uniform", **kw):
    code = {"f16": W.PEAK_F16_F32, "bf16": W.PEAK_BF16_BF16, "f32": W.PEAK_F32_F32}[t]
    return W.GemmCase("pin", code, ta, tb, M, N, K, dist=dist, **kw)


def _run(oracle, c, A, B, C0=None, alpha=None, beta=None):
    alpha = c.alpha if alpha is None else alpha
    beta = c.beta if beta is None else beta
    return oracle.gemm(T[c.in_type], T[c.out_type], c.transA, c.transB, c.M, c.N, c.K, alpha, A, c.lda, B, c.ldb,
                       beta, C0, c.ldc)


def _stored(op_mat, trans, t, ld_pad=0):
    """Store a logical op() matrix (float64 values exactly representable in t) with an optional pitch pad."""
    m = op_mat.T if trans else op_mat
    return W._padded(np.ascontiguousarray(m, dtype=np.float32), t, m.shape[1] + ld_pad)


@pytest.mark.parametrize("t", ["f16", "bf16", "f32"])
@pytest.mark.parametrize("ta,tb", [(0, 0), (0, 1), (1, 0), (1, 1)])
def test_identity_and_permutation(oracle, t, ta, tb):
    rng = np.random.default_rng(10 + 2 * ta + tb)
    n, N = 37, 23
    X = W.to_float64(W.encode(rng.standard_normal((n, N)).astype(np.float32), t), t)   # exact values of type t
    perm = rng.permutation(n)
    P = np.zeros((n, n))
    P[np.arange(n), perm] = -1.0                      # signed permutation: row i of C = -row perm[i] of X
    c = _case(t, ta, tb, n, N, n, pad_a=3, pad_b=5)
    A, B = _stored(np.eye(n), ta, t, 3), _stored(X, tb, t, 5)
    ref, S = _run(oracle, c, A, B)
    assert np.array_equal(ref, X) and np.array_equal(S, np.abs(X))
    ref, _ = _run(oracle, c, _stored(P, ta, t, 3), B)
    assert np.array_equal(ref, -X[perm])
    # identity on the right: C == A
    Y = W.to_float64(W.encode(rng.standard_normal((N, n)).astype(np.float32), t), t)
    c2 = _case(t, ta, tb, N, n, n, pad_a=3, pad_b=5)
    ref, _ = _run(oracle, c2, _stored(Y, ta, t, 3), _stored(np.eye(n), tb, t, 5))
    assert np.array_equal(ref, Y)


@pytest.mark.parametrize("t", ["f16", "bf16", "f32"])
@pytest.mark.parametrize("ta,tb", [(0, 0), (0, 1), (1, 0), (1, 1)])
def test_rank1_closed_form(oracle, t, ta, tb):
    rng = np.random.default_rng(20)
    M, N, K = 19, 31, 45
    u, v = rng.integers(-3, 4, M), rng.integers(-3, 4, K)
    w, z = rng.integers(-3, 4, K), rng.integers(-3, 4, N)
    A = np.outer(u, v).astype(np.float64)              # A_ik = u_i v_k
    B = np.outer(w, z).astype(np.float64)              # B_kj = w_k z_j
    c = _case(t, ta, tb, M, N, K)
    ref, S = _run(oracle, c, _stored(A, ta, t), _stored(B, tb, t))
    assert np.array_equal(ref, float(v @ w) * np.outer(u, z))
    assert np.array_equal(S, float(np.abs(v) @ np.abs(w)) * np.outer(np.abs(u), np.abs(z)))
    # special case A_ik = a_i, B_kj = b_j  ->  K a_i b_j
    ref, _ = _run(oracle, c, _stored(np.outer(u, np.ones(K)), ta, t), _stored(np.outer(np.ones(K), z), tb, t))
    assert np.array_equal(ref, K * np.outer(u, z))


@pytest.mark.parametrize("t", ["f16", "bf16", "f32"])
@pytest.mark.parametrize("ta,tb", [(0, 0), (0, 1), (1, 0), (1, 1)])
def test_exact_small_integers(oracle, t, ta, tb):
    """Entries in [-4, 4]: the result is an integer computed exactly by int64 matmul."""
    c = _case(t, ta, tb, 33, 65, 129, dist="smallint", pad_a=1, pad_b=2, pad_c=3, beta=-3.0, alpha=2.0)
    A, B, C0 = W.make_inputs(c)
    Ai = W.to_float64(A[:, :c.a_shape[1]], c.in_type).astype(np.int64)
    Bi = W.to_float64(B[:, :c.b_shape[1]], c.in_type).astype(np.int64)
    Ci = W.to_float64(C0[:, :c.N], c.out_type).astype(np.int64)
    opA = Ai.T if ta else Ai
    opB = Bi.T if tb else Bi
    ref, S = _run(oracle, c, A, B, C0)
    assert np.array_equal(ref, (2 * (opA @ opB) - 3 * Ci).astype(np.float64))
    assert np.array_equal(S, (np.abs(opA) @ np.abs(opB)).astype(np.float64))


@pytest.mark.parametrize("t", ["f16", "bf16", "f32"])
@pytest.mark.parametrize("ta,tb", [(0, 0), (0, 1), (1, 0), (1, 1)])
def test_against_numpy_float64(oracle, t, ta, tb):
    rng = np.random.default_rng(30)
    for (M, N, K) in [(1, 1, 1), (7, 5, 3), (64, 48, 80), (50, 70, 33)]:
        for alpha, beta in [(1.0, 0.0), (-1.0, 1.0), (0.5, 2.0), (2.0, -0.5)]:
            c = _case(t, ta, tb, M, N, K, pad_a=2, pad_b=1, pad_c=4, alpha=alpha, beta=beta,
                      case=int(rng.integers(1 << 20)))
            A, B, C0 = W.make_inputs(c, need_c0=True)
            a = W.to_float64(A[:, :c.a_shape[1]], c.in_type)
            b = W.to_float64(B[:, :c.b_shape[1]], c.in_type)
            c0 = W.to_float64(C0[:, :N], c.out_type)
            opA, opB = (a.T if ta else a), (b.T if tb else b)
            want = alpha * (opA @ opB) + beta * c0
            ref, S = _run(oracle, c, A, B, C0)
            scale = np.abs(alpha) * (np.abs(opA) @ np.abs(opB)) + np.abs(beta * c0)
            assert np.all(np.abs(ref - want) <= 1e-13 * scale + 1e-300)
            assert np.all(np.abs(S - np.abs(opA) @ np.abs(opB)) <= 1e-13 * S)
            assert np.all(S * abs(alpha) + np.abs(beta * c0) >= np.abs(ref) * (1 - 1e-12))


def test_alpha_beta_invariants(oracle):
    c = _case("bf16", 0, 0, 21, 34, 55, beta=1.0)
    A, B, C0 = W.make_inputs(c)
    c0 = W.to_float64(C0, "bf16")
    # alpha = 0, beta = 1: C unchanged
    ref, _ = _run(oracle, c, A, B, C0, alpha=0.0, beta=1.0)
    assert np.array_equal(ref, c0)
    # beta = 0: C0 is not read (NaN there does not reach the result; a null C0 is accepted)
    nanC = W.poison_c(c)
    r1, _ = _run(oracle, c, A, B, nanC, alpha=1.0, beta=0.0)
    r2, _ = _run(oracle, c, A, B, None, alpha=1.0, beta=0.0)
    assert not np.isnan(r1).any() and np.array_equal(r1, r2)
    # alpha = 0 and beta = 0: all zeros
    r0, _ = _run(oracle, c, A, B, nanC, alpha=0.0, beta=0.0)
    assert np.array_equal(r0, np.zeros_like(r0))
    # power-of-two scaling is exact
    r4, _ = _run(oracle, c, A, B, None, alpha=4.0, beta=0.0)
    assert np.array_equal(r4, 4.0 * r1)
    # ref(alpha, beta) = alpha * ref(1, 0) + beta * C0, to fp64 rounding
    r, _ = _run(oracle, c, A, B, C0, alpha=0.5, beta=2.0)
    assert np.allclose(r, 0.5 * r1 + 2.0 * c0, rtol=1e-14, atol=0)
    # A = 0: C = beta * C0
    Z = np.zeros_like(A)
    rz, Sz = _run(oracle, c, Z, B, C0, alpha=1.0, beta=1.0)
    assert np.array_equal(rz, c0) and np.array_equal(Sz, np.zeros_like(Sz))
    # K = 0: empty sum
    ck = _case("bf16", 0, 0, 21, 34, 0, beta=1.0)
    rk, Sk = oracle.gemm(1, 1, 0, 0, 21, 34, 0, 1.0, np.zeros((21, 1), np.uint16), 1, np.zeros((1, 34), np.uint16),
                         34, 2.0, C0, 34)
    assert np.array_equal(rk, 2.0 * c0) and not Sk.any()
    assert ck.K == 0


def test_layout_consistency_and_entry_points_agree(oracle):
    """NN on (A, B), TN on (A^T, B), NT on (A, B^T), TT on (A^T, B^T) give the same ref bit for bit;
    the per-element, sub-grid and full-matrix entry points agree bit for bit."""
    rng = np.random.default_rng(40)
    M, N, K = 45, 52, 67
    a = W.to_float64(W.encode(rng.uniform(-1, 1, (M, K)).astype(np.float32), "f16"), "f16")
    b = W.to_float64(W.encode(rng.uniform(-1, 1, (K, N)).astype(np.float32), "f16"), "f16")
    outs = []
    for ta in (0, 1):
        for tb in (0, 1):
            c = _case("f16", ta, tb, M, N, K, pad_a=ta + 1, pad_b=tb + 2)
            A, B = _stored(a, ta, "f16", ta + 1), _stored(b, tb, "f16", tb + 2)
            outs.append(_run(oracle, c, A, B))
    for r, s in outs[1:]:
        assert np.array_equal(r, outs[0][0]) and np.array_equal(s, outs[0][1])
    c = _case("f16", 1, 0, M, N, K, pad_a=2, pad_b=2)
    A, B = _stored(a, 1, "f16", 2), _stored(b, 0, "f16", 2)
    rows, cols = np.array([0, 7, 44, 13]), np.array([51, 0, 3])
    rs, ss = oracle.gemm_submatrix(0, 2, 1, 0, M, N, K, 1.0, A, c.lda, B, c.ldb, 0.0, None, N, rows, cols)
    assert np.array_equal(rs, outs[0][0][np.ix_(rows, cols)]) and np.array_equal(ss, outs[0][1][np.ix_(rows, cols)])
    ii, jj = np.meshgrid(rows, cols, indexing="ij")
    rp, sp = oracle.gemm_points(0, 2, 1, 0, M, N, K, 1.0, A, c.lda, B, c.ldb, 0.0, None, N, ii.ravel(), jj.ravel())
    assert np.array_equal(rp.reshape(rs.shape), rs) and np.array_equal(sp.reshape(ss.shape), ss)


@pytest.mark.parametrize("t", ["bf16", "f16", "f32"])
@pytest.mark.parametrize("ta,tb", [(1, 0), (0, 1), (0, 0), (1, 1)])
def test_indexed_entry_points_with_old_c(oracle, t, ta, tb):
    """The sub-grid and listed-point entry points with beta != 0: their gather of old C (padded pitch, stored
    output type) must give the full-matrix result bit for bit, and agree with numpy's float64
    alpha * (op(A) @ op(B)) + beta * C0 at the same places -- a wrong row/column index, a missing pitch or a
    dropped beta term in the indexed paths fails here.  Small-integer inputs make the second check exact."""
    M, N, K = 37, 53, 41
    rng = np.random.default_rng(77 + 2 * ta + tb)
    rows = np.array([36, 0, 5, 5, 20, 1])          # unsorted, with a repeat
    cols = np.array([52, 3, 0, 17, 51, 3, 30])
    for dist, (alpha, beta) in [("uniform", (0.5, 2.0)), ("uniform", (1.0, 1.0)), ("smallint", (2.0, -3.0))]:
        c = _case(t, ta, tb, M, N, K, dist=dist, pad_a=3, pad_b=1, pad_c=5, alpha=alpha, beta=beta,
                  case=int(rng.integers(1 << 20)))
        A, B, C0 = W.make_inputs(c)
        assert c.ldc == N + 5 and C0.shape == (M, N + 5)
        full, Sfull = _run(oracle, c, A, B, C0)
        a = W.to_float64(A[:, :c.a_shape[1]], c.in_type)
        b = W.to_float64(B[:, :c.b_shape[1]], c.in_type)
        c0 = W.to_float64(C0[:, :N], c.out_type)
        opA, opB = (a.T if ta else a), (b.T if tb else b)
        want = (alpha * (opA @ opB) + beta * c0)[np.ix_(rows, cols)]
        scale = (abs(alpha) * (np.abs(opA) @ np.abs(opB)) + np.abs(beta * c0))[np.ix_(rows, cols)]
        rs, ss = oracle.gemm_submatrix(T[c.in_type], T[c.out_type], ta, tb, M, N, K, alpha, A, c.lda, B,
                                       c.ldb, beta, C0, c.ldc, rows, cols)
        assert np.array_equal(rs, full[np.ix_(rows, cols)]) and np.array_equal(ss, Sfull[np.ix_(rows, cols)])
        ii, jj = np.meshgrid(rows, cols, indexing="ij")
        rp, sp = oracle.gemm_points(T[c.in_type], T[c.out_type], ta, tb, M, N, K, alpha, A, c.lda, B, c.ldb, beta, C0, c.ldc,
                                    ii.ravel(), jj.ravel())
        assert np.array_equal(rp.reshape(rs.shape), rs) and np.array_equal(sp.reshape(ss.shape), ss)
        if dist == "smallint":
            assert np.array_equal(rs, want)
        else:
            assert np.all(np.abs(rs - want) <= 1e-13 * scale + 1e-300)
        # beta really enters: dropping the old-C term would change the answer
        r0, _ = oracle.gemm_submatrix(T[c.in_type], T[c.out_type], ta, tb, M, N, K, alpha, A, c.lda, B, c.ldb, 0.0,
                                      None, c.ldc, rows, cols)
        if dist == "smallint":
            assert np.array_equal(rs - r0, beta * c0[np.ix_(rows, cols)])
        assert not np.array_equal(rs, r0)


def test_rectangular_not_transposed(oracle):
    """A deliberately asymmetric case: mixing up M/N, or transposing an operand, changes the answer."""
    M, N, K = 3, 5, 2
    a = np.array([[1, 2], [3, 4], [5, 6]], dtype=np.float64)
    b = np.array([[1, 0, -1, 2, 0], [0, 1, 1, 0, -2]], dtype=np.float64)
    want = np.array([[1, 2, 1, 2, -4], [3, 4, 1, 6, -8], [5, 6, 1, 10, -12]], dtype=np.float64)
    c = _case("f32", 0, 0, M, N, K)
    ref, _ = _run(oracle, c, _stored(a, 0, "f32"), _stored(b, 0, "f32"))
    assert np.array_equal(ref, want)


def test_bad_arguments_rejected(oracle):
    z = np.zeros((4, 4), np.uint16)
    with pytest.raises(ValueError):
        oracle.gemm(0, 2, 0, 0, 4, 4, 4, 1.0, z, 3, z, 4, 0.0, None, 4)      # lda < K
    with pytest.raises(ValueError):
        oracle.gemm(0, 2, 0, 0, 4, 4, 4, 1.0, z, 4, z, 4, 1.0, None, 4)      # beta != 0 without C0
    with pytest.raises(ValueError):
        oracle.gemm_points(0, 2, 0, 0, 4, 4, 4, 1.0, z, 4, z, 4, 0.0, None, 4, [4], [0])   # row out of range


# ---------------------------------------------------------------- fused tail (bias + activation)
def test_bias_act_closed_forms(oracle):
    from scipy import special, stats
    rng = np.random.default_rng(50)
    x = np.concatenate([rng.standard_normal((6, 40)) * 3, np.array([[0.0, -0.0, 1.0, -1.0, 8.0, -8.0, 1e-9, -1e-9] * 5])])
    bias = rng.standard_normal(40)
    # identity and ReLU against numpy
    assert np.array_equal(oracle.bias_act(x, None, oracle.ACT_NONE), x)
    assert np.array_equal(oracle.bias_act(x, bias, oracle.ACT_NONE), x + bias[None, :])
    assert np.array_equal(oracle.bias_act(x, bias, oracle.ACT_RELU), np.maximum(x + bias[None, :], 0.0))
    # GELU: x * Phi(x) with scipy's normal CDF, and the erf form with scipy's erf (independent implementations)
    g = oracle.bias_act(x, None, oracle.ACT_GELU)
    assert np.allclose(g, x * stats.norm.cdf(x), rtol=1e-13, atol=1e-15)
    assert np.allclose(g, 0.5 * x * (1 + special.erf(x / np.sqrt(2))), rtol=1e-14, atol=0)
    # textbook values: gelu(0) = 0, gelu(1) = Phi(1) = 0.8413447460685429..., and gelu(x) - gelu(-x) = x
    one = oracle.bias_act(np.array([[0.0, 1.0]]), None, oracle.ACT_GELU)
    assert one[0, 0] == 0.0 and abs(one[0, 1] - 0.8413447460685429) < 1e-15
    assert np.allclose(g - oracle.bias_act(-x, None, oracle.ACT_GELU), x, rtol=1e-14, atol=1e-300)
    # the bias is added per column, before the activation: a bias of -x's column maximum zeroes ReLU everywhere
    big = -(np.abs(x).max(axis=0) + 1.0)
    assert not oracle.bias_act(x, big, oracle.ACT_RELU).any()
    # NaN is not swallowed by ReLU; arguments are checked
    assert np.isnan(oracle.bias_act(np.array([[np.nan]]), None, oracle.ACT_RELU)[0, 0])
    with pytest.raises(ValueError):
        oracle.bias_act(x, bias[:3], oracle.ACT_NONE)
    with pytest.raises(ValueError):
        oracle.bias_act(x, None, 7)


# ---------------------------------------------------------------- 8-bit floats
def test_decode_fp8_exhaustive(oracle):
    """All 256 patterns of each 8-bit format against torch's float8 types (an independent library decoder),
    plus the format's landmark values."""
    import torch
    bits = np.arange(256, dtype=np.uint8)
    for t, tt in ((oracle.E4M3, torch.float8_e4m3fn), (oracle.E5M2, torch.float8_e5m2)):
        want = torch.from_numpy(bits.copy()).view(tt).to(torch.float32).numpy().astype(np.float64)
        got = oracle.decode(t, bits)
        nan = np.isnan(want)
        assert np.array_equal(np.isnan(got), nan)
        assert np.array_equal(got[~nan], want[~nan])
        assert np.array_equal(np.signbit(got[~nan]), np.signbit(want[~nan]))
    d4 = lambda b: oracle.decode(oracle.E4M3, [b])[0]
    d5 = lambda b: oracle.decode(oracle.E5M2, [b])[0]
    assert d4(0x7E) == 448.0 and np.isnan(d4(0x7F)) and d4(0x38) == 1.0 and d4(0x01) == 2.0 ** -9 and d4(0xC0) == -2.0
    assert d5(0x7B) == 57344.0 and np.isinf(d5(0x7C)) and np.isnan(d5(0x7D)) and d5(0x3C) == 1.0 and d5(0x01) == 2.0 ** -16


def test_fp8_gemm_exact_integers(oracle):
    """E4M3 / E5M2 inputs holding small integers: the oracle's result equals int64 matmul exactly."""
    import torch
    rng = np.random.default_rng(60)
    for t, tt in ((oracle.E4M3, torch.float8_e4m3fn), (oracle.E5M2, torch.float8_e5m2)):
        M, N, K = 9, 14, 37
        a = rng.integers(-4, 5, (M, K)); b = rng.integers(-4, 5, (N, K))       # NT: B stored N x K
        A = torch.from_numpy(a.astype(np.float32)).to(tt).view(torch.uint8).numpy()
        B = torch.from_numpy(b.astype(np.float32)).to(tt).view(torch.uint8).numpy()
        ref, S = oracle.gemm(t, oracle.F32, 0, 1, M, N, K, 1.0, A, K, B, K, 0.0, None, N)
        assert np.array_equal(ref, (a @ b.T).astype(np.float64))
        assert np.array_equal(S, (np.abs(a) @ np.abs(b).T).astype(np.float64))


@pytest.mark.parametrize("t", ["f16", "bf16", "f32"])
def test_residual_add_matches_library_decode(oracle, t):
    """The residual operand of the fused tail: x + R with R decoded from its stored bits, padded pitch honoured.
    Checked against numpy addition of library-decoded values (exact: one fp64 addition either way), on random
    bit patterns that include subnormals and infinities, and against a misplaced pitch."""
    rng = np.random.default_rng(90)
    rows, cols, ldr = 13, 21, 29
    x = rng.standard_normal((rows, cols))
    if t == "f32":
        R = rng.standard_normal((rows, ldr)).astype(np.float32)
        R[0, :4] = [np.float32(1e-42), np.float32(-3e38), np.inf, -0.0]
        vals = R.astype(np.float64)
    else:
        R = rng.integers(0, 1 << 16, size=(rows, ldr), dtype=np.uint64).astype(np.uint16)
        vals = W.to_float64(R, t)
    got = oracle.residual_add(x, R, T[t], ldr)
    with np.errstate(invalid="ignore"):
        want = x + vals[:, :cols]
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan) and np.array_equal(got[~nan], want[~nan])
    assert not np.array_equal(np.nan_to_num(got), np.nan_to_num(x))
    # a wrong pitch would read other elements: the dense copy with ldr = cols must agree as well
    dense = np.ascontiguousarray(R[:, :cols])
    got2 = oracle.residual_add(x, dense, T[t], cols)
    assert np.array_equal(np.isnan(got2), nan) and np.array_equal(got2[~nan], want[~nan])
    with pytest.raises(ValueError):
        oracle.residual_add(x, R, T[t], cols - 1)
