"""CPU oracle for dense GEMM -- TEST INFRASTRUCTURE ONLY.

Thin ctypes wrapper around ``oracle_gemm.c`` (plain C, fp64 accumulation, own
bit-level decoders).  Only the tests, the smoke check and the benchmark's CPU
baseline leg may import this package; the CUDA library never does, and this
package never imports the CUDA library or its Python binding.

The arithmetic is in the C file, which follows the paper's statement of the
matmul problem (section 2.2) widened to ``alpha*op(A)*op(B) + beta*C`` over
row-major storage.  This module only builds the shared object with gcc and
marshals numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

F16, BF16, F32, E4M3, E5M2 = 0, 1, 2, 3, 4
_NP_STORE = {F16: np.uint16, BF16: np.uint16, F32: np.uint32}

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle_gemm.c")
_SO = os.path.join(_HERE, "liboracle_gemm.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile oracle_gemm.c with gcc (OpenMP) into liboracle_gemm.so."""
    with _lock:
        stale = (not os.path.exists(_SO)) or os.path.getmtime(_SO) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _SO + f".tmp{os.getpid()}"
            cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-fno-fast-math",
                   "-ffp-contract=off", "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, dbl, vp, ci = ctypes.c_int64, ctypes.c_double, ctypes.c_void_p, ctypes.c_int
        lib.oracle_decode_f16.restype = dbl
        lib.oracle_decode_f16.argtypes = [ctypes.c_uint16]
        lib.oracle_decode_bf16.restype = dbl
        lib.oracle_decode_bf16.argtypes = [ctypes.c_uint16]
        lib.oracle_decode_f32.restype = dbl
        lib.oracle_decode_f32.argtypes = [ctypes.c_uint32]
        lib.oracle_decode_e4m3.restype = dbl
        lib.oracle_decode_e4m3.argtypes = [ctypes.c_uint8]
        lib.oracle_decode_e5m2.restype = dbl
        lib.oracle_decode_e5m2.argtypes = [ctypes.c_uint8]
        lib.oracle_round.restype = ci
        lib.oracle_round.argtypes = [ci, vp, i64, vp]
        common = [ci, ci, ci, ci, i64, i64, i64, dbl, vp, i64, vp, i64, dbl, vp, i64]
        lib.oracle_gemm.restype = ci
        lib.oracle_gemm.argtypes = common + [vp, vp]
        lib.oracle_gemm_points.restype = ci
        lib.oracle_gemm_points.argtypes = common + [i64, vp, vp, vp, vp]
        lib.oracle_gemm_submatrix.restype = ci
        lib.oracle_gemm_submatrix.argtypes = common + [i64, vp, i64, vp, vp, vp]
        lib.oracle_bias_act.restype = ci
        lib.oracle_bias_act.argtypes = [vp, i64, i64, vp, ci]
        lib.oracle_residual_add.restype = ci
        lib.oracle_residual_add.argtypes = [vp, i64, i64, ci, vp, i64]
        _lib = lib
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _store(a, t):
    """View `a` as the stored-bits array the C side expects (no copy if possible)."""
    if a is None:
        return None
    a = np.ascontiguousarray(a)
    if t in (E4M3, E5M2):
        if a.dtype != np.uint8:
            raise TypeError("8-bit float operands must be uint8 bit patterns")
        return a
    if t == F32:
        if a.dtype == np.float32:
            return a.view(np.uint32)
        if a.dtype != np.uint32:
            raise TypeError("F32 operands must be float32 or uint32 bit patterns")
        return a
    if a.dtype == np.float16 and t == F16:
        return a.view(np.uint16)
    if a.dtype != np.uint16:
        raise TypeError("16-bit operands must be uint16 bit patterns (or float16 for F16)")
    return a


def _min_elems(rows, ld):
    return 0 if rows == 0 else (rows - 1) * ld + 1


def _check_sizes(transA, transB, M, N, K, A, lda, B, ldb, C0, ldc, beta):
    ra, ca = (K, M) if transA else (M, K)
    rb, cb = (N, K) if transB else (K, N)
    if ra and A.size < (ra - 1) * lda + ca:
        raise ValueError("A too small for its shape / lda")
    if rb and B.size < (rb - 1) * ldb + cb:
        raise ValueError("B too small for its shape / ldb")
    if beta != 0 and M and N:
        if C0 is None or C0.size < (M - 1) * ldc + N:
            raise ValueError("C0 too small for its shape / ldc")


def decode(t: int, bits) -> np.ndarray:
    """Decode stored bit patterns to float64 with the oracle's own decoders."""
    lib = _load()
    fn = {F16: lib.oracle_decode_f16, BF16: lib.oracle_decode_bf16, F32: lib.oracle_decode_f32,
          E4M3: lib.oracle_decode_e4m3, E5M2: lib.oracle_decode_e5m2}[t]
    flat = np.asarray(bits).ravel()
    return np.array([fn(int(b)) for b in flat], dtype=np.float64).reshape(np.shape(bits))


def round_to(t: int, x) -> np.ndarray:
    """Round float64 values to storage type `t` (one rounding, ties to even); returns the bit patterns."""
    lib = _load()
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty(x.shape, dtype=_NP_STORE[t])
    rc = lib.oracle_round(t, _ptr(x), x.size, _ptr(out))
    if rc:
        raise ValueError(f"oracle_round failed: {rc}")
    return out


def gemm(in_type, c_type, transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C0, ldc, want_S=True):
    """Full-matrix oracle.  Returns (ref, S): float64 arrays of shape (M, N); S is None if not wanted."""
    lib = _load()
    A, B, C0 = _store(A, in_type), _store(B, in_type), _store(C0, c_type)
    _check_sizes(transA, transB, M, N, K, A, lda, B, ldb, C0, ldc, beta)
    ref = np.empty((M, N), dtype=np.float64)
    S = np.empty((M, N), dtype=np.float64) if want_S else None
    rc = lib.oracle_gemm(in_type, c_type, int(transA), int(transB), M, N, K, float(alpha), _ptr(A), lda,
                         _ptr(B), ldb, float(beta), _ptr(C0), ldc, _ptr(ref), _ptr(S))
    if rc:
        raise ValueError(f"oracle_gemm failed: {rc}")
    return ref, S


def gemm_points(in_type, c_type, transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C0, ldc, si, sj,
                want_S=True):
    """Oracle at the listed (si[t], sj[t]) elements.  Returns (ref, S) of shape (len(si),)."""
    lib = _load()
    A, B, C0 = _store(A, in_type), _store(B, in_type), _store(C0, c_type)
    _check_sizes(transA, transB, M, N, K, A, lda, B, ldb, C0, ldc, beta)
    si = np.ascontiguousarray(si, dtype=np.int64)
    sj = np.ascontiguousarray(sj, dtype=np.int64)
    if si.shape != sj.shape or si.ndim != 1:
        raise ValueError("si, sj must be 1-D and of equal length")
    ref = np.empty(si.shape, dtype=np.float64)
    S = np.empty(si.shape, dtype=np.float64) if want_S else None
    rc = lib.oracle_gemm_points(in_type, c_type, int(transA), int(transB), M, N, K, float(alpha), _ptr(A), lda,
                                _ptr(B), ldb, float(beta), _ptr(C0), ldc, si.size, _ptr(si), _ptr(sj),
                                _ptr(ref), _ptr(S))
    if rc:
        raise ValueError(f"oracle_gemm_points failed: {rc}")
    return ref, S


def gemm_submatrix(in_type, c_type, transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C0, ldc, rows, cols,
                   want_S=True):
    """Oracle on the rows x cols sub-grid of C.  Returns (ref, S) of shape (len(rows), len(cols))."""
    lib = _load()
    A, B, C0 = _store(A, in_type), _store(B, in_type), _store(C0, c_type)
    _check_sizes(transA, transB, M, N, K, A, lda, B, ldb, C0, ldc, beta)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    cols = np.ascontiguousarray(cols, dtype=np.int64)
    ref = np.empty((rows.size, cols.size), dtype=np.float64)
    S = np.empty((rows.size, cols.size), dtype=np.float64) if want_S else None
    rc = lib.oracle_gemm_submatrix(in_type, c_type, int(transA), int(transB), M, N, K, float(alpha), _ptr(A),
                                   lda, _ptr(B), ldb, float(beta), _ptr(C0), ldc, rows.size, _ptr(rows),
                                   cols.size, _ptr(cols), _ptr(ref), _ptr(S))
    if rc:
        raise ValueError(f"oracle_gemm_submatrix failed: {rc}")
    return ref, S


ACT_NONE, ACT_RELU, ACT_GELU = 0, 1, 2


def bias_act(ref, bias=None, act=ACT_NONE) -> np.ndarray:
    """Fused tail on top of a computed ref (2-D): ref + bias[col], then the activation; returns a new array."""
    lib = _load()
    x = np.array(ref, dtype=np.float64, order="C", copy=True)
    if x.ndim != 2:
        raise ValueError("ref must be 2-D")
    b = None if bias is None else np.ascontiguousarray(bias, dtype=np.float64)
    if b is not None and b.shape != (x.shape[1],):
        raise ValueError("bias must have one value per column")
    rc = lib.oracle_bias_act(_ptr(x), x.shape[0], x.shape[1], _ptr(b), int(act))
    if rc:
        raise ValueError(f"oracle_bias_act failed: {rc}")
    return x


def residual_add(x, R, r_type: int, ldr: int) -> np.ndarray:
    """x (2-D float64) + the residual matrix R (stored bits of type r_type, row pitch ldr); returns a new array."""
    lib = _load()
    out = np.array(x, dtype=np.float64, order="C", copy=True)
    if out.ndim != 2:
        raise ValueError("x must be 2-D")
    Rb = _store(R, r_type)
    rows, cols = out.shape
    if rows and Rb.size < (rows - 1) * ldr + cols:
        raise ValueError("R too small for its shape / ldr")
    rc = lib.oracle_residual_add(_ptr(out), rows, cols, int(r_type), _ptr(Rb), int(ldr))
    if rc:
        raise ValueError(f"oracle_residual_add failed: {rc}")
    return out


def num_threads() -> int:
    """Threads the OpenMP loops will use (OMP_NUM_THREADS or the affinity mask)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env and env.isdigit() and int(env) > 0:
        return int(env)
    return len(os.sched_getaffinity(0))
