"""ctypes binding to libpeak_gemm.so: the same names as the C ABI (include/peak_gemm.h), argument
marshalling only.  Every computation happens in the CUDA library; there is no Python or CPU fallback --
if the shared object is missing, loading fails with an error that says how to build it.

Pointers may be given as torch tensors (``data_ptr()`` is taken), numpy arrays (host entry point), or
plain integers.  Streams may be ``torch.cuda.Stream`` objects, integers or None (default stream).
"""
from __future__ import annotations

import ctypes
import os

PEAK_F16_F32, PEAK_BF16_BF16, PEAK_F32_F32, PEAK_F16_F16, PEAK_BF16_F32 = 0, 1, 2, 3, 4
PEAK_E4M3_BF16, PEAK_E4M3_F32, PEAK_E5M2_BF16, PEAK_E5M2_F32 = 5, 6, 7, 8
PEAK_OK, PEAK_ERR_INVALID_VALUE, PEAK_ERR_ARCH, PEAK_ERR_CUDA, PEAK_ERR_UNSUPPORTED, PEAK_ERR_TIMEOUT, \
    PEAK_ERR_NO_MEMORY, PEAK_ERR_WORKSPACE_TOO_SMALL = range(8)
PEAK_VARIANT_AUTO, PEAK_VARIANT_FALLBACK, PEAK_VARIANT_UMMA_1CTA, PEAK_VARIANT_UMMA_2CTA, PEAK_VARIANT_SGEMM, \
    PEAK_VARIANT_SCALE, PEAK_VARIANT_NONE = range(7)

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpeak_gemm.so")
_lib = None

EXPORTS = ["peak_gemm", "peak_gemm_variant", "peak_gemm_host", "peak_release_staging", "peak_gemm_xcheck_f64",
           "peak_query_variant", "peak_tile_coord", "peak_set_tuning", "peak_check", "peak_kernel_launches", "peak_last_cuda_error",
           "peak_status_string", "peak_variant_string", "peak_version", "peak_gemm_static_ws", "peak_static_ws_bytes", "peak_multicast_available", "peak_gemm_fused",
           "peak_gemm_fused_variant", "peak_gemm_strided_batched", "peak_last_kernel", "peak_selftest_per_device_once",
           "peak_gemm_fused_residual", "peak_gemm_fused_residual_variant", "peak_tuned_table_load",
           "peak_tuned_table_entries", "peak_tuned_lookup"]


class PeakError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = peak_status_string(status)
        if status == PEAK_ERR_CUDA:
            msg += f" (cudaError {peak_last_cuda_error()})"
        super().__init__(f"{where}: {msg}")


def load():
    """Load the CUDA library (once).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2512_19018_b200.build` "
            "(nvcc, sm_100a).  There is no fallback path.")
    lib = ctypes.CDLL(LIB_PATH)
    i, i64, f, vp = ctypes.c_int, ctypes.c_int64, ctypes.c_float, ctypes.c_void_p
    gemm_args = [i, i, i, i64, i64, i64, f, vp, i64, vp, i64, f, vp, i64, vp]
    lib.peak_gemm.restype = i
    lib.peak_gemm.argtypes = gemm_args
    lib.peak_gemm_variant.restype = i
    lib.peak_gemm_variant.argtypes = [i] + gemm_args
    lib.peak_gemm_host.restype = i
    lib.peak_gemm_host.argtypes = gemm_args
    lib.peak_gemm_static_ws.restype = i
    lib.peak_gemm_static_ws.argtypes = gemm_args[:-1] + [i, vp]
    lib.peak_static_ws_bytes.restype = ctypes.c_size_t
    lib.peak_static_ws_bytes.argtypes = []
    lib.peak_gemm_fused.restype = i
    lib.peak_gemm_fused.argtypes = gemm_args[:-1] + [vp, i, vp]
    lib.peak_gemm_fused_variant.restype = i
    lib.peak_gemm_fused_variant.argtypes = [i] + gemm_args[:-1] + [vp, i, vp]
    lib.peak_gemm_fused_residual.restype = i
    lib.peak_gemm_fused_residual.argtypes = gemm_args[:-1] + [vp, i, vp, i64, vp]
    lib.peak_gemm_fused_residual_variant.restype = i
    lib.peak_gemm_fused_residual_variant.argtypes = [i] + gemm_args[:-1] + [vp, i, vp, i64, vp]
    lib.peak_gemm_strided_batched.restype = i
    lib.peak_gemm_strided_batched.argtypes = [i, i, i, i64, i64, i64, f, vp, i64, i64, vp, i64, i64, f, vp, i64, i64,
                                              i64, vp]
    lib.peak_multicast_available.restype = i
    lib.peak_multicast_available.argtypes = []
    lib.peak_release_staging.restype = i
    lib.peak_release_staging.argtypes = []
    lib.peak_gemm_xcheck_f64.restype = i
    lib.peak_gemm_xcheck_f64.argtypes = [i, i, i, i64, i64, i64, f, vp, i64, vp, i64, f, vp, i64, vp, i64, vp]
    lib.peak_query_variant.restype = i
    lib.peak_query_variant.argtypes = [i, i, i, i64, i64, i64, f, vp, i64, vp, i64, f, vp, i64]
    lib.peak_tile_coord.restype = i
    lib.peak_tile_coord.argtypes = [i64, i64, i64, i64, ctypes.POINTER(i64), ctypes.POINTER(i64)]
    lib.peak_set_tuning.restype = i
    lib.peak_set_tuning.argtypes = [i, i]
    lib.peak_check.restype = i
    lib.peak_check.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32)]
    lib.peak_kernel_launches.restype = i64
    lib.peak_kernel_launches.argtypes = []
    lib.peak_last_cuda_error.restype = i
    lib.peak_last_cuda_error.argtypes = []
    lib.peak_last_kernel.restype = i
    lib.peak_last_kernel.argtypes = [ctypes.c_char_p, ctypes.c_size_t]
    lib.peak_selftest_per_device_once.restype = i
    lib.peak_selftest_per_device_once.argtypes = []
    lib.peak_tuned_table_load.restype = i
    lib.peak_tuned_table_load.argtypes = [ctypes.c_char_p]
    lib.peak_tuned_table_entries.restype = i
    lib.peak_tuned_table_entries.argtypes = []
    lib.peak_tuned_lookup.restype = i
    lib.peak_tuned_lookup.argtypes = [i, i, i, i64, i64, i64, f, ctypes.POINTER(i), ctypes.POINTER(i)]
    lib.peak_status_string.restype = ctypes.c_char_p
    lib.peak_status_string.argtypes = [i]
    lib.peak_variant_string.restype = ctypes.c_char_p
    lib.peak_variant_string.argtypes = [i]
    lib.peak_version.restype = i
    lib.peak_version.argtypes = []
    _lib = lib
    return lib


def _ptr(x):
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):          # torch tensor
        return x.data_ptr()
    if hasattr(x, "ctypes"):            # numpy array
        return x.ctypes.data
    raise TypeError(f"cannot take a pointer from {type(x)}")


def _stream(s):
    if s is None:
        return None
    if isinstance(s, int):
        return s
    return s.cuda_stream                # torch.cuda.Stream


def _raise(rc, where):
    if rc != PEAK_OK:
        raise PeakError(rc, where)
    return rc


def peak_gemm(dtype, transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, stream=None, check=True):
    rc = load().peak_gemm(dtype, int(transA), int(transB), M, N, K, alpha, _ptr(A), lda, _ptr(B), ldb, beta,
                          _ptr(C), ldc, _stream(stream))
    return _raise(rc, "peak_gemm") if check else rc


def peak_gemm_variant(variant, dtype, transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, stream=None,
                      check=True):
    rc = load().peak_gemm_variant(variant, dtype, int(transA), int(transB), M, N, K, alpha, _ptr(A), lda, _ptr(B),
                                  ldb, beta, _ptr(C), ldc, _stream(stream))
    return _raise(rc, "peak_gemm_variant") if check else rc


def peak_gemm_host(dtype, transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, stream=None, check=True):
    rc = load().peak_gemm_host(dtype, int(transA), int(transB), M, N, K, alpha, _ptr(A), lda, _ptr(B), ldb, beta,
                               _ptr(C), ldc, _stream(stream))
    return _raise(rc, "peak_gemm_host") if check else rc


def peak_gemm_static_ws(dtype, transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, splits, stream=None,
                        check=True):
    """Split-K GEMM whose partial tiles live in the library's fixed 32 MiB array: no allocation at call time."""
    rc = load().peak_gemm_static_ws(dtype, int(transA), int(transB), M, N, K, alpha, _ptr(A), lda, _ptr(B), ldb, beta,
                                    _ptr(C), ldc, int(splits), _stream(stream))
    return _raise(rc, "peak_gemm_static_ws") if check else rc


def peak_static_ws_bytes() -> int:
    return load().peak_static_ws_bytes()


PEAK_ACT_NONE, PEAK_ACT_RELU, PEAK_ACT_GELU = 0, 1, 2


def peak_gemm_fused(dtype, transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, bias, activation, stream=None,
                    check=True, variant=None):
    """C = act(alpha*op(A)*op(B) + beta*C + bias); `variant` (optional) names the kernel family."""
    lib = load()
    if variant is None:
        rc = lib.peak_gemm_fused(dtype, int(transA), int(transB), M, N, K, alpha, _ptr(A), lda, _ptr(B), ldb, beta,
                                 _ptr(C), ldc, _ptr(bias), int(activation), _stream(stream))
    else:
        rc = lib.peak_gemm_fused_variant(int(variant), dtype, int(transA), int(transB), M, N, K, alpha, _ptr(A), lda,
                                         _ptr(B), ldb, beta, _ptr(C), ldc, _ptr(bias), int(activation), _stream(stream))
    return _raise(rc, "peak_gemm_fused") if check else rc


def peak_gemm_fused_variant(variant, dtype, transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, bias,
                            activation, stream=None, check=True):
    return peak_gemm_fused(dtype, transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, bias, activation,
                           stream, check, variant)


def peak_gemm_fused_residual(dtype, transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, bias, activation, R,
                             ldr, stream=None, check=True, variant=None):
    """C = act(alpha*op(A)*op(B) + beta*C + bias) + R; `variant` (optional) names the kernel family."""
    lib = load()
    if variant is None:
        rc = lib.peak_gemm_fused_residual(dtype, int(transA), int(transB), M, N, K, alpha, _ptr(A), lda, _ptr(B), ldb,
                                          beta, _ptr(C), ldc, _ptr(bias), int(activation), _ptr(R), ldr, _stream(stream))
    else:
        rc = lib.peak_gemm_fused_residual_variant(int(variant), dtype, int(transA), int(transB), M, N, K, alpha, _ptr(A),
                                                  lda, _ptr(B), ldb, beta, _ptr(C), ldc, _ptr(bias), int(activation),
                                                  _ptr(R), ldr, _stream(stream))
    return _raise(rc, "peak_gemm_fused_residual") if check else rc


def peak_gemm_fused_residual_variant(variant, dtype, transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, bias,
                                     activation, R, ldr, stream=None, check=True):
    return peak_gemm_fused_residual(dtype, transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, bias, activation,
                                    R, ldr, stream, check, variant)


def peak_gemm_strided_batched(dtype, transA, transB, M, N, K, alpha, A, lda, strideA, B, ldb, strideB, beta, C, ldc,
                              strideC, batch, stream=None, check=True):
    rc = load().peak_gemm_strided_batched(dtype, int(transA), int(transB), M, N, K, alpha, _ptr(A), lda, strideA,
                                          _ptr(B), ldb, strideB, beta, _ptr(C), ldc, strideC, batch, _stream(stream))
    return _raise(rc, "peak_gemm_strided_batched") if check else rc


def peak_multicast_available() -> bool:
    return bool(load().peak_multicast_available())


def peak_release_staging():
    return load().peak_release_staging()


def peak_gemm_xcheck_f64(dtype, transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C0, ldc, Cref, ldcref,
                         stream=None, check=True):
    rc = load().peak_gemm_xcheck_f64(dtype, int(transA), int(transB), M, N, K, alpha, _ptr(A), lda, _ptr(B), ldb,
                                     beta, _ptr(C0), ldc, _ptr(Cref), ldcref, _stream(stream))
    return _raise(rc, "peak_gemm_xcheck_f64") if check else rc


def peak_query_variant(dtype, transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc):
    return load().peak_query_variant(dtype, int(transA), int(transB), M, N, K, alpha, _ptr(A), lda, _ptr(B), ldb,
                                     beta, _ptr(C), ldc)


def peak_tile_coord(tile, tiles_m, tiles_n, group):
    tm, tn = ctypes.c_int64(-1), ctypes.c_int64(-1)
    rc = load().peak_tile_coord(tile, tiles_m, tiles_n, group, ctypes.byref(tm), ctypes.byref(tn))
    if rc != PEAK_OK:
        raise PeakError(rc, "peak_tile_coord")
    return tm.value, tn.value


PEAK_TUNE_RASTER_GROUP, PEAK_TUNE_TILE_N, PEAK_TUNE_SPLIT_K, PEAK_TUNE_EPILOGUE, PEAK_TUNE_SGEMM_FMA, \
    PEAK_TUNE_TAIL_SPLIT, PEAK_TUNE_DEPENDENT_LAUNCH, PEAK_TUNE_SGEMM_COPY, PEAK_TUNE_WAIT_MS, \
    PEAK_TUNE_INJECT_STALL, PEAK_TUNE_MULTICAST, PEAK_TUNE_BALANCED_GRID, PEAK_TUNE_EPILOGUE_WARPS, \
    PEAK_TUNE_K_ORDER, PEAK_TUNE_SWAP_AB, PEAK_TUNE_SGEMM_TRANSPOSE, PEAK_TUNE_SHORT_A, PEAK_TUNE_CLUSTER_K, PEAK_TUNE_SHARE, PEAK_TUNE_NARROW = \
    0, 1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 11, 12, 13, 14, 15, 16, 17, 18, 19
PEAK_TUNE_COUNT = 20


def peak_set_tuning(key: int, value: int) -> int:
    return _raise(load().peak_set_tuning(key, value), "peak_set_tuning")


def peak_check(stream=None):
    """Synchronise the stream and return (status, detail word)."""
    d = ctypes.c_uint32(0)
    rc = load().peak_check(_stream(stream), ctypes.byref(d))
    return rc, d.value


def peak_kernel_launches() -> int:
    return load().peak_kernel_launches()


def peak_last_cuda_error() -> int:
    return load().peak_last_cuda_error()


def peak_last_kernel() -> str:
    """Name and launch configuration of the kernel this thread's last GEMM call launched."""
    buf = ctypes.create_string_buffer(256)
    _raise(load().peak_last_kernel(buf, 256), "peak_last_kernel")
    return buf.value.decode()


def peak_selftest_per_device_once() -> int:
    return load().peak_selftest_per_device_once()


def peak_tuned_table_load(path) -> int:
    """Replace the tuning table with the JSON file at `path` (None / "" empties it); returns the entry count."""
    return load().peak_tuned_table_load(None if not path else os.fsencode(path))


def peak_tuned_table_entries() -> int:
    return load().peak_tuned_table_entries()


def peak_tuned_lookup(dtype, transA, transB, M, N, K, beta):
    """(variant, {key: value}) of the table entry that covers the problem, or None."""
    v = ctypes.c_int(0)
    knobs = (ctypes.c_int * PEAK_TUNE_COUNT)()
    if not load().peak_tuned_lookup(dtype, int(transA), int(transB), M, N, K, beta, ctypes.byref(v), knobs):
        return None
    return v.value, {k: knobs[k] for k in range(PEAK_TUNE_COUNT) if knobs[k]}


def peak_status_string(status: int) -> str:
    return load().peak_status_string(status).decode()


def peak_variant_string(variant: int) -> str:
    return load().peak_variant_string(variant).decode()


def peak_version() -> int:
    return load().peak_version()
