"""Seeded synthetic inputs for the GEMM workloads.

This module only *makes data*: it draws random numbers, rounds them to the
storage type with numpy / torch conversions, and lays them out with a leading
dimension.  It holds none of the GEMM arithmetic and is the one module that the
oracle-side tests and the CUDA-side tests both import, so that the two sides
see byte-identical inputs.

The paper's workload is square random matrices (n = 2048, 4096; fp32 or fp16;
section 4.3); it uses no dataset.  The cases below add the shapes, layouts and
value distributions of the benchmark configurations this library is measured on.

Storage convention (row-major, as in the paper's section 2.2):
  A is stored (K x M if transA else M x K) with row pitch lda,
  B is stored (N x K if transB else K x N) with row pitch ldb,
  C is stored M x N with row pitch ldc.
16-bit operands are returned as uint16 bit patterns, fp32 ones as float32.
Padding columns (index >= logical width, < ld) hold a NaN pattern so that any
read of them shows up in the result.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np
import torch

BASE_SEED = 0x5045414B  # "PEAK"

# dtype pair codes of the C ABI (include/peak_gemm.h)
PEAK_F16_F32, PEAK_BF16_BF16, PEAK_F32_F32, PEAK_F16_F16, PEAK_BF16_F32 = 0, 1, 2, 3, 4
PEAK_E4M3_BF16, PEAK_E4M3_F32, PEAK_E5M2_BF16, PEAK_E5M2_F32 = 5, 6, 7, 8
IN_TYPE = {PEAK_F16_F32: "f16", PEAK_BF16_BF16: "bf16", PEAK_F32_F32: "f32", PEAK_F16_F16: "f16",
           PEAK_BF16_F32: "bf16", PEAK_E4M3_BF16: "e4m3", PEAK_E4M3_F32: "e4m3", PEAK_E5M2_BF16: "e5m2",
           PEAK_E5M2_F32: "e5m2"}
OUT_TYPE = {PEAK_F16_F32: "f32", PEAK_BF16_BF16: "bf16", PEAK_F32_F32: "f32", PEAK_F16_F16: "f16",
            PEAK_BF16_F32: "f32", PEAK_E4M3_BF16: "bf16", PEAK_E4M3_F32: "f32", PEAK_E5M2_BF16: "bf16",
            PEAK_E5M2_F32: "f32"}
NP_STORE = {"f16": np.uint16, "bf16": np.uint16, "f32": np.float32, "e4m3": np.uint8, "e5m2": np.uint8}
ELEM_BYTES = {"f16": 2, "bf16": 2, "f32": 4, "e4m3": 1, "e5m2": 1}
NAN_BITS = {"f16": 0x7E00, "bf16": 0x7FC0, "e4m3": 0x7F, "e5m2": 0x7E}
_TORCH_FP8 = {"e4m3": torch.float8_e4m3fn, "e5m2": torch.float8_e5m2}


@dataclass(frozen=True)
class GemmCase:
    """One GEMM problem: shape, layout, scalars and the input distribution."""
    name: str
    dtype: int                # PEAK_* pair code
    transA: bool
    transB: bool
    M: int
    N: int
    K: int
    alpha: float = 1.0
    beta: float = 0.0
    dist: str = "uniform"     # uniform | normal_rsqrtk | transformer | smallint | ones
    pad_a: int = 0            # lda = minimal + pad_a (elements)
    pad_b: int = 0
    pad_c: int = 0
    config: int = 0           # index into the benchmark configuration list (for the seed)
    case: int = 0

    @property
    def in_type(self) -> str:
        return IN_TYPE[self.dtype]

    @property
    def out_type(self) -> str:
        return OUT_TYPE[self.dtype]

    @property
    def a_shape(self):
        return (self.K, self.M) if self.transA else (self.M, self.K)

    @property
    def b_shape(self):
        return (self.N, self.K) if self.transB else (self.K, self.N)

    @property
    def lda(self) -> int:
        return self.a_shape[1] + self.pad_a

    @property
    def ldb(self) -> int:
        return self.b_shape[1] + self.pad_b

    @property
    def ldc(self) -> int:
        return self.N + self.pad_c

    @property
    def layout(self) -> str:
        return ("T" if self.transA else "N") + ("T" if self.transB else "N")

    @property
    def seed(self) -> int:
        return BASE_SEED + 1000 * self.config + self.case

    @property
    def flops(self) -> float:
        return 2.0 * self.M * self.N * self.K

    def min_bytes(self) -> int:
        """Least HBM traffic: read A and B once, write C once (and read it once if beta != 0)."""
        si, so = ELEM_BYTES[self.in_type], ELEM_BYTES[self.out_type]
        c = self.M * self.N * so
        return (self.M * self.K + self.K * self.N) * si + c * (2 if self.beta != 0 else 1)

    def with_(self, **kw) -> "GemmCase":
        return replace(self, **kw)


def encode(values_f32: np.ndarray, t: str) -> np.ndarray:
    """Round float32 values to storage type t (library conversions, ties to even)."""
    if t == "f32":
        return np.ascontiguousarray(values_f32, dtype=np.float32)
    if t == "f16":
        return values_f32.astype(np.float16).view(np.uint16)
    if t == "bf16":
        tt = torch.from_numpy(np.ascontiguousarray(values_f32, dtype=np.float32)).to(torch.bfloat16)
        return tt.view(torch.int16).numpy().view(np.uint16)
    if t in _TORCH_FP8:
        tt = torch.from_numpy(np.ascontiguousarray(values_f32, dtype=np.float32)).to(_TORCH_FP8[t])
        return tt.view(torch.uint8).numpy()
    raise ValueError(t)


def to_float64(stored: np.ndarray, t: str) -> np.ndarray:
    """Library decode of stored values (for pins that must not use the oracle's own decoders)."""
    if t == "f32":
        return stored.astype(np.float64)
    if t == "f16":
        return stored.view(np.float16).astype(np.float64)
    if t == "bf16":
        return (stored.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    if t in _TORCH_FP8:
        tt = torch.from_numpy(np.ascontiguousarray(stored)).view(_TORCH_FP8[t]).to(torch.float32)
        return tt.numpy().astype(np.float64)
    raise ValueError(t)


def _draw(rng: np.random.Generator, shape, kind: str, scale: float = 1.0) -> np.ndarray:
    if kind == "uniform":        # i.i.d. uniform on [-1, 1)
        x = rng.random(shape, dtype=np.float32)
        x *= 2.0
        x -= 1.0
    elif kind == "normal":
        x = rng.standard_normal(shape, dtype=np.float32)
        if scale != 1.0:
            x *= np.float32(scale)
    elif kind == "smallint":     # integers in [-4, 4]
        x = rng.integers(-4, 5, size=shape).astype(np.float32)
    elif kind == "ones":
        x = np.ones(shape, dtype=np.float32)
    else:
        raise ValueError(kind)
    return x


def _padded(vals: np.ndarray, t: str, ld: int) -> np.ndarray:
    rows, cols = vals.shape
    enc = encode(vals, t)
    if ld == cols:
        return enc
    out = np.empty((rows, ld), dtype=NP_STORE[t])
    if t == "f32":
        out[:, cols:] = np.nan
    else:
        out[:, cols:] = NAN_BITS[t]
    out[:, :cols] = enc
    return out


def make_inputs(case: GemmCase, need_c0: bool | None = None):
    """Return (A, B, C0) numpy arrays in storage layout; C0 is None unless beta != 0 (or need_c0)."""
    rng = np.random.Generator(np.random.Philox(case.seed))
    d = case.dist
    if d == "uniform":
        ka = kb = kc = ("uniform", 1.0)
    elif d == "normal_rsqrtk":   # both operands normal(0,1) / sqrt(K)
        s = 1.0 / float(np.sqrt(max(case.K, 1)))
        ka = kb = ("normal", s)
        kc = ("normal", 1.0)
    elif d == "transformer":     # activations normal(0,1), weights normal(0,0.02), C0 normal(0,1)
        ka, kb, kc = ("normal", 1.0), ("normal", 0.02), ("normal", 1.0)
    elif d == "smallint":
        ka = kb = kc = ("smallint", 1.0)
    elif d == "ones":
        ka = kb = kc = ("ones", 1.0)
    else:
        raise ValueError(d)
    A = _padded(_draw(rng, case.a_shape, *ka), case.in_type, case.lda)
    B = _padded(_draw(rng, case.b_shape, *kb), case.in_type, case.ldb)
    want_c = (case.beta != 0) if need_c0 is None else need_c0
    C0 = _padded(_draw(rng, (case.M, case.N), *kc), case.out_type, case.ldc) if want_c else None
    return A, B, C0


def poison_c(case: GemmCase) -> np.ndarray:
    """A C buffer full of NaN patterns: with beta == 0 nothing of it may survive or propagate."""
    t = case.out_type
    if t == "f32":
        return np.full((case.M, case.ldc), np.nan, dtype=np.float32)
    return np.full((case.M, case.ldc), NAN_BITS[t], dtype=np.uint16)


# ---------------------------------------------------------------------------
# The benchmark configurations (index = position in the configuration list).
# ---------------------------------------------------------------------------

def config0() -> GemmCase:
    """fp16 512^3 NN, alpha=1 beta=0, uniform[-1,1], fp32 output."""
    return GemmCase("fp16_512_nn", PEAK_F16_F32, False, False, 512, 512, 512, 1.0, 0.0, "uniform", config=0)


def config1() -> GemmCase:
    """bf16 4096^3 NN, alpha=1 beta=0, normal(0,1)/sqrt(K), bf16 output."""
    return GemmCase("bf16_4096_nn", PEAK_BF16_BF16, False, False, 4096, 4096, 4096, 1.0, 0.0, "normal_rsqrtk",
                    config=1)


def config2(n: int, layout: str) -> GemmCase:
    """fp16 n^3 sweep, NN or TN, uniform[-1,1], fp32 output."""
    ta = layout[0] == "T"
    tb = layout[1] == "T"
    return GemmCase(f"fp16_{n}_{layout.lower()}", PEAK_F16_F32, ta, tb, n, n, n, 1.0, 0.0, "uniform", config=2,
                    case=n // 1024 * 4 + 2 * ta + tb)


def config3(which: int) -> GemmCase:
    """bf16 transformer-layer GEMMs, 16384 tokens, NT (weights stored N x K), alpha=1 beta=1."""
    shapes = [(16384, 4096, 4096), (16384, 14336, 4096), (16384, 4096, 14336)]
    M, N, K = shapes[which]
    return GemmCase(f"bf16_tfm_{M}x{N}x{K}_nt", PEAK_BF16_BF16, False, True, M, N, K, 1.0, 1.0, "transformer",
                    config=3, case=which)


def config4_sgemm(n: int) -> GemmCase:
    """fp32 SGEMM n^3 NN on CUDA cores, uniform[-1,1]."""
    return GemmCase(f"fp32_{n}_nn", PEAK_F32_F32, False, False, n, n, n, 1.0, 0.0, "uniform", config=4,
                    case=n // 1024)


def config4_ragged(which: int) -> GemmCase:
    """bf16 TN ragged / skinny shapes, alpha=0.5 beta=2, uniform[-1,1] (C0 included)."""
    shapes = [(5000, 3000, 2500), (16, 4096, 4096), (128, 14336, 4096)]
    M, N, K = shapes[which]
    return GemmCase(f"bf16_{M}x{N}x{K}_tn", PEAK_BF16_BF16, True, False, M, N, K, 0.5, 2.0, "uniform", config=4,
                    case=100 + which)


def short_k_workload(k: int = 128) -> GemmCase:
    """bf16 8192 x 8192 x k NT with a short k (a rank-k update): the output, not the operands, bounds the launch."""
    return GemmCase(f"bf16_8192x8192x{k}_nt", PEAK_BF16_BF16, False, True, 8192, 8192, k, 1.0, 0.0, "uniform", config=4,
                    case=200 + k // 64)


def bench_workload() -> GemmCase:
    """The configuration the headline throughput is quoted on."""
    return config1()


def fp8_workload(n: int, in_type: str = "e4m3", layout: str = "NT") -> GemmCase:
    """8-bit float inputs, bf16 output, n^3 (default NT: A row-major, B stored N x K, both with K innermost):
    uniform[-1, 1] values so that the operands use the formats' range (normal / sqrt(K) would fall into the
    subnormals)."""
    dt = PEAK_E4M3_BF16 if in_type == "e4m3" else PEAK_E5M2_BF16
    ta, tb = layout[0] == "T", layout[1] == "T"
    return GemmCase(f"{in_type}_{n}_{layout.lower()}", dt, ta, tb, n, n, n, 1.0, 0.0, "uniform", config=5,
                    case=n + (0 if layout == "NT" else 1 + 2 * ta + tb))


def target_workload() -> GemmCase:
    """bf16 8192^3 NN: the shape the 70 %-of-peak target is stated for (same recipe as config1)."""
    return GemmCase("bf16_8192_nn", PEAK_BF16_BF16, False, False, 8192, 8192, 8192, 1.0, 0.0, "normal_rsqrtk",
                    config=1, case=1)
