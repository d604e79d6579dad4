"""Builds libpeak_gemm.so (the CUDA library behind the C ABI) in-tree with nvcc for sm_100a.

Usage:  python -m paper_2512_19018_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ_DIR = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "libpeak_gemm.so")
# optional single-GPU plug-in (cluster-multicast loads): built only where its source is present
MC_SOURCE = os.path.join(CSRC, "umma_gemm_mc.cu")
MC_LIB = os.path.join(HERE, "libpeak_gemm_mc.so")
SOURCES = ["api.cu", "fallback_gemm.cu", "sgemm.cu", "sgemm_tma.cu", "tuned_table.cu", "umma_gemm.cu"]
HEADERS = [os.path.join(CSRC, h) for h in ("common.cuh", "ptx.cuh", "umma_device.cuh", "umma_clusterk.cuh", "umma_host.cuh",
                                           "mc_plugin.h")] + [
    os.path.join(os.path.dirname(HERE), "include", "peak_gemm.h")]
MC_HEADERS = [os.path.join(CSRC, "umma_share_mc.cuh")]  # plug-in only (multicast copies)
NVCC_FLAGS = ["-std=c++17", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    os.makedirs(OBJ_DIR, exist_ok=True)
    nvcc = _nvcc()
    objs = []
    procs = []
    for src in SOURCES:
        s = os.path.join(CSRC, src)
        o = os.path.join(OBJ_DIR, src.replace(".cu", ".o"))
        objs.append(o)
        if force or _stale(o, [s] + HEADERS):
            cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-c", s, "-o", o]
            procs.append((cmd, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    for cmd, p in procs:
        out, _ = p.communicate()
        if verbose or p.returncode:
            sys.stderr.write(" ".join(cmd) + "\n" + out + "\n")
        if p.returncode:
            raise RuntimeError("nvcc failed: " + " ".join(cmd))
    if force or procs or _stale(LIB, objs):
        tmp = LIB + f".tmp{os.getpid()}"
        cmd = [nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp] + objs + ["-ldl"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, LIB)
    if os.path.exists(MC_SOURCE) and (force or _stale(MC_LIB, [MC_SOURCE] + HEADERS + MC_HEADERS)):
        tmp = MC_LIB + f".tmp{os.getpid()}"
        cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-shared", MC_SOURCE, "-o", tmp]
        r = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
        if verbose or r.returncode:
            sys.stderr.write(" ".join(cmd) + "\n" + r.stdout + "\n")
        if r.returncode:
            raise RuntimeError("nvcc failed: " + " ".join(cmd))
        os.replace(tmp, MC_LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
