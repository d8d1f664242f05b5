"""Build the C-ABI shared library (sm_100a only) with nvcc, in-tree.

    python -m paper_2602_19128_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
ROOT = PKG.parent
CSRC = PKG / "csrc"
LIB = PKG / "libmoe_b200.so"
SOURCES = ["moe_api.cu", "moe_route.cu", "moe_gemm_tc.cu", "moe_gemm_tc_pair.cu", "moe_gemm_tc_ring.cu", "moe_gemm_tc_fp8w.cu", "moe_gemm_tc_mx.cu", "moe_gemm_tc_mx_pair.cu", "moe_gemm_tc_mx_ring.cu", "moe_mx.cu", "moe_tc_host.cu", "moe_gemm_validation.cu", "gqa_decode.cu"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def needs_build() -> bool:
    if not LIB.exists():
        return True
    deps = [CSRC / s for s in SOURCES] + list(CSRC.glob("*.cuh")) + [ROOT / "include" / "moe.h", ROOT / "include" / "gqa_decode.h"]
    return any(d.stat().st_mtime > LIB.stat().st_mtime for d in deps)


def build_library(force: bool = False, verbose: bool = False) -> Path:
    if not force and not needs_build():
        return LIB
    tmp = LIB.with_suffix(f".{os.getpid()}.tmp.so")
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC,-fvisibility=hidden", "-shared", "-cudart", "static",
           "-I", str(ROOT / "include"), "-I", str(CSRC)]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [str(CSRC / s) for s in SOURCES] + ["-o", str(tmp)]
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
