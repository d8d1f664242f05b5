"""ctypes loader for the CPU oracle of the paged grouped-query decode attention (TEST INFRASTRUCTURE, not the
product).  Only tests, the smoke check and the benchmark's CPU-baseline leg may import this module.  It compiles
``gqa_oracle.c`` with gcc into a double-precision build (``f64``: parity is judged against it) and a float build
(``f32``: its distance from the double build is the arithmetic's own error bar) and wraps the entry point with
numpy marshalling.  It imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "gqa_oracle.c"
_BUILD = _HERE / "_build"


def build(force: bool = False) -> dict:
    """Compile the oracle (gcc, OpenMP) for both arithmetic types; returns the .so paths."""
    _BUILD.mkdir(exist_ok=True)
    out = {}
    for name, real in (("f32", "float"), ("f64", "double")):
        so = _BUILD / f"libgqa_oracle_{name}.so"
        if force or not so.exists() or so.stat().st_mtime < _SRC.stat().st_mtime:
            tmp = so.with_suffix(f".{os.getpid()}.tmp")
            subprocess.run(["gcc", "-std=c11", "-O2", "-fno-fast-math", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
                            f"-DREAL={real}", str(_SRC), "-o", str(tmp), "-lm"], check=True)
            os.replace(tmp, so)
        out[name] = so
    return out


class GqaOracle:
    def __init__(self, precision: str = "f64"):
        assert precision in ("f32", "f64")
        self.real = np.float32 if precision == "f32" else np.float64
        self.lib = ctypes.CDLL(str(build()[precision]))
        assert self.lib.gqa_oracle_real_bytes() == np.dtype(self.real).itemsize
        self.lib.gqa_oracle_paged_decode.restype = ctypes.c_int
        self.lib.gqa_oracle_paged_decode.argtypes = [ctypes.c_void_p] * 6 + [ctypes.c_int] * 6 + [ctypes.c_double,
                                                                                                  ctypes.c_void_p, ctypes.c_void_p]
        self.num_threads = int(self.lib.gqa_oracle_num_threads())

    def paged_decode(self, q, k_cache, v_cache, kv_indptr, kv_indices, kv_last_page_len, sm_scale: float):
        """q [B,Hq,D], k_cache / v_cache [num_pages,P,Hkv,D] as uint16 bf16 bit patterns; int32 page tables.
        Returns (out [B,Hq,D], lse [B,Hq]) in the build's arithmetic type."""
        arrs = [np.ascontiguousarray(a) for a in (q, k_cache, v_cache)]
        assert all(a.dtype == np.uint16 for a in arrs), "bf16 data must be passed as its uint16 bit pattern"
        q, k_cache, v_cache = arrs
        tabs = [np.ascontiguousarray(a, dtype=np.int32) for a in (kv_indptr, kv_indices, kv_last_page_len)]
        B, Hq, D = q.shape
        num_pages, P, Hkv, D2 = k_cache.shape
        assert D2 == D and v_cache.shape == k_cache.shape and tabs[0].shape == (B + 1,) and tabs[2].shape == (B,)
        if tabs[1].size == 0:
            tabs[1] = np.zeros(1, dtype=np.int32)
        out = np.empty((B, Hq, D), dtype=self.real)
        lse = np.empty((B, Hq), dtype=self.real)
        st = self.lib.gqa_oracle_paged_decode(q.ctypes.data, k_cache.ctypes.data, v_cache.ctypes.data, tabs[0].ctypes.data,
                                              tabs[1].ctypes.data, tabs[2].ctypes.data, B, Hq, Hkv, D, P, num_pages,
                                              float(sm_scale), out.ctypes.data, lse.ctypes.data)
        if st != 0:
            raise ValueError(f"gqa_oracle_paged_decode: status {st}")
        return out, lse


_cache = {}


def get(precision: str = "f64") -> GqaOracle:
    if precision not in _cache:
        _cache[precision] = GqaOracle(precision)
    return _cache[precision]
