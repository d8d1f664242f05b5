"""ctypes loader for the CPU oracle (TEST INFRASTRUCTURE, not the product).

Only tests, the smoke check and the benchmark's CPU-baseline / reference legs may import
this module.  It compiles ``moe_oracle.c`` with gcc into two shared objects -- one with
every floating-point operation in float (``f32``, the precision the layer is specified in)
and one in double (``f64``, the error bar for the float build) -- and wraps their entry
points with numpy-array marshalling.  It imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "moe_oracle.c"
_BUILD = _HERE / "_build"

_c_i32p = ctypes.POINTER(ctypes.c_int32)
_c_f32p = ctypes.POINTER(ctypes.c_float)
_c_u16p = ctypes.POINTER(ctypes.c_uint16)


def build(force: bool = False) -> dict[str, Path]:
    """Compile the oracle (gcc, OpenMP) for both arithmetic types; returns the .so paths."""
    _BUILD.mkdir(exist_ok=True)
    out = {}
    for name, real in (("f32", "float"), ("f64", "double")):
        so = _BUILD / f"liboracle_{name}.so"
        if force or not so.exists() or so.stat().st_mtime < _SRC.stat().st_mtime:
            tmp = so.with_suffix(f".{os.getpid()}.tmp")
            cmd = ["gcc", "-std=c11", "-O2", "-fno-fast-math", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
                   f"-DREAL={real}", str(_SRC), "-o", str(tmp), "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, so)
        out[name] = so
    return out


class Oracle:
    """One precision build of the oracle.  Arrays in, arrays out; bf16 tensors travel as uint16."""

    def __init__(self, precision: str = "f32"):
        assert precision in ("f32", "f64")
        self.precision = precision
        self.real = np.float32 if precision == "f32" else np.float64
        self.lib = ctypes.CDLL(str(build()[precision]))
        assert self.lib.moe_oracle_real_bytes() == np.dtype(self.real).itemsize
        for fn in ("moe_oracle_route", "moe_oracle_permute", "moe_oracle_expert_ffn", "moe_oracle_forward",
                   "moe_oracle_forward_sampled", "moe_oracle_sorted_intermediates", "moe_oracle_forward_local",
                   "moe_oracle_permute_local", "moe_oracle_forward_fp8w", "moe_oracle_mx_quantize",
                   "moe_oracle_forward_mxfp8", "moe_oracle_forward_mxfp8_sampled", "moe_oracle_route_grouped",
                   "moe_oracle_forward_sampled_grouped"):
            getattr(self.lib, fn).restype = ctypes.c_int
        self.lib.moe_oracle_e4m3_decode.restype = ctypes.c_float
        self.lib.moe_oracle_e4m3_decode.argtypes = [ctypes.c_uint8]
        for fn in ("moe_oracle_exp_fixed", "moe_oracle_sigmoid_fixed"):
            getattr(self.lib, fn).restype = ctypes.c_float
            getattr(self.lib, fn).argtypes = [ctypes.c_float]
        self.lib.moe_oracle_route_grouped.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int,
                                                      ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_float,
                                                      ctypes.c_void_p, ctypes.c_void_p]
        self.lib.moe_oracle_e4m3_encode.restype = ctypes.c_uint8
        self.lib.moe_oracle_e4m3_encode.argtypes = [ctypes.c_float]

    # -- helpers ---------------------------------------------------------------------------
    @staticmethod
    def _ptr(a: np.ndarray):
        return ctypes.c_void_p(a.ctypes.data)

    @staticmethod
    def _u16(a) -> np.ndarray:
        a = np.ascontiguousarray(a)
        assert a.dtype == np.uint16, "bf16 data must be passed as its uint16 bit pattern"
        return a

    @staticmethod
    def _check(status: int, what: str):
        if status != 0:
            raise RuntimeError(f"{what} failed with oracle status {status}")

    @property
    def num_threads(self) -> int:
        return int(self.lib.moe_oracle_num_threads())

    # -- entry points ----------------------------------------------------------------------
    def route(self, router_logits: np.ndarray, top_k: int):
        l = np.ascontiguousarray(router_logits, dtype=np.float32)
        T, E = l.shape
        ids = np.empty((T, top_k), np.int32)
        w = np.empty((T, top_k), self.real)
        self._check(self.lib.moe_oracle_route(self._ptr(l), T, E, top_k, self._ptr(ids), self._ptr(w)), "route")
        return ids, w

    def exp_fixed(self, x: float) -> float:
        return float(self.lib.moe_oracle_exp_fixed(ctypes.c_float(x)))

    def sigmoid_fixed(self, x: float) -> float:
        return float(self.lib.moe_oracle_sigmoid_fixed(ctypes.c_float(x)))

    def route_grouped(self, router_logits: np.ndarray, top_k: int, n_group: int, topk_group: int, bias=None,
                      scale: float = 1.0):
        """Grouped sigmoid router: (ids [T,k] in rank order, weights [T,k])."""
        l = np.ascontiguousarray(router_logits, dtype=np.float32)
        T, E = l.shape
        b = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
        assert b is None or b.shape == (E,)
        ids = np.empty((T, top_k), np.int32)
        w = np.empty((T, top_k), self.real)
        self._check(self.lib.moe_oracle_route_grouped(self._ptr(l), None if b is None else self._ptr(b), T, E, top_k,
                                                      n_group, topk_group, ctypes.c_float(scale), self._ptr(ids),
                                                      self._ptr(w)), "route_grouped")
        return ids, w

    def forward_sampled_grouped(self, x, router_logits, experts: dict, I: int, top_k: int, tokens, n_group: int,
                                topk_group: int, bias=None, scale: float = 1.0):
        """forward_sampled with the grouped sigmoid router."""
        x = self._u16(x)
        l = np.ascontiguousarray(router_logits, dtype=np.float32)
        T, H = x.shape
        E = l.shape[1]
        tokens = np.ascontiguousarray(tokens, dtype=np.int32)
        b = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
        p13 = (ctypes.c_void_p * E)()
        p2 = (ctypes.c_void_p * E)()
        keep = []
        for e, (a, c) in experts.items():
            a, c = self._u16(a), self._u16(c)
            assert a.shape == (2 * I, H) and c.shape == (H, I)
            keep.append((a, c))
            p13[e] = a.ctypes.data
            p2[e] = c.ctypes.data
        out = np.empty((len(tokens), H), self.real)
        self._check(self.lib.moe_oracle_forward_sampled_grouped(
            self._ptr(x), self._ptr(l), None if b is None else self._ptr(b), n_group, topk_group, ctypes.c_float(scale),
            p13, p2, T, H, I, E, top_k, self._ptr(tokens), len(tokens), self._ptr(out)), "forward_sampled_grouped")
        return out

    def permute(self, topk_ids: np.ndarray, E: int):
        ids = np.ascontiguousarray(topk_ids, dtype=np.int32)
        T, k = ids.shape
        offsets = np.empty(E + 1, np.int32)
        s2f = np.empty(T * k, np.int32)
        f2s = np.empty(T * k, np.int32)
        self._check(self.lib.moe_oracle_permute(self._ptr(ids), T, k, E, self._ptr(offsets), self._ptr(s2f),
                                                self._ptr(f2s)), "permute")
        return offsets, s2f, f2s

    def expert_ffn(self, x_row, w13_e, w2_e):
        x_row, w13_e, w2_e = self._u16(x_row), self._u16(w13_e), self._u16(w2_e)
        H = x_row.shape[0]
        I = w13_e.shape[0] // 2
        assert w13_e.shape == (2 * I, H) and w2_e.shape == (H, I)
        y = np.empty(H, self.real)
        self._check(self.lib.moe_oracle_expert_ffn(self._ptr(x_row), self._ptr(w13_e), self._ptr(w2_e), H, I,
                                                   self._ptr(y)), "expert_ffn")
        return y

    def forward(self, x, router_logits, w13, w2, top_k: int):
        x, w13, w2 = self._u16(x), self._u16(w13), self._u16(w2)
        l = np.ascontiguousarray(router_logits, dtype=np.float32)
        T, H = x.shape
        E, I2, _ = w13.shape
        I = I2 // 2
        assert w13.shape == (E, 2 * I, H) and w2.shape == (E, H, I) and l.shape == (T, E)
        out = np.empty((T, H), self.real)
        self._check(self.lib.moe_oracle_forward(self._ptr(x), self._ptr(l), self._ptr(w13), self._ptr(w2), T, H, I, E,
                                                top_k, self._ptr(out)), "forward")
        return out

    def forward_sampled(self, x, router_logits, experts: dict, I: int, top_k: int, tokens):
        """Layer output for the listed tokens.  ``experts`` maps expert id -> (w13_e, w2_e) uint16
        arrays; only the experts those tokens route to need to be present."""
        x = self._u16(x)
        l = np.ascontiguousarray(router_logits, dtype=np.float32)
        T, H = x.shape
        E = l.shape[1]
        tokens = np.ascontiguousarray(tokens, dtype=np.int32)
        p13 = (ctypes.c_void_p * E)()
        p2 = (ctypes.c_void_p * E)()
        keep = []
        for e, (a, b) in experts.items():
            a, b = self._u16(a), self._u16(b)
            assert a.shape == (2 * I, H) and b.shape == (H, I)
            keep.append((a, b))
            p13[e] = a.ctypes.data
            p2[e] = b.ctypes.data
        out = np.empty((len(tokens), H), self.real)
        self._check(self.lib.moe_oracle_forward_sampled(self._ptr(x), self._ptr(l), p13, p2, T, H, I, E, top_k,
                                                        self._ptr(tokens), len(tokens), self._ptr(out)),
                    "forward_sampled")
        return out

    def forward_local(self, x, router_logits, w13_local, w2_local, E: int, top_k: int, local_offset: int):
        """Partial layer output of a device that holds experts [local_offset, local_offset + n_local)."""
        x, w13_local, w2_local = self._u16(x), self._u16(w13_local), self._u16(w2_local)
        l = np.ascontiguousarray(router_logits, dtype=np.float32)
        T, H = x.shape
        n_local, I2, _ = w13_local.shape
        I = I2 // 2
        assert l.shape == (T, E) and w2_local.shape == (n_local, H, I)
        out = np.empty((T, H), self.real)
        self._check(self.lib.moe_oracle_forward_local(self._ptr(x), self._ptr(l), self._ptr(w13_local),
                                                      self._ptr(w2_local), T, H, I, E, top_k, local_offset, n_local,
                                                      self._ptr(out)), "forward_local")
        return out

    def permute_local(self, topk_ids: np.ndarray, local_offset: int, n_local: int):
        ids = np.ascontiguousarray(topk_ids, dtype=np.int32)
        T, k = ids.shape
        offsets = np.empty(n_local + 1, np.int32)
        s2f = np.empty(T * k, np.int32)
        f2s = np.empty(T * k, np.int32)
        self._check(self.lib.moe_oracle_permute_local(self._ptr(ids), T, k, local_offset, n_local, self._ptr(offsets),
                                                      self._ptr(s2f), self._ptr(f2s)), "permute_local")
        return offsets, s2f, f2s

    def e4m3_decode(self, code: int) -> float:
        return float(self.lib.moe_oracle_e4m3_decode(int(code) & 0xFF))

    def forward_fp8w(self, x, router_logits, w13_q, w13_scale, w2_q, w2_scale, top_k: int):
        """The layer with FP8 (E4M3) weights and one fp32 scale per 128 x 128 block."""
        x = self._u16(x)
        l = np.ascontiguousarray(router_logits, dtype=np.float32)
        w13_q = np.ascontiguousarray(w13_q, dtype=np.uint8)
        w2_q = np.ascontiguousarray(w2_q, dtype=np.uint8)
        w13_scale = np.ascontiguousarray(w13_scale, dtype=np.float32)
        w2_scale = np.ascontiguousarray(w2_scale, dtype=np.float32)
        T, H = x.shape
        E, I2, _ = w13_q.shape
        I = I2 // 2
        assert w13_q.shape == (E, 2 * I, H) and w2_q.shape == (E, H, I) and l.shape == (T, E)
        assert w13_scale.shape == (E, 2 * I // 128, H // 128) and w2_scale.shape == (E, H // 128, I // 128)
        out = np.empty((T, H), self.real)
        self._check(self.lib.moe_oracle_forward_fp8w(self._ptr(x), self._ptr(l), self._ptr(w13_q), self._ptr(w13_scale),
                                                     self._ptr(w2_q), self._ptr(w2_scale), T, H, I, E, top_k,
                                                     self._ptr(out)), "forward_fp8w")
        return out

    def e4m3_encode(self, value: float) -> int:
        return int(self.lib.moe_oracle_e4m3_encode(ctypes.c_float(value)))

    def mx_quantize(self, values: np.ndarray):
        """Rows of fp32 values [R,K] -> (E4M3 codes [R,K], E8M0 scale bytes [R,K/32]), blocks of 32 along K."""
        v = np.ascontiguousarray(values, dtype=np.float32)
        R, K = v.shape
        codes = np.empty((R, K), np.uint8)
        scales = np.empty((R, K // 32), np.uint8)
        self._check(self.lib.moe_oracle_mx_quantize(self._ptr(v), R, K, self._ptr(codes), self._ptr(scales)), "mx_quantize")
        return codes, scales

    def forward_mxfp8(self, x, router_logits, w13_q, w13_s, w2_q, w2_s, top_k: int, intermediates: bool = False):
        """The layer in MX FP8 (E4M3 codes, one E8M0 scale byte per 32 elements along the contraction).
        With ``intermediates`` also returns, per flat assignment t*k+j, h before quantisation [A,I] and its
        quantised codes [A,I] and scale bytes [A,I/32]."""
        x = self._u16(x)
        l = np.ascontiguousarray(router_logits, dtype=np.float32)
        w13_q, w13_s = np.ascontiguousarray(w13_q, dtype=np.uint8), np.ascontiguousarray(w13_s, dtype=np.uint8)
        w2_q, w2_s = np.ascontiguousarray(w2_q, dtype=np.uint8), np.ascontiguousarray(w2_s, dtype=np.uint8)
        T, H = x.shape
        E, I2, _ = w13_q.shape
        I = I2 // 2
        assert w13_q.shape == (E, 2 * I, H) and w2_q.shape == (E, H, I) and l.shape == (T, E)
        assert w13_s.shape == (E, 2 * I, H // 32) and w2_s.shape == (E, H, I // 32)
        out = np.empty((T, H), self.real)
        A = T * top_k
        h_pre = np.empty((A, I), self.real) if intermediates else None
        h_q = np.empty((A, I), np.uint8) if intermediates else None
        h_s = np.empty((A, I // 32), np.uint8) if intermediates else None
        opt = lambda a: self._ptr(a) if a is not None else None
        self._check(self.lib.moe_oracle_forward_mxfp8(self._ptr(x), self._ptr(l), self._ptr(w13_q), self._ptr(w13_s),
                                                      self._ptr(w2_q), self._ptr(w2_s), T, H, I, E, top_k,
                                                      self._ptr(out), opt(h_pre), opt(h_q), opt(h_s)), "forward_mxfp8")
        return (out, h_pre, h_q, h_s) if intermediates else out

    def forward_mxfp8_sampled(self, x, router_logits, experts: dict, I: int, top_k: int, tokens):
        """The MX FP8 layer for the listed tokens.  ``experts`` maps expert id -> (w13_q [2I,H], w13_s [2I,H/32],
        w2_q [H,I], w2_s [H,I/32]) uint8 arrays; only the experts those tokens route to need to be present."""
        x = self._u16(x)
        l = np.ascontiguousarray(router_logits, dtype=np.float32)
        T, H = x.shape
        E = l.shape[1]
        tokens = np.ascontiguousarray(tokens, dtype=np.int32)
        tabs = [(ctypes.c_void_p * E)() for _ in range(4)]
        keep = []
        for e, arrays in experts.items():
            arrays = [np.ascontiguousarray(a, dtype=np.uint8) for a in arrays]
            assert arrays[0].shape == (2 * I, H) and arrays[1].shape == (2 * I, H // 32)
            assert arrays[2].shape == (H, I) and arrays[3].shape == (H, I // 32)
            keep.append(arrays)
            for tab, a in zip(tabs, arrays):
                tab[e] = a.ctypes.data
        out = np.empty((len(tokens), H), self.real)
        self._check(self.lib.moe_oracle_forward_mxfp8_sampled(self._ptr(x), self._ptr(l), *tabs, T, H, I, E, top_k,
                                                              self._ptr(tokens), len(tokens), self._ptr(out)),
                    "forward_mxfp8_sampled")
        return out

    def sorted_intermediates(self, x, w13, w2, topk_ids, sorted_to_flat):
        x, w13, w2 = self._u16(x), self._u16(w13), self._u16(w2)
        ids = np.ascontiguousarray(topk_ids, dtype=np.int32)
        s2f = np.ascontiguousarray(sorted_to_flat, dtype=np.int32)
        T, H = x.shape
        E, I2, _ = w13.shape
        I = I2 // 2
        k = ids.shape[1]
        h = np.empty((T * k, I), self.real)
        y = np.empty((T * k, H), self.real)
        self._check(self.lib.moe_oracle_sorted_intermediates(self._ptr(x), self._ptr(w13), self._ptr(w2),
                                                             self._ptr(ids), self._ptr(s2f), T, H, I, E, k,
                                                             self._ptr(h), self._ptr(y)), "sorted_intermediates")
        return h, y


_cache: dict[str, Oracle] = {}


def get(precision: str = "f32") -> Oracle:
    if precision not in _cache:
        _cache[precision] = Oracle(precision)
    return _cache[precision]
