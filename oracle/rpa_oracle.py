"""ctypes front end of the fp64 CPU oracle (``rpa_oracle.c``).

TEST INFRASTRUCTURE ONLY.  Only the tests, the smoke check and the benchmark's CPU-baseline leg
may import this module.  It marshals numpy arrays into the C checker and holds no arithmetic of
the method itself: the definition lives in ``rpa_oracle.c`` (the paper's problem statement,
Section 2.4 and Section 3; Algorithm 1's result in closed form).

All tensors are numpy arrays; bf16 values travel as their uint16 bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rpa_oracle.c")
_LIB = os.path.join(_HERE, "librpa_oracle.so")


def build(force: bool = False) -> str:
    """Compile the C checker with gcc (OpenMP) next to its source; returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


class _Shape(ctypes.Structure):
    _fields_ = [
        ("num_q_heads", ctypes.c_int32),
        ("num_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32),
        ("page_size", ctypes.c_int32),
        ("num_pages", ctypes.c_int32),
        ("max_pages_per_seq", ctypes.c_int32),
        ("causal", ctypes.c_int32),
        ("scale", ctypes.c_double),
        ("kv_fp8", ctypes.c_int32),
        ("k_scale", ctypes.c_float),
        ("v_scale", ctypes.c_float),
        ("q_scale", ctypes.c_float),
    ]


@dataclass(frozen=True)
class OracleShape:
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    page_size: int
    num_pages: int
    max_pages_per_seq: int
    scale: float
    causal: bool = True
    kv_fp8: bool = False  # FP8 E4M3 cache (uint8 codes) with per-tensor scales
    k_scale: float = 1.0
    v_scale: float = 1.0
    q_scale: float = 0.0  # > 0: Q is taken in E4M3 precision with this per-tensor scale (FP8 cache only)

    def _c(self) -> _Shape:
        return _Shape(self.num_q_heads, self.num_kv_heads, self.head_dim, self.page_size, self.num_pages,
                      self.max_pages_per_seq, 1 if self.causal else 0, float(self.scale), 1 if self.kv_fp8 else 0,
                      float(self.k_scale), float(self.v_scale), float(self.q_scale))

    @property
    def cache_dtype(self):
        return np.uint8 if self.kv_fp8 else np.uint16


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64
        sp = ctypes.POINTER(_Shape)
        lib.rpa_oracle_threads.restype = ctypes.c_int
        lib.rpa_oracle_update_cache.argtypes = [sp, vp, vp, vp, vp, vp, vp, i32]
        lib.rpa_oracle_attend_rows.argtypes = [sp, vp, vp, vp, vp, vp, i32, vp, i64, vp]
        lib.rpa_oracle_forward.argtypes = [sp, vp, vp, vp, vp, vp, vp, vp, i32, vp]
        lib.rpa_oracle_e4m3_to_double.argtypes = [ctypes.c_uint8]
        lib.rpa_oracle_e4m3_to_double.restype = ctypes.c_double
        lib.rpa_oracle_float_to_e4m3.argtypes = [ctypes.c_float]
        lib.rpa_oracle_float_to_e4m3.restype = ctypes.c_uint8
        _lib = lib
    return _lib


def threads() -> int:
    """OpenMP threads the checker will use."""
    return int(_load().rpa_oracle_threads())


def _arr(x, dtype, name):
    a = np.ascontiguousarray(x)
    if a.dtype != dtype:
        raise TypeError(f"{name}: expected {dtype}, got {a.dtype}")
    return a


def _ptr(a):
    return ctypes.c_void_p(a.ctypes.data)


def _check(rc, what):
    if rc != 0:
        raise ValueError(f"{what}: oracle rejected the inputs (code {rc})")


def e4m3_to_double(code: int) -> float:
    return float(_load().rpa_oracle_e4m3_to_double(int(code) & 0xFF))


def float_to_e4m3(x: float) -> int:
    return int(_load().rpa_oracle_float_to_e4m3(float(np.float32(x))))


def update_cache(shape: OracleShape, new_k, new_v, kv_cache, page_table, cu_q_lens, kv_lens) -> None:
    """Step 1 only, in place on ``kv_cache`` (uint16 bf16 bits, or uint8 E4M3 codes for an FP8 cache;
    [num_pages, page_size, 2*h_kv, d])."""
    new_k, new_v = _arr(new_k, np.uint16, "new_k"), _arr(new_v, np.uint16, "new_v")
    if kv_cache.dtype != shape.cache_dtype or not kv_cache.flags.c_contiguous:
        raise TypeError(f"kv_cache must be a contiguous {shape.cache_dtype.__name__} array (it is updated in place)")
    pt, cu, kl = _arr(page_table, np.int32, "page_table"), _arr(cu_q_lens, np.int32, "cu_q_lens"), _arr(kv_lens, np.int32, "kv_lens")
    sh = shape._c()
    _check(_load().rpa_oracle_update_cache(ctypes.byref(sh), _ptr(new_k), _ptr(new_v), _ptr(kv_cache), _ptr(pt),
                                           _ptr(cu), _ptr(kl), len(kl)), "update_cache")


def attend_rows(shape: OracleShape, q, kv_cache, page_table, cu_q_lens, kv_lens, rows) -> np.ndarray:
    """Step 2 for the listed (sequence, token-in-sequence, query head) triples on an updated cache.

    Returns float64 [len(rows), d]."""
    q = _arr(q, np.uint16, "q")
    kv_cache = _arr(kv_cache, shape.cache_dtype, "kv_cache")
    pt, cu, kl = _arr(page_table, np.int32, "page_table"), _arr(cu_q_lens, np.int32, "cu_q_lens"), _arr(kv_lens, np.int32, "kv_lens")
    rows = _arr(np.asarray(rows, dtype=np.int32).reshape(-1, 3), np.int32, "rows")
    out = np.zeros((rows.shape[0], shape.head_dim), dtype=np.float64)
    sh = shape._c()
    _check(_load().rpa_oracle_attend_rows(ctypes.byref(sh), _ptr(q), _ptr(kv_cache), _ptr(pt), _ptr(cu), _ptr(kl),
                                          len(kl), _ptr(rows), rows.shape[0], _ptr(out)), "attend_rows")
    return out


def forward(shape: OracleShape, q, new_k, new_v, kv_cache, page_table, cu_q_lens, kv_lens) -> np.ndarray:
    """The whole call: cache update in place on ``kv_cache``, then attention for every token and head.

    Returns float64 [T, h_q, d] with T = cu_q_lens[-1]."""
    q = _arr(q, np.uint16, "q")
    new_k, new_v = _arr(new_k, np.uint16, "new_k"), _arr(new_v, np.uint16, "new_v")
    if kv_cache.dtype != shape.cache_dtype or not kv_cache.flags.c_contiguous:
        raise TypeError(f"kv_cache must be a contiguous {shape.cache_dtype.__name__} array (it is updated in place)")
    pt, cu, kl = _arr(page_table, np.int32, "page_table"), _arr(cu_q_lens, np.int32, "cu_q_lens"), _arr(kv_lens, np.int32, "kv_lens")
    T = int(cu[-1])
    out = np.zeros((T, shape.num_q_heads, shape.head_dim), dtype=np.float64)
    sh = shape._c()
    _check(_load().rpa_oracle_forward(ctypes.byref(sh), _ptr(q), _ptr(new_k), _ptr(new_v), _ptr(kv_cache), _ptr(pt),
                                      _ptr(cu), _ptr(kl), len(kl), _ptr(out)), "forward")
    return out
