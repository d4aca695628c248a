"""Thin ctypes binding of ``librpa_b200.so`` (see ``include/rpa.h``).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.  There is no
fallback -- if the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "librpa_b200.so")

RPA_OK = 0
STATUS_NAMES = {0: "RPA_OK", 1: "RPA_ERR_INVALID_ARG", 2: "RPA_ERR_UNSUPPORTED", 3: "RPA_ERR_CAPACITY",
                4: "RPA_ERR_PLAN_MISMATCH", 5: "RPA_ERR_CUDA", 6: "RPA_ERR_TIMEOUT"}
CASE_NAMES = {0: "empty", 1: "decode", 2: "prefill", 3: "mixed"}
ABLATE_UPDATE = 1
ABLATE_OVERLAP = 2

EXPORTS = ["rpa_create", "rpa_destroy", "rpa_plan", "rpa_forward", "rpa_forward_host", "rpa_forward_host_submit",
           "rpa_forward_host_wait", "rpa_plan_info",
           "rpa_plan_dump", "rpa_poll_status", "rpa_set_ablation", "rpa_set_kv_chunk", "rpa_set_kernel_timing",
           "rpa_get_kernel_timing", "rpa_forward_static", "rpa_set_tile_min_q", "rpa_set_tile_pair", "rpa_selftest_bounded_wait", "rpa_set_validation", "rpa_plan_device", "rpa_plan_device_dump",
           "rpa_status_string",
           "rpa_last_cuda_error"]


class RpaError(RuntimeError):
    def __init__(self, status: int, what: str, detail: str = ""):
        self.status = status
        super().__init__(f"{what}: {STATUS_NAMES.get(status, status)}" + (f" ({detail})" if detail else ""))


class rpa_config_t(ctypes.Structure):
    _fields_ = [("num_q_heads", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("page_size", ctypes.c_int32), ("num_pages", ctypes.c_int32), ("max_pages_per_seq", ctypes.c_int32),
                ("max_num_seqs", ctypes.c_int32), ("max_num_tokens", ctypes.c_int32), ("sm_scale", ctypes.c_float),
                ("causal", ctypes.c_int32), ("kv_dtype", ctypes.c_int32), ("k_scale", ctypes.c_float),
                ("v_scale", ctypes.c_float), ("q_scale", ctypes.c_float)]


class rpa_plan_info_t(ctypes.Structure):
    _fields_ = [("batch_case", ctypes.c_int32), ("num_seqs", ctypes.c_int32), ("num_tokens", ctypes.c_int32),
                ("num_decode_seqs", ctypes.c_int32), ("num_prefill_seqs", ctypes.c_int32),
                ("num_row_items", ctypes.c_int32), ("num_tile_items", ctypes.c_int32),
                ("num_combine_groups", ctypes.c_int32), ("kv_chunk_tokens", ctypes.c_int32),
                ("gpu_launches", ctypes.c_int32), ("algorithmic_bytes", ctypes.c_int64),
                ("algorithmic_flops", ctypes.c_int64), ("workspace_bytes", ctypes.c_int64),
                ("row_bytes", ctypes.c_int64), ("tile_flops", ctypes.c_int64), ("tile_kernel", ctypes.c_int32),
                ("tile_short_items", ctypes.c_int32)]

    def as_dict(self) -> dict:
        return {k: getattr(self, k) for k, _ in self._fields_}


_lib = None


def load_library(path: Optional[str] = None) -> ctypes.CDLL:
    """Load the CUDA library; raises if it has not been built (``python -m paper_2604_15464_b200.build``)."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise FileNotFoundError(f"{p} not found: build it with paper_2604_15464_b200.build.build(); there is no fallback")
    lib = ctypes.CDLL(p)
    vp, i32 = ctypes.c_void_p, ctypes.c_int32
    lib.rpa_create.argtypes = [ctypes.POINTER(rpa_config_t), ctypes.c_int, ctypes.POINTER(vp)]
    lib.rpa_destroy.argtypes = [vp]
    lib.rpa_destroy.restype = None
    lib.rpa_plan.argtypes = [vp, vp, vp, i32, vp]
    lib.rpa_forward.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, vp, vp]
    lib.rpa_forward_host.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, vp, vp]
    lib.rpa_forward_host_submit.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, vp, vp]
    lib.rpa_forward_host_wait.argtypes = [vp]
    lib.rpa_plan_info.argtypes = [vp, ctypes.POINTER(rpa_plan_info_t)]
    lib.rpa_plan_dump.argtypes = [vp, vp, i32, vp, i32, vp, i32]
    lib.rpa_poll_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_uint32)]
    lib.rpa_set_ablation.argtypes = [vp, ctypes.c_uint32]
    lib.rpa_set_kv_chunk.argtypes = [vp, i32]
    lib.rpa_set_tile_min_q.argtypes = [vp, i32]
    lib.rpa_set_tile_pair.argtypes = [vp, i32]
    lib.rpa_selftest_bounded_wait.argtypes = [vp, vp]
    lib.rpa_set_validation.argtypes = [vp, i32]
    lib.rpa_plan_device.argtypes = [vp, vp, vp, i32, vp]
    lib.rpa_plan_device_dump.argtypes = [vp, vp, vp, i32, vp, i32, vp, i32]
    lib.rpa_set_kernel_timing.argtypes = [vp, i32]
    lib.rpa_get_kernel_timing.argtypes = [vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(i32)]
    lib.rpa_forward_static.argtypes = [ctypes.POINTER(rpa_config_t), vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, vp, vp]
    lib.rpa_status_string.argtypes = [ctypes.c_int]
    lib.rpa_status_string.restype = ctypes.c_char_p
    lib.rpa_last_cuda_error.argtypes = [vp]
    lib.rpa_last_cuda_error.restype = ctypes.c_char_p
    if path is None:
        _lib = lib
    return lib


@dataclass
class RpaConfig:
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    page_size: int
    num_pages: int
    max_pages_per_seq: int
    max_num_seqs: int
    max_num_tokens: int
    sm_scale: float = 0.0
    causal: bool = True
    kv_fp8: bool = False  # FP8 E4M3 cache with per-tensor scales
    k_scale: float = 1.0
    v_scale: float = 1.0
    q_scale: float = 0.0  # > 0: Q is quantised to E4M3 with this per-tensor scale as well (FP8 cache only)

    def _c(self) -> rpa_config_t:
        return rpa_config_t(self.num_q_heads, self.num_kv_heads, self.head_dim, self.page_size, self.num_pages,
                            self.max_pages_per_seq, self.max_num_seqs, self.max_num_tokens, self.sm_scale,
                            1 if self.causal else 0, 1 if self.kv_fp8 else 0, self.k_scale, self.v_scale, self.q_scale)


def _dev_ptr(t) -> int:
    return 0 if t is None else int(t.data_ptr())


def _host_i32(x) -> np.ndarray:
    a = np.ascontiguousarray(np.asarray(x), dtype=np.int32)
    return a


def rpa_forward_static(config: RpaConfig, q, new_k, new_v, kv_cache, page_table, cu_q_lens, kv_lens,
                       cu_q_lens_host, kv_lens_host, out, stream: int = 0) -> None:
    """The handle-free entry point for callers that cannot allocate device memory: plans on the host
    and runs on the current device out of the library's built-in scratch.  Tensor arguments are
    device tensors as for ``Rpa.rpa_forward``; the two ``*_host`` arguments are host int32 arrays."""
    lib = load_library()
    cu, kl = _host_i32(cu_q_lens_host), _host_i32(kv_lens_host)
    if len(cu) != len(kl) + 1:
        raise ValueError("cu_q_lens_host must have num_seqs + 1 entries")
    cfg = config._c()
    st = lib.rpa_forward_static(ctypes.byref(cfg), _dev_ptr(q), _dev_ptr(new_k), _dev_ptr(new_v), _dev_ptr(kv_cache),
                                _dev_ptr(page_table), _dev_ptr(cu_q_lens), _dev_ptr(kv_lens), cu.ctypes.data,
                                kl.ctypes.data, len(kl), _dev_ptr(out), stream)
    if st != RPA_OK:
        raise RpaError(st, "rpa_forward_static")


class Rpa:
    """One library handle.  ``device`` < 0 gives a planning-only handle that makes no CUDA call."""

    def __init__(self, config: RpaConfig, device: int = 0, library_path: Optional[str] = None):
        # library_path: another build of the same library (the bounds-checked one, say)
        self._lib = load_library(library_path)
        self.config = config
        self.device = device
        self._h = ctypes.c_void_p()
        cfg = config._c()
        st = self._lib.rpa_create(ctypes.byref(cfg), device, ctypes.byref(self._h))
        if st != RPA_OK:
            raise RpaError(st, "rpa_create")

    @classmethod
    def for_meta(cls, meta, device: int = 0, **over) -> "Rpa":
        """Handle sized for a ``workloads.BatchMeta``."""
        cfg = RpaConfig(meta.num_q_heads, meta.num_kv_heads, meta.head_dim, meta.page_size, meta.num_pages,
                        meta.max_pages_per_seq, max(meta.num_seqs, 1), max(meta.token_capacity, 1), meta.scale,
                        meta.causal, meta.kv_fp8, meta.k_scale, meta.v_scale, getattr(meta, "q_scale", 0.0))
        library_path = over.pop("library_path", None)
        for k, v in over.items():
            setattr(cfg, k, v)
        return cls(cfg, device, library_path)

    def close(self) -> None:
        if getattr(self, "_h", None) and self._h.value:
            self._lib.rpa_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int, what: str) -> None:
        if st != RPA_OK:
            detail = self._lib.rpa_last_cuda_error(self._h).decode() if st == 5 else ""
            raise RpaError(st, what, detail)

    # -- the C-ABI calls, same names ------------------------------------------------------------
    def rpa_plan(self, cu_q_lens_host, kv_lens_host, stream: int = 0) -> None:
        cu, kl = _host_i32(cu_q_lens_host), _host_i32(kv_lens_host)
        if len(cu) != len(kl) + 1:
            raise ValueError("cu_q_lens must have num_seqs + 1 entries")
        self._num_seqs = len(kl)
        self._check(self._lib.rpa_plan(self._h, cu.ctypes.data, kl.ctypes.data, len(kl), stream), "rpa_plan")

    def rpa_plan_device(self, cu_q_lens, kv_lens, stream: int = 0, num_seqs: Optional[int] = None) -> None:
        """Plan on the device from the device copies of the lengths (int32 CUDA tensors)."""
        n = int(kv_lens.shape[0]) if num_seqs is None else num_seqs
        self._num_seqs = n
        self._check(self._lib.rpa_plan_device(self._h, _dev_ptr(cu_q_lens), _dev_ptr(kv_lens), n, stream), "rpa_plan_device")

    def rpa_plan_device_dump(self, row_capacity: int, tile_capacity: int, group_capacity: int):
        """(counts [8], row_items, tile_items, combine_groups) of the device-made plan; waits for the device."""
        counts = np.zeros(8, np.int32)
        rows = np.zeros((row_capacity, 8), np.int32)
        tiles = np.zeros((tile_capacity, 8), np.int32)
        groups = np.zeros((group_capacity, 8), np.int32)
        self._check(self._lib.rpa_plan_device_dump(self._h, counts.ctypes.data, rows.ctypes.data, row_capacity,
                                                   tiles.ctypes.data, tile_capacity, groups.ctypes.data, group_capacity),
                    "rpa_plan_device_dump")
        return counts, rows[: counts[0]], tiles[: counts[1]], groups[: counts[2]]

    def rpa_forward(self, q, new_k, new_v, kv_cache, page_table, cu_q_lens, kv_lens, out, stream: int = 0,
                    num_seqs: Optional[int] = None) -> None:
        n = int(kv_lens.shape[0]) if num_seqs is None else num_seqs
        self._check(self._lib.rpa_forward(self._h, _dev_ptr(q), _dev_ptr(new_k), _dev_ptr(new_v), _dev_ptr(kv_cache),
                                          _dev_ptr(page_table), _dev_ptr(cu_q_lens), _dev_ptr(kv_lens), n,
                                          _dev_ptr(out), stream), "rpa_forward")

    def rpa_forward_host(self, q_host, new_k_host, new_v_host, kv_cache, page_table_host, cu_q_lens_host,
                         kv_lens_host, out_host, stream: int = 0) -> None:
        """Host tensors (torch CPU, ideally pinned) for everything but the device-resident cache."""
        n = int(kv_lens_host.shape[0])
        self._check(self._lib.rpa_forward_host(self._h, _dev_ptr(q_host), _dev_ptr(new_k_host), _dev_ptr(new_v_host),
                                               _dev_ptr(kv_cache), _dev_ptr(page_table_host),
                                               _dev_ptr(cu_q_lens_host), _dev_ptr(kv_lens_host), n,
                                               _dev_ptr(out_host), stream), "rpa_forward_host")

    def rpa_forward_host_submit(self, q_host, new_k_host, new_v_host, kv_cache, page_table_host, cu_q_lens_host,
                                kv_lens_host, out_host, stream: int = 0) -> None:
        """rpa_forward_host without the wait: the step's copies overlap its neighbours' kernels."""
        n = int(kv_lens_host.shape[0])
        self._check(self._lib.rpa_forward_host_submit(self._h, _dev_ptr(q_host), _dev_ptr(new_k_host),
                                                      _dev_ptr(new_v_host), _dev_ptr(kv_cache),
                                                      _dev_ptr(page_table_host), _dev_ptr(cu_q_lens_host),
                                                      _dev_ptr(kv_lens_host), n, _dev_ptr(out_host), stream),
                    "rpa_forward_host_submit")

    def rpa_forward_host_wait(self) -> None:
        """Blocks until the oldest outstanding submitted step has delivered its output."""
        self._check(self._lib.rpa_forward_host_wait(self._h), "rpa_forward_host_wait")

    def rpa_plan_info(self) -> dict:
        info = rpa_plan_info_t()
        self._check(self._lib.rpa_plan_info(self._h, ctypes.byref(info)), "rpa_plan_info")
        d = info.as_dict()
        d["batch_case_name"] = CASE_NAMES.get(d["batch_case"], "?")
        return d

    def rpa_plan_dump(self):
        """(row_items [R,8], tile_items [Tl,8], combine_groups [G,8]) as int32 arrays."""
        info = self.rpa_plan_info()
        rows = np.zeros((info["num_row_items"], 8), np.int32)
        tiles = np.zeros((info["num_tile_items"], 8), np.int32)
        groups = np.zeros((info["num_combine_groups"], 8), np.int32)
        self._check(self._lib.rpa_plan_dump(self._h, rows.ctypes.data, len(rows), tiles.ctypes.data, len(tiles),
                                            groups.ctypes.data, len(groups)), "rpa_plan_dump")
        return rows, tiles, groups

    def rpa_poll_status(self, stream: int = 0) -> int:
        word = ctypes.c_uint32()
        st = self._lib.rpa_poll_status(self._h, stream, ctypes.byref(word))
        if st not in (0, 6, 1):
            self._check(st, "rpa_poll_status")
        return int(word.value)

    def rpa_selftest_bounded_wait(self, stream: int = 0) -> None:
        self._check(self._lib.rpa_selftest_bounded_wait(self._h, stream), "rpa_selftest_bounded_wait")

    def rpa_set_validation(self, enable: bool) -> None:
        self._check(self._lib.rpa_set_validation(self._h, 1 if enable else 0), "rpa_set_validation")

    def rpa_set_ablation(self, mask: int) -> None:
        self._check(self._lib.rpa_set_ablation(self._h, mask), "rpa_set_ablation")

    def rpa_set_kv_chunk(self, tokens: int) -> None:
        self._check(self._lib.rpa_set_kv_chunk(self._h, tokens), "rpa_set_kv_chunk")

    def rpa_set_tile_min_q(self, tokens: int) -> None:
        self._check(self._lib.rpa_set_tile_min_q(self._h, tokens), "rpa_set_tile_min_q")

    def rpa_set_tile_pair(self, mode: int) -> None:
        self._check(self._lib.rpa_set_tile_pair(self._h, mode), "rpa_set_tile_pair")

    def rpa_set_kernel_timing(self, enable: bool) -> None:
        self._check(self._lib.rpa_set_kernel_timing(self._h, 1 if enable else 0), "rpa_set_kernel_timing")

    def rpa_get_kernel_timing(self) -> dict:
        """{"row" | "tile" | "combine": (total_ms, launches)} for the launches recorded since enabling."""
        ms = (ctypes.c_float * 3)()
        n = (ctypes.c_int32 * 3)()
        self._check(self._lib.rpa_get_kernel_timing(self._h, ms, n), "rpa_get_kernel_timing")
        return {name: (float(ms[i]), int(n[i])) for i, name in enumerate(("row", "tile", "combine"))}

    # -- convenience ----------------------------------------------------------------------------
    def run_batch(self, batch, out=None, stream: int = 0):
        """plan + forward on a ``workloads.Batch``; returns ``out`` (bf16 [token_capacity, h_q, d])."""
        import torch

        if out is None:
            out = torch.zeros_like(batch.q)
        self.rpa_plan(batch.meta.cu_q_lens, batch.meta.kv_lens, stream)
        self.rpa_forward(batch.q, batch.new_k, batch.new_v, batch.kv_cache, batch.page_table, batch.cu_q_lens,
                         batch.kv_lens, out, stream)
        return out
