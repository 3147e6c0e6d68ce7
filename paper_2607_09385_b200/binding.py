"""ctypes binding of the C ABI in ``include/steel_attn.h`` (argument marshalling only).

Every function here has the name and meaning of its C counterpart; tensors are passed as raw
device pointers taken from torch tensors (host pointers for the ``steel_attn_host_*`` calls), the
stream as ``torch.cuda.current_stream()``.
There is no fallback: if the shared library is missing and cannot be built, importing the
binding's functions raises.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

from . import build as _build

STEEL_OK, STEEL_ERR_INVALID_ARG, STEEL_ERR_UNSUPPORTED = 0, 1, 2
STEEL_ERR_ALLOC, STEEL_ERR_CUDA, STEEL_ERR_TIMEOUT = 3, 4, 5
STEEL_MASK_CAUSAL, STEEL_MASK_WINDOW, STEEL_MASK_BITMAP = 1, 2, 4

EXPORTS = (
    "steel_attn_create", "steel_attn_run", "steel_attn_last_status", "steel_attn_destroy",
    "steel_attn_get_stats", "steel_attn_plan_host", "steel_attn_run_noalloc",
    "steel_attn_debug_stall", "steel_attn_debug_clock_probe",
    "steel_attn_host_create", "steel_attn_host_run", "steel_attn_host_last_status", "steel_attn_host_chunks",
    "steel_attn_host_destroy",
    "steel_status_string",
)


class MaskDesc(ctypes.Structure):
    _fields_ = [("flags", ctypes.c_uint32), ("block_q", ctypes.c_int32), ("block_kv", ctypes.c_int32),
                ("window", ctypes.c_int64), ("bitmap", ctypes.c_void_p)]


class Params(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("heads_q", ctypes.c_int32), ("heads_kv", ctypes.c_int32),
                ("seq_q", ctypes.c_int32), ("seq_kv", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("scale", ctypes.c_float), ("mask", MaskDesc), ("policy", ctypes.c_int32),
                ("exp_emulation", ctypes.c_int32)]


class Stats(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in (
        "kept_tiles", "partial_tiles", "total_tiles", "exec_tiles", "exec_partial", "work_items",
        "steps", "kv_tile_loads", "list_entries", "max_cta_steps", "grid")] + [
        ("effective_flop", ctypes.c_double), ("useful_flop", ctypes.c_double)]

    def as_dict(self) -> dict:
        return {n: getattr(self, n) for n, _ in self._fields_}


class SteelError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {steel_status_string(status)} (status {status})")


_lib = None


def library_path() -> str:
    return _build.LIB_PATH


def load_library():
    """Load libsteel_attn.so (building it with nvcc first if it is missing or stale)."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB_PATH
    if os.environ.get("STEEL_ATTN_NO_BUILD") != "1":
        try:
            path = _build.build_library()
        except Exception as exc:  # stale library with no compiler: use what is there
            if not os.path.exists(_build.LIB_PATH):
                raise RuntimeError(f"libsteel_attn.so is missing and could not be built: {exc}") from exc
    if not os.path.exists(path):
        raise RuntimeError("libsteel_attn.so is missing: run paper_2607_09385_b200.build.build_library()")
    lib = ctypes.CDLL(path)
    vp = ctypes.c_void_p
    lib.steel_attn_create.argtypes = [ctypes.POINTER(Params), ctypes.POINTER(vp)]
    lib.steel_attn_run.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    lib.steel_attn_last_status.argtypes = [vp, vp]
    lib.steel_attn_destroy.argtypes = [vp]
    lib.steel_attn_get_stats.argtypes = [vp, ctypes.POINTER(Stats)]
    lib.steel_attn_plan_host.argtypes = [ctypes.POINTER(Params), ctypes.POINTER(Stats), vp, ctypes.c_int64,
                                         ctypes.POINTER(ctypes.c_int64)]
    lib.steel_attn_debug_stall.argtypes = [vp, ctypes.c_int32, ctypes.c_int64]
    lib.steel_attn_debug_clock_probe.argtypes = [vp, vp]
    lib.steel_attn_run_noalloc.argtypes = [ctypes.POINTER(Params), vp, vp, vp, vp, vp, vp]
    lib.steel_attn_host_create.argtypes = [ctypes.POINTER(Params), ctypes.c_int32, ctypes.POINTER(vp)]
    lib.steel_attn_host_run.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    lib.steel_attn_host_last_status.argtypes = [vp, vp]
    lib.steel_attn_host_chunks.argtypes = [vp]
    lib.steel_attn_host_destroy.argtypes = [vp]
    lib.steel_status_string.argtypes = [ctypes.c_int]
    lib.steel_status_string.restype = ctypes.c_char_p
    for name in EXPORTS[:-1]:
        getattr(lib, name).restype = ctypes.c_int
    _lib = lib
    return lib


def make_params(batch, heads_q, heads_kv, seq_q, seq_kv, head_dim, scale, flags=0, block_q=128,
                block_kv=128, window=0, bitmap=None, policy=0, exp_emulation=0):
    """Build a ``steel_attn_params_t``; returns (params, keepalive) where keepalive holds the
    host bitmap array the descriptor points to."""
    keep = None
    ptr = None
    if bitmap is not None:
        keep = np.ascontiguousarray(bitmap, dtype=np.uint32)
        ptr = keep.ctypes.data
    mask = MaskDesc(flags, block_q, block_kv, window, ptr)
    return Params(batch, heads_q, heads_kv, seq_q, seq_kv, head_dim, scale, mask, policy, exp_emulation), keep


def steel_status_string(status: int) -> str:
    return load_library().steel_status_string(int(status)).decode()


def steel_attn_create(params: Params) -> int:
    handle = ctypes.c_void_p()
    st = load_library().steel_attn_create(ctypes.byref(params), ctypes.byref(handle))
    if st != STEEL_OK:
        raise SteelError(st, "steel_attn_create")
    return handle.value


def steel_attn_run(handle: int, q_ptr: int, k_ptr: int, v_ptr: int, o_ptr: int, lse_ptr, stream: int) -> None:
    st = load_library().steel_attn_run(handle, q_ptr, k_ptr, v_ptr, o_ptr, lse_ptr, stream)
    if st != STEEL_OK:
        raise SteelError(st, "steel_attn_run")


def steel_attn_last_status(handle: int, stream: int) -> int:
    return load_library().steel_attn_last_status(handle, stream)


def steel_attn_destroy(handle) -> None:
    st = load_library().steel_attn_destroy(handle)
    if st != STEEL_OK:
        raise SteelError(st, "steel_attn_destroy")


def steel_attn_get_stats(handle: int) -> dict:
    s = Stats()
    st = load_library().steel_attn_get_stats(handle, ctypes.byref(s))
    if st != STEEL_OK:
        raise SteelError(st, "steel_attn_get_stats")
    return s.as_dict()


def steel_attn_plan_host(params: Params, want_tiles: bool = False, capacity: int = 1 << 22):
    """Host-only planning.  Returns (status, stats dict or None, tiles int32 [n, 6] or None)."""
    s = Stats()
    n = ctypes.c_int64(0)
    tiles = np.zeros((capacity, 6), dtype=np.int32) if want_tiles else None
    st = load_library().steel_attn_plan_host(ctypes.byref(params), ctypes.byref(s),
                                             tiles.ctypes.data if want_tiles else None, capacity,
                                             ctypes.byref(n))
    if st != STEEL_OK:
        return st, None, None
    return st, s.as_dict(), (tiles[: n.value].copy() if want_tiles else None)


def steel_attn_run_noalloc(params: Params, q_ptr: int, k_ptr: int, v_ptr: int, o_ptr: int, lse_ptr,
                           stream: int) -> int:
    """The allocation-free call: plans, runs and waits; returns the status code (see the header for
    who needs it, its size limits and why overlapping calls race)."""
    return load_library().steel_attn_run_noalloc(ctypes.byref(params), q_ptr, k_ptr, v_ptr, o_ptr, lse_ptr,
                                                 stream)


def steel_attn_debug_stall(handle: int, cta: int, timeout_cycles: int = 0) -> None:
    st = load_library().steel_attn_debug_stall(handle, cta, timeout_cycles)
    if st != STEEL_OK:
        raise SteelError(st, "steel_attn_debug_stall")


def steel_attn_debug_clock_probe(handle: int, device_pair_ptr) -> None:
    st = load_library().steel_attn_debug_clock_probe(handle, device_pair_ptr)
    if st != STEEL_OK:
        raise SteelError(st, "steel_attn_debug_clock_probe")


def steel_attn_host_create(params: Params, max_chunks: int) -> int:
    handle = ctypes.c_void_p()
    st = load_library().steel_attn_host_create(ctypes.byref(params), max_chunks, ctypes.byref(handle))
    if st != STEEL_OK:
        raise SteelError(st, "steel_attn_host_create")
    return handle.value


def steel_attn_host_run(handle: int, q_ptr: int, k_ptr: int, v_ptr: int, o_ptr: int, lse_ptr, stream: int) -> None:
    """All five pointers are HOST addresses (page-locked memory makes the call asynchronous)."""
    st = load_library().steel_attn_host_run(handle, q_ptr, k_ptr, v_ptr, o_ptr, lse_ptr, stream)
    if st != STEEL_OK:
        raise SteelError(st, "steel_attn_host_run")


def steel_attn_host_last_status(handle: int, stream: int) -> int:
    return load_library().steel_attn_host_last_status(handle, stream)


def steel_attn_host_chunks(handle: int) -> int:
    return load_library().steel_attn_host_chunks(handle)


def steel_attn_host_destroy(handle) -> None:
    st = load_library().steel_attn_host_destroy(handle)
    if st != STEEL_OK:
        raise SteelError(st, "steel_attn_host_destroy")


class SteelAttention:
    """Convenience owner of one handle: ``SteelAttention(...).run(q, k, v)`` on CUDA torch tensors."""

    def __init__(self, batch, heads_q, heads_kv, seq_q, seq_kv, head_dim, scale, flags=0, block=128,
                 window=0, bitmap=None, policy=0, exp_emulation=0):
        self.params, self._keep = make_params(batch, heads_q, heads_kv, seq_q, seq_kv, head_dim, scale,
                                              flags, block, block, window, bitmap, policy, exp_emulation)
        self.shape_q = (batch, heads_q, seq_q, head_dim)
        self.shape_kv = (batch, heads_kv, seq_kv, head_dim)
        self.handle = steel_attn_create(self.params)

    def stats(self) -> dict:
        return steel_attn_get_stats(self.handle)

    def run(self, q, k, v, o=None, lse=None, want_lse: bool = True):
        import torch
        assert q.is_cuda and q.dtype == torch.bfloat16 and q.is_contiguous() and tuple(q.shape) == self.shape_q
        for t in (k, v):
            assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous() and tuple(t.shape) == self.shape_kv
        if o is None:
            o = torch.empty_like(q)
        if lse is None and want_lse:
            lse = torch.empty(self.shape_q[:3], dtype=torch.float32, device=q.device)
        stream = torch.cuda.current_stream(q.device).cuda_stream
        steel_attn_run(self.handle, q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(),
                       lse.data_ptr() if lse is not None else None, stream)
        return o, lse

    def last_status(self) -> int:
        import torch
        return steel_attn_last_status(self.handle, torch.cuda.current_stream().cuda_stream)

    def close(self) -> None:
        if self.handle:
            steel_attn_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class SteelAttentionHost:
    """Owner of one host-memory attention object: ``run`` takes CPU torch tensors (bf16 bit patterns
    as int16 or bfloat16; page-locked for overlap) and fills ``o`` / ``lse`` in host memory."""

    def __init__(self, batch, heads_q, heads_kv, seq_q, seq_kv, head_dim, scale, flags=0, block=128,
                 window=0, bitmap=None, max_chunks=4, policy=0, exp_emulation=0):
        self.params, self._keep = make_params(batch, heads_q, heads_kv, seq_q, seq_kv, head_dim, scale,
                                              flags, block, block, window, bitmap, policy, exp_emulation)
        self.shape_q = (batch, heads_q, seq_q, head_dim)
        self.shape_kv = (batch, heads_kv, seq_kv, head_dim)
        self.handle = steel_attn_host_create(self.params, max_chunks)

    @property
    def chunks(self) -> int:
        return steel_attn_host_chunks(self.handle)

    def run(self, q, k, v, o, lse=None):
        import torch
        for t, shape in ((q, self.shape_q), (k, self.shape_kv), (v, self.shape_kv), (o, self.shape_q)):
            assert not t.is_cuda and t.element_size() == 2 and t.is_contiguous() and tuple(t.shape) == shape
        if lse is not None:
            assert (not lse.is_cuda and lse.dtype == torch.float32 and lse.is_contiguous()
                    and tuple(lse.shape) == self.shape_q[:3])
        stream = torch.cuda.current_stream().cuda_stream
        steel_attn_host_run(self.handle, q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(),
                            lse.data_ptr() if lse is not None else None, stream)
        return o, lse

    def last_status(self) -> int:
        import torch
        return steel_attn_host_last_status(self.handle, torch.cuda.current_stream().cuda_stream)

    def close(self) -> None:
        if self.handle:
            steel_attn_host_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
