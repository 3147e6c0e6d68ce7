"""ctypes loader for the C oracle (``steel_oracle.c``).  Test infrastructure only.

The functions here marshal numpy arrays; all arithmetic lives in the C file, whose header
states what each routine computes and which passage of the paper it follows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "steel_oracle.c")
_LIB = os.path.join(_HERE, "libsteel_oracle.so")
_lib = None


class _CProblem(ctypes.Structure):
    _fields_ = [
        ("batch", ctypes.c_int32), ("heads_q", ctypes.c_int32), ("heads_kv", ctypes.c_int32),
        ("seq_q", ctypes.c_int32), ("seq_kv", ctypes.c_int32), ("head_dim", ctypes.c_int32),
        ("scale", ctypes.c_double), ("flags", ctypes.c_uint32),
        ("block_q", ctypes.c_int32), ("block_kv", ctypes.c_int32),
        ("window", ctypes.c_int64), ("bitmap", ctypes.c_void_p),
    ]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP threads over rows) if it is out of date."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, i64 = ctypes.c_void_p, ctypes.c_int64
        lib.steel_oracle_rows.argtypes = [vp, vp, vp, vp, vp, i64, vp, vp, vp]
        lib.steel_oracle_rows.restype = None
        lib.steel_oracle_alg1_blocks.argtypes = [vp, vp, vp, vp, vp, i64, vp, vp, vp]
        lib.steel_oracle_alg1_blocks.restype = None
        lib.steel_oracle_classify.argtypes = [vp, ctypes.c_int, ctypes.c_int, ctypes.c_int]
        lib.steel_oracle_classify.restype = ctypes.c_int
        lib.steel_oracle_allowed.argtypes = [vp, ctypes.c_int, i64, i64]
        lib.steel_oracle_allowed.restype = ctypes.c_int
        lib.steel_oracle_count_tiles.argtypes = [vp, vp]
        lib.steel_oracle_count_tiles.restype = None
        lib.steel_oracle_max_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


class OracleProblem:
    """Shapes, scale and mask descriptor of one attention problem (host-side)."""

    def __init__(self, batch, heads_q, heads_kv, seq_q, seq_kv, head_dim, scale,
                 flags=0, block_q=128, block_kv=128, window=0, bitmap=None):
        assert heads_q % heads_kv == 0
        self.bitmap = None
        if bitmap is not None:
            self.bitmap = np.ascontiguousarray(bitmap, dtype=np.uint32)
        self.c = _CProblem(batch, heads_q, heads_kv, seq_q, seq_kv, head_dim, float(scale),
                           flags, block_q, block_kv, window,
                           self.bitmap.ctypes.data if self.bitmap is not None else None)
        self.batch, self.heads_q, self.heads_kv = batch, heads_q, heads_kv
        self.seq_q, self.seq_kv, self.head_dim = seq_q, seq_kv, head_dim
        self.block_q, self.block_kv = block_q, block_kv

    @property
    def ptr(self):
        return ctypes.addressof(self.c)


def _bits(x, shape):
    a = np.ascontiguousarray(x, dtype=np.uint16)
    assert a.shape == tuple(shape), (a.shape, shape)
    return a


def _qkv(p: OracleProblem, q, k, v):
    q = _bits(q, (p.batch, p.heads_q, p.seq_q, p.head_dim))
    k = _bits(k, (p.batch, p.heads_kv, p.seq_kv, p.head_dim))
    v = _bits(v, (p.batch, p.heads_kv, p.seq_kv, p.head_dim))
    return q, k, v


def rows(p: OracleProblem, q, k, v, row_list, want_probs: bool = False):
    """Dense-definition attention for the listed (b, h, i) rows.

    Returns (O [n, d] fp64, LSE [n] fp64) and, if asked, the probability rows [n, S_kv].
    """
    q, k, v = _qkv(p, q, k, v)
    r = np.ascontiguousarray(row_list, dtype=np.int64).reshape(-1, 3)
    n = r.shape[0]
    o = np.empty((n, p.head_dim), dtype=np.float64)
    lse = np.empty(n, dtype=np.float64)
    probs = np.empty((n, p.seq_kv), dtype=np.float64) if want_probs else None
    _load().steel_oracle_rows(p.ptr, q.ctypes.data, k.ctypes.data, v.ctypes.data,
                              r.ctypes.data, n, o.ctypes.data, lse.ctypes.data,
                              probs.ctypes.data if want_probs else None)
    return (o, lse, probs) if want_probs else (o, lse)


def all_rows(p: OracleProblem):
    """Row list covering every (b, h, i) of the problem, in output order."""
    b, h, i = np.meshgrid(np.arange(p.batch), np.arange(p.heads_q), np.arange(p.seq_q),
                          indexing="ij")
    return np.stack([b.ravel(), h.ravel(), i.ravel()], axis=1).astype(np.int64)


def alg1_blocks(p: OracleProblem, q, k, v, block_list):
    """Algorithm 1 (tile-skipping online softmax) for the listed (b, h, I) query blocks.

    Returns (O [n, B_q, d], LSE [n, B_q], executed tiles [n]).
    """
    q, k, v = _qkv(p, q, k, v)
    bl = np.ascontiguousarray(block_list, dtype=np.int64).reshape(-1, 3)
    n = bl.shape[0]
    o = np.zeros((n, p.block_q, p.head_dim), dtype=np.float64)
    lse = np.zeros((n, p.block_q), dtype=np.float64)
    executed = np.zeros(n, dtype=np.int64)
    _load().steel_oracle_alg1_blocks(p.ptr, q.ctypes.data, k.ctypes.data, v.ctypes.data,
                                     bl.ctypes.data, n, o.ctypes.data, lse.ctypes.data,
                                     executed.ctypes.data)
    return o, lse, executed


def classify(p: OracleProblem, h: int, i_blk: int, j_blk: int) -> int:
    """0 = fully masked, 1 = unmasked, 2 = partially masked (brute force over the tile)."""
    return _load().steel_oracle_classify(p.ptr, h, i_blk, j_blk)


def allowed(p: OracleProblem, h: int, i: int, j: int) -> bool:
    return bool(_load().steel_oracle_allowed(p.ptr, h, i, j))


def count_tiles(p: OracleProblem):
    """Per-head (kept, partial) tile counts by brute force; int64 array [heads_q, 2]."""
    counts = np.zeros((p.heads_q, 2), dtype=np.int64)
    _load().steel_oracle_count_tiles(p.ptr, counts.ctypes.data)
    return counts


def max_threads() -> int:
    return _load().steel_oracle_max_threads()
