"""The C ABI library loads and exports every function the public header declares; argument
validation returns the documented status codes (no GPU needed)."""
import ctypes
import os
import re

import numpy as np
import torch

from paper_2607_09385_b200 import binding as B


def header_functions(repo_root):
    text = open(os.path.join(repo_root, "include", "steel_attn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(steel_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(repo_root):
    lib = B.load_library()
    names = header_functions(repo_root)
    assert set(names) == set(B.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_struct_layouts_match_header():
    assert ctypes.sizeof(B.MaskDesc) == 32 and ctypes.sizeof(B.Params) == 72
    assert ctypes.sizeof(B.Stats) == 13 * 8


def test_status_strings():
    assert B.steel_status_string(0) == "ok"
    assert "timed out" in B.steel_status_string(B.STEEL_ERR_TIMEOUT)
    assert len({B.steel_status_string(i) for i in range(6)}) == 6


def plan(**kw):
    args = dict(batch=1, heads_q=2, heads_kv=1, seq_q=256, seq_kv=256, head_dim=128, scale=0.1, flags=1)
    args.update(kw)
    p, keep = B.make_params(**args)
    return B.steel_attn_plan_host(p)[0]


def test_validation_codes():
    assert plan() == B.STEEL_OK
    assert plan(batch=0) == B.STEEL_ERR_INVALID_ARG
    assert plan(heads_q=3, heads_kv=2) == B.STEEL_ERR_INVALID_ARG
    assert plan(scale=0.0) == B.STEEL_ERR_INVALID_ARG
    assert plan(scale=float("nan")) == B.STEEL_ERR_INVALID_ARG
    assert plan(scale=-1.0) == B.STEEL_ERR_INVALID_ARG
    assert plan(flags=8) == B.STEEL_ERR_INVALID_ARG
    assert plan(flags=3, window=0) == B.STEEL_ERR_INVALID_ARG
    assert plan(flags=5, bitmap=None) == B.STEEL_ERR_INVALID_ARG
    assert plan(head_dim=96) == B.STEEL_ERR_UNSUPPORTED
    assert plan(block_q=32, block_kv=32) == B.STEEL_ERR_UNSUPPORTED
    assert plan(block_q=64, block_kv=128) == B.STEEL_ERR_UNSUPPORTED
    assert plan(flags=5, bitmap=np.ones((2, 2, 1), np.uint32)) == B.STEEL_OK
    lib = B.load_library()
    assert lib.steel_attn_plan_host(None, ctypes.byref(B.Stats()), None, 0, None) == B.STEEL_ERR_INVALID_ARG
    assert lib.steel_attn_destroy(None) == B.STEEL_OK
    assert lib.steel_attn_get_stats(None, None) == B.STEEL_ERR_INVALID_ARG
    assert plan(policy=7) == B.STEEL_ERR_INVALID_ARG
    assert plan(policy=-1) == B.STEEL_ERR_INVALID_ARG
    assert plan(exp_emulation=4) == B.STEEL_ERR_INVALID_ARG
    assert plan(exp_emulation=3, policy=2) == B.STEEL_OK
    assert lib.steel_attn_create(None, None) == B.STEEL_ERR_INVALID_ARG


def test_create_without_gpu_fails_loudly():
    """No CPU fallback: on a machine without a CUDA device create reports STEEL_ERR_CUDA."""
    if torch.cuda.is_available():
        return
    p, _ = B.make_params(1, 1, 1, 256, 256, 64, 0.125, 1, 64, 64)
    handle = ctypes.c_void_p(123)
    st = B.load_library().steel_attn_create(ctypes.byref(p), ctypes.byref(handle))
    assert st == B.STEEL_ERR_CUDA and handle.value is None


def test_host_entry_points_argument_checks_and_no_gpu():
    """The host-memory form validates before touching CUDA and has no CPU fallback either."""
    lib = B.load_library()
    handle = ctypes.c_void_p(123)
    assert lib.steel_attn_host_create(None, 4, ctypes.byref(handle)) == B.STEEL_ERR_INVALID_ARG
    assert handle.value is None
    p, _ = B.make_params(1, 4, 3, 256, 256, 64, 0.125, 1, 64, 64)  # heads_q % heads_kv != 0
    assert lib.steel_attn_host_create(ctypes.byref(p), 4, ctypes.byref(handle)) == B.STEEL_ERR_INVALID_ARG
    assert lib.steel_attn_host_create(ctypes.byref(p), 4, None) == B.STEEL_ERR_INVALID_ARG
    assert lib.steel_attn_host_run(None, None, None, None, None, None, None) == B.STEEL_ERR_INVALID_ARG
    assert lib.steel_attn_host_last_status(None, None) == B.STEEL_ERR_INVALID_ARG
    assert lib.steel_attn_host_chunks(None) == 0
    assert lib.steel_attn_host_destroy(None) == B.STEEL_OK
    if not torch.cuda.is_available():
        p, _ = B.make_params(2, 2, 2, 256, 256, 64, 0.125, 1, 64, 64)
        handle = ctypes.c_void_p(123)
        st = lib.steel_attn_host_create(ctypes.byref(p), 2, ctypes.byref(handle))
        assert st == B.STEEL_ERR_CUDA and handle.value is None
