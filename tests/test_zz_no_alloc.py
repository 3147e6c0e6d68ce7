"""The allocation-free entry point, called through the C ABI, against the handle-based one.

steel_attn_run_noalloc serves callers that may not allocate device memory (a locked framework
memory pool, a latency path that cannot take cudaMalloc's implicit synchronisation, a fixed memory
budget): its work lists live in a fixed array inside the library.  That array is shared by every
call and keeps the previous call's contents, so the test makes two calls in a row with different
problems and checks each against steel_attn_run on the same inputs.  This file is collected last
on purpose: a run that stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

from paper_2607_09385_b200 import binding as B
from paper_2607_09385_b200 import inputs

import helpers as H

pytestmark = pytest.mark.gpu
CAUSAL, WINDOW, BITMAP = inputs.MASK_CAUSAL, inputs.MASK_WINDOW, inputs.MASK_BITMAP


def run_both(w, seed):
    data = inputs.make_inputs(w, seed)
    q, k, v = (H.to_device(data[x]) for x in "qkv")
    # handle-based path
    attn = H.make_attention(w, data["bitmap"])
    o_ref, lse_ref = attn.run(q, k, v)
    assert attn.last_status() == B.STEEL_OK
    attn.close()
    # allocation-free path: no handle, outputs pre-filled so that unwritten rows would show
    params, keep = B.make_params(w.batch, w.heads_q, w.heads_kv, w.seq, w.seq, w.head_dim, w.scale, w.flags,
                                 w.block, w.block, w.window, data["bitmap"])
    o = torch.full_like(q, float("nan"))
    lse = torch.full((w.batch, w.heads_q, w.seq), float("nan"), dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    args = (params, q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), lse.data_ptr(), stream)
    # The first call on a device loads the kernels and resolves the array's address, so it is made
    # before measuring.  torch's own counters cannot see an allocation made inside the library (its
    # CUDA runtime is linked statically and bypasses torch's caching allocator): the device's free
    # memory is compared instead, around a second call with no torch allocation in between.
    st = B.steel_attn_run_noalloc(*args)
    assert st == B.STEEL_OK, B.steel_status_string(st)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    st = B.steel_attn_run_noalloc(*args)
    free_after, _ = torch.cuda.mem_get_info()
    assert st == B.STEEL_OK, B.steel_status_string(st)
    assert free_after == free_before, (free_before, free_after)
    # same kernel, same plan: the two paths agree within the tolerances the parity tests use
    err_o = (o.float() - o_ref.float()).abs()
    assert not torch.isnan(o.float()).any() and not torch.isnan(lse).any()
    assert float(err_o.max()) <= H.TOL_O_MAX and float(err_o.mean()) <= H.TOL_O_MEAN
    fin = torch.isfinite(lse_ref)
    assert torch.equal(torch.isfinite(lse), fin)
    assert float((lse[fin] - lse_ref[fin]).abs().max()) <= H.TOL_LSE
    return data, o, lse


def test_noalloc_matches_handle_path_on_two_calls_in_a_row():
    # first call: bitmap mask (explicit step lists in the shared array), GQA
    w1 = inputs.Workload("noalloc_bitmap", 1, 4, 2, 2048, 128, 128, CAUSAL | BITMAP, keep_prob=0.35)
    d1, o1, lse1 = run_both(w1, seed=41)
    H.assert_parity(w1, d1, o1, lse1, H.sampled_rows(w1, range(4), 2, 32))
    # second call: a smaller causal-window problem with head_dim 64; stale lists of the first call
    # are still in the array when it starts
    w2 = inputs.Workload("noalloc_window", 2, 2, 1, 640, 64, 64, CAUSAL | WINDOW, window=200)
    d2, o2, lse2 = run_both(w2, seed=42)
    H.assert_parity(w2, d2, o2, lse2, H.all_rows(w2))
    # and the first problem again, after the second overwrote the lists
    run_both(w1, seed=41)


def test_noalloc_rejects_plans_beyond_the_fixed_array():
    # 32 heads x 2048 query tiles = 32768 work items > 16384: refused, nothing launched
    params, _ = B.make_params(1, 32, 32, 262144, 262144, 128, 0.1, CAUSAL)
    t = torch.zeros(16, dtype=torch.bfloat16, device="cuda")
    st = B.steel_attn_run_noalloc(params, t.data_ptr(), t.data_ptr(), t.data_ptr(), t.data_ptr(), None, 0)
    assert st == B.STEEL_ERR_UNSUPPORTED
    assert B.steel_attn_run_noalloc(params, None, t.data_ptr(), t.data_ptr(), t.data_ptr(), None, 0) == B.STEEL_ERR_INVALID_ARG
