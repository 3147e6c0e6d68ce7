"""The host-memory entry points (steel_attn_host_*) through the C ABI.

Operands start in host memory and results end there; the library cuts the problem into chunks
(batch elements, or KV-head groups with their slice of the bitmap) and overlaps copies with
kernels.  The tests compare the host path with the oracle and with steel_attn_run on the same
inputs, for both ways of chunking, page-locked and pageable memory, and repeated calls.
"""
import numpy as np
import pytest
import torch

from paper_2607_09385_b200 import binding as B
from paper_2607_09385_b200 import inputs

import helpers as H

pytestmark = pytest.mark.gpu
CAUSAL, WINDOW, BITMAP = inputs.MASK_CAUSAL, inputs.MASK_WINDOW, inputs.MASK_BITMAP


def host_tensors(w, data, pinned=True):
    t = {x: torch.from_numpy(np.ascontiguousarray(data[x]).view(np.int16)) for x in "qkv"}
    o = torch.full(t["q"].shape, 0x7FC0, dtype=torch.int16)  # bf16 NaN pattern: unwritten rows show
    lse = torch.full((w.batch, w.heads_q, w.seq), float("nan"), dtype=torch.float32)
    if pinned:
        t = {x: y.pin_memory() for x, y in t.items()}
        o, lse = o.pin_memory(), lse.pin_memory()
    return t, o, lse


def run_host(w, data, max_chunks, pinned=True, want_lse=True, repeat=1):
    attn = B.SteelAttentionHost(w.batch, w.heads_q, w.heads_kv, w.seq, w.seq, w.head_dim, w.scale, w.flags,
                                w.block, w.window, data["bitmap"], max_chunks=max_chunks)
    t, o, lse = host_tensors(w, data, pinned)
    for _ in range(repeat):
        attn.run(t["q"], t["k"], t["v"], o, lse if want_lse else None)
    assert attn.last_status() == B.STEEL_OK
    chunks = attn.chunks
    attn.close()
    return o.view(torch.bfloat16), lse, chunks


def run_device(w, data):
    attn, o, lse = H.run_gpu(w, data)
    attn.close()
    return o.cpu(), lse.cpu()


def assert_close_to_device(w, data, o, lse):
    o_dev, lse_dev = run_device(w, data)
    assert not torch.isnan(o.float()).any() and not torch.isnan(lse).any()
    err = (o.float() - o_dev.float()).abs()
    assert float(err.max()) <= H.TOL_O_MAX and float(err.mean()) <= H.TOL_O_MEAN
    fin = torch.isfinite(lse_dev)
    assert torch.equal(torch.isfinite(lse), fin)
    assert float((lse[fin] - lse_dev[fin]).abs().max()) <= H.TOL_LSE


def parity_on_host(w, data, o, lse, rows):
    return H.assert_parity(w, data, o.cuda(), lse.cuda(), rows)


def test_single_chunk_is_bit_identical_to_the_device_call():
    w = inputs.Workload("host_one", 1, 4, 2, 1024, 128, 128, CAUSAL)
    data = inputs.make_inputs(w, 51)
    o, lse, chunks = run_host(w, data, max_chunks=1)
    assert chunks == 1
    o_dev, lse_dev = run_device(w, data)
    assert torch.equal(o.view(torch.int16), o_dev.view(torch.int16))
    assert torch.equal(lse, lse_dev)


def test_head_chunks_with_bitmap_slices():
    # batch 1: chunks are KV-head groups; every chunk plans its own slice of the per-head bitmap
    w = inputs.Workload("host_heads", 1, 8, 4, 1536, 128, 128, CAUSAL | BITMAP, keep_prob=0.4)
    data = inputs.make_inputs(w, 52)
    o, lse, chunks = run_host(w, data, max_chunks=4, repeat=2)
    assert chunks == 4
    parity_on_host(w, data, o, lse, H.sampled_rows(w, range(8), 1, 64))
    assert_close_to_device(w, data, o, lse)


def test_head_chunk_count_is_a_divisor():
    # 6 KV heads, at most 4 chunks: 3 chunks of 2 KV heads (4 query heads) each
    w = inputs.Workload("host_div", 1, 12, 6, 700, 64, 64, CAUSAL | WINDOW, window=300)
    data = inputs.make_inputs(w, 53)
    o, lse, chunks = run_host(w, data, max_chunks=4)
    assert chunks == 3
    parity_on_host(w, data, o, lse, H.sampled_rows(w, range(12), 1, 64))
    assert_close_to_device(w, data, o, lse)


def test_batch_chunks_share_one_plan():
    # batch 4, at most 2 chunks: two chunks of two batch elements; the bitmap is shared across the batch
    w = inputs.Workload("host_batch", 4, 2, 1, 640, 128, 128, BITMAP, keep_prob=0.5)
    data = inputs.make_inputs(w, 54)
    o, lse, chunks = run_host(w, data, max_chunks=2)
    assert chunks == 2
    parity_on_host(w, data, o, lse, H.all_rows(w)[::7])
    assert_close_to_device(w, data, o, lse)


def test_pageable_memory_and_no_lse():
    w = inputs.Workload("host_pageable", 2, 2, 2, 512, 64, 64, CAUSAL)
    data = inputs.make_inputs(w, 55)
    o, lse, chunks = run_host(w, data, max_chunks=8, pinned=False, want_lse=False)
    assert chunks == 2
    assert torch.isnan(lse).all()  # untouched
    o_dev, _ = run_device(w, data)
    assert torch.equal(o.view(torch.int16), o_dev.view(torch.int16))


def test_host_call_is_ordered_with_the_callers_stream():
    # The call starts after earlier work on the stream (a device-side producer of the host inputs is
    # emulated by a host copy queued on the stream) and later work on the stream sees its results.
    w = inputs.Workload("host_order", 1, 4, 4, 1024, 128, 128, CAUSAL)
    data = inputs.make_inputs(w, 56)
    t, o, lse = host_tensors(w, data)
    staged = {x: torch.zeros_like(t[x]).pin_memory() for x in "qkv"}
    dev_src = {x: t[x].cuda() for x in "qkv"}
    attn = B.SteelAttentionHost(w.batch, w.heads_q, w.heads_kv, w.seq, w.seq, w.head_dim, w.scale, w.flags,
                                w.block, w.window, None, max_chunks=4)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for x in "qkv":
            staged[x].copy_(dev_src[x], non_blocking=True)  # inputs reach host memory on this stream
        attn.run(staged["q"], staged["k"], staged["v"], o, lse)
        o_back = o.cuda(non_blocking=True)  # queued after the call on the same stream
    stream.synchronize()
    assert attn.last_status() == B.STEEL_OK
    attn.close()
    o_dev, lse_dev = run_device(w, data)
    assert torch.equal(o_back.cpu(), o_dev.view(torch.int16))
    assert torch.equal(lse, lse_dev)


def test_host_argument_errors():
    params, _ = B.make_params(1, 4, 3, 256, 256, 128, 0.1, CAUSAL)  # heads_q not a multiple of heads_kv
    with pytest.raises(B.SteelError) as e:
        B.steel_attn_host_create(params, 2)
    assert e.value.status == B.STEEL_ERR_INVALID_ARG
    params, _ = B.make_params(1, 4, 4, 256, 256, 96, 0.1, CAUSAL)  # head_dim outside {64, 128}
    with pytest.raises(B.SteelError) as e:
        B.steel_attn_host_create(params, 2)
    assert e.value.status == B.STEEL_ERR_UNSUPPORTED
    params, _ = B.make_params(1, 2, 2, 256, 256, 64, 0.1, CAUSAL)
    h = B.steel_attn_host_create(params, 2)
    lib = B.load_library()
    assert lib.steel_attn_host_run(h, None, None, None, None, None, None) == B.STEEL_ERR_INVALID_ARG
    assert lib.steel_attn_host_chunks(None) == 0
    B.steel_attn_host_destroy(h)
    B.steel_attn_host_destroy(None)
