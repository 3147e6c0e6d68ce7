"""Bounded device-side waits: when a role never gets what it waits for, the kernel gives up after
the configured number of cycles, returns normally and reports STEEL_ERR_TIMEOUT; the context and
the handle stay usable.  The stall is made with the library's test hook (one CTA's producer
withholds its commands); nothing faults, traps or spins without a limit."""
import time

import pytest
import torch

from paper_2607_09385_b200 import binding, inputs

import helpers as H

pytestmark = pytest.mark.gpu


def test_wait_expiry_sets_status_and_context_stays_usable():
    w = inputs.Workload("stall", 1, 4, 2, 1024, 128, 128, inputs.MASK_CAUSAL)
    data = inputs.make_inputs(w, seed=91)
    attn, o, lse = H.run_gpu(w, data)                      # normal run first
    q, k, v = (H.to_device(data[x]) for x in "qkv")
    binding.steel_attn_debug_stall(attn.handle, 0, 200_000_000)   # about 0.1 s of SM clock
    t0 = time.time()
    attn.run(q, k, v)
    status = attn.last_status()                            # synchronises the stream
    elapsed = time.time() - t0
    assert status == binding.STEEL_ERR_TIMEOUT
    assert elapsed < 30.0
    assert attn.last_status() == binding.STEEL_OK          # the status word was cleared by the read
    binding.steel_attn_debug_stall(attn.handle, -1, 0)     # hook off, default bound restored
    o2, lse2 = attn.run(q, k, v)
    assert attn.last_status() == binding.STEEL_OK
    assert torch.equal(o.view(torch.int16), o2.view(torch.int16)) and torch.equal(lse, lse2)
    H.assert_parity(w, data, o2, lse2, H.sampled_rows(w, range(4), 1, 32))
    with pytest.raises(binding.SteelError):
        binding.steel_attn_debug_stall(attn.handle, 10_000, 0)     # no such CTA
    attn.close()
