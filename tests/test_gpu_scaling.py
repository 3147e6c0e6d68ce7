"""Runtime scales with the number of kept tiles (the paper's mask case (i), Sec. "The STEEL Pipeline":
a fully masked tile is skipped, so it must cost neither memory traffic nor tensor-core work): the same
shape at block-bitmap keep probabilities 0.05 ... 1.0, CUDA-event time against the exact kept-tile
count, and parity with the oracle at the two extreme densities."""
import numpy as np
import pytest
import torch

from paper_2607_09385_b200 import binding, inputs

import helpers as H

pytestmark = pytest.mark.gpu


def test_time_is_linear_in_kept_tiles_and_extremes_match_the_oracle():
    base = inputs.Workload("keep_sweep", 1, 16, 16, 8192, 128, 128, inputs.MASK_CAUSAL | inputs.MASK_BITMAP)
    data = inputs.make_inputs(base, seed=21)
    q, k, v = (H.to_device(data[x]) for x in "qkv")
    tiles, ms = [], []
    for keep in (0.05, 0.125, 0.25, 0.5, 1.0):
        bitmap = inputs.block_bitmap(base.heads_q, base.tiles, base.tiles, keep, seed=21)
        d = dict(data, bitmap=bitmap)
        attn = H.make_attention(base, bitmap)
        o = torch.full_like(q, float("nan"))
        lse = torch.full((1, base.heads_q, base.seq), float("nan"), dtype=torch.float32, device="cuda")
        for _ in range(5):
            attn.run(q, k, v, o, lse)
        torch.cuda.synchronize()
        reps = 20
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            attn.run(q, k, v, o, lse)
        e1.record()
        torch.cuda.synchronize()
        assert attn.last_status() == binding.STEEL_OK
        st = attn.stats()
        bits = sum(bin(int(x)).count("1") for x in bitmap.ravel())
        assert st["kept_tiles"] == bits          # the draw's exact count, not the expectation
        tiles.append(st["kept_tiles"])
        ms.append(e0.elapsed_time(e1) / reps)
        if keep in (0.05, 1.0):
            H.assert_parity(base, d, o, lse, H.sampled_rows(base, range(0, 16, 3), 4, 256))
        attn.close()
    x, y = np.array(tiles, dtype=np.float64), np.array(ms, dtype=np.float64)
    slope, intercept = np.polyfit(x, y, 1)
    r2 = 1.0 - ((y - (intercept + slope * x)) ** 2).sum() / ((y - y.mean()) ** 2).sum()
    assert slope > 0 and r2 >= 0.99, (tiles, ms, slope, intercept, r2)
    # twenty times fewer tiles must not cost the same time: the sparsest case is several times faster
    assert y[0] < 0.35 * y[-1], (tiles, ms)
