"""Every output row of the large configurations against a plain fp32 PyTorch attention computed in
chunks on the GPU (dense scores, explicit mask from the predicate, softmax, matmul).  The CPU oracle
stays the authority (sampled rows, tests/test_gpu_parity.py) -- it cannot cover 131072^2 scores --
and this test extends the element-by-element comparison to all rows with an implementation that
shares nothing with the kernel."""
import numpy as np
import pytest
import torch

from paper_2607_09385_b200 import inputs

import helpers as H

pytestmark = pytest.mark.gpu
CAUSAL, WINDOW, BITMAP = inputs.MASK_CAUSAL, inputs.MASK_WINDOW, inputs.MASK_BITMAP


def reference_rows(w, q, k, v, bitmap_bits, h, r0, r1):
    """fp32 attention for rows r0..r1 of query head h: returns (O [rows, d], LSE [rows])."""
    g = h // (w.heads_q // w.heads_kv)
    s = (q[0, h, r0:r1].float() @ k[0, g].float().T) * w.scale
    i = torch.arange(r0, r1, device=q.device)[:, None]
    j = torch.arange(w.seq, device=q.device)[None, :]
    mask = torch.ones_like(s, dtype=torch.bool)
    if w.flags & CAUSAL:
        mask &= j <= i
    if w.flags & WINDOW:
        mask &= (i - j) < w.window
    if w.flags & BITMAP:
        mask &= bitmap_bits[h][(i // w.block).expand_as(mask), (j // w.block).expand_as(mask)]
    s = s.masked_fill(~mask, float("-inf"))
    lse = torch.logsumexp(s, dim=1)
    p = torch.exp(s - lse[:, None])
    return p @ v[0, g].float(), lse


@pytest.mark.parametrize("name,heads", [("c3", None), ("c4", None), ("c5", (0, 9, 18, 31))])
def test_all_rows_against_fp32_torch(name, heads):
    torch.backends.cuda.matmul.allow_tf32 = False
    w = inputs.workload(name)
    data = inputs.make_inputs(w)
    attn, o, lse = H.run_gpu(w, data, poison=(name != "c5"))
    q, k, v = (H.to_device(data[x]) for x in "qkv")
    bits = None
    if w.flags & BITMAP:
        t = w.tiles
        words = torch.from_numpy(data["bitmap"].astype(np.int64)).cuda()
        jj = torch.arange(t, device="cuda")
        bits = ((words[:, :, jj >> 5] >> (jj & 31)) & 1).bool()           # [heads, T, T]
    chunk = 2048 if w.seq <= 32768 else 512
    worst_o = worst_l = 0.0
    sum_abs = 0.0
    count = 0
    for h in (heads if heads is not None else range(w.heads_q)):
        for r0 in range(0, w.seq, chunk):
            o_ref, lse_ref = reference_rows(w, q, k, v, bits, h, r0, r0 + chunk)
            d_o = (o[0, h, r0:r0 + chunk].float() - o_ref).abs()
            worst_o = max(worst_o, float(d_o.max()))
            sum_abs += float(d_o.sum())
            count += d_o.numel()
            worst_l = max(worst_l, float((lse[0, h, r0:r0 + chunk] - lse_ref).abs().max()))
    assert worst_o <= H.TOL_O_MAX and sum_abs / count <= H.TOL_O_MEAN and worst_l <= H.TOL_LSE, \
        (name, worst_o, sum_abs / count, worst_l)
    attn.close()
