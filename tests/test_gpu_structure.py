"""Structural GPU probes with closed-form answers derived from the mask alone.  Random-input
parity cannot see one missing or doubled tile in a long row (it moves O and LSE by about
128 / n); these probes can: every executed tile leaves its own mark on every row."""
import numpy as np
import pytest
import torch

from paper_2607_09385_b200 import binding, inputs

import helpers as H

pytestmark = pytest.mark.gpu
CAUSAL, WINDOW, BITMAP = inputs.MASK_CAUSAL, inputs.MASK_WINDOW, inputs.MASK_BITMAP


def expected_mass(w, bitmap, h, rows):
    """For Q = 0 and V[j, c] = [(j // block) % d == c]: O[i, c] = visible keys of row i in key blocks
    congruent to c, divided by the number n_i of visible keys; LSE_i = ln n_i.  Built from the
    predicate (causal / window intervals, bitmap bits) with torch ops, independent of the planner."""
    dev = rows.device
    T, bm, d = w.seq // w.block, w.block, w.head_dim
    i = rows[:, None].to(torch.int64)
    blk_lo = (torch.arange(T, device=dev, dtype=torch.int64) * bm)[None, :]
    hi = torch.full_like(i, w.seq - 1)
    lo = torch.zeros_like(i)
    if w.flags & CAUSAL:
        hi = torch.minimum(hi, i)
    if w.flags & WINDOW:
        lo = torch.maximum(lo, i - w.window + 1)
    vis = (torch.minimum(hi, blk_lo + bm - 1) - torch.maximum(lo, blk_lo) + 1).clamp_(min=0).float()
    if w.flags & BITMAP:
        words = torch.from_numpy(bitmap[h].astype(np.int64)).to(dev)            # [T, words]
        J = torch.arange(T, device=dev)
        bits = ((words[:, J >> 5] >> (J & 31)[None, :]) & 1).float()            # [T_q, T_kv]
        vis = vis * bits[(rows // bm).long()]
    n = vis.sum(dim=1)
    pad = (-T) % d
    if pad:
        vis = torch.nn.functional.pad(vis, (0, pad))
    mass = vis.view(vis.shape[0], -1, d).sum(dim=1)
    return mass / n[:, None], torch.log(n)


@pytest.mark.parametrize("name", ["c1", "c2", "c3", "c4", "c5"])
def test_mass_per_block_probe_all_rows(name):
    w = inputs.workload(name)
    bitmap = inputs.block_bitmap(w.heads_q, w.tiles, w.tiles, w.keep_prob) if w.flags & BITMAP else None
    attn = H.make_attention(w, bitmap)
    q = torch.zeros((w.batch, w.heads_q, w.seq, w.head_dim), dtype=torch.bfloat16, device="cuda")
    k = torch.randn((w.batch, w.heads_kv, w.seq, w.head_dim), device="cuda").to(torch.bfloat16)
    j = torch.arange(w.seq, device="cuda")
    v1 = torch.nn.functional.one_hot((j // w.block) % w.head_dim, w.head_dim).to(torch.bfloat16)
    v = v1[None, None].expand(w.batch, w.heads_kv, -1, -1).contiguous()
    o = torch.full_like(q, float("nan"))
    lse = torch.full((w.batch, w.heads_q, w.seq), float("nan"), device="cuda")
    attn.run(q, k, v, o, lse)
    assert attn.last_status() == binding.STEEL_OK
    chunk = 8192
    for h in range(w.heads_q):
        for r0 in range(0, w.seq, chunk):
            rows = torch.arange(r0, min(r0 + chunk, w.seq), device="cuda")
            exp_o, exp_lse = expected_mass(w, bitmap, h, rows)
            got = o[0, h, rows].float()
            assert torch.allclose(got, exp_o, rtol=6e-3, atol=1e-6), (name, h, r0, (got - exp_o).abs().max().item())
            assert torch.allclose(lse[0, h, rows], exp_lse, rtol=0, atol=2e-5 * max(1.0, float(exp_lse.max())))
    attn.close()


@pytest.mark.parametrize("flags,window,block", [(CAUSAL, 0, 128), (CAUSAL | WINDOW, 384, 128),
                                                (CAUSAL | WINDOW, 200, 128), (CAUSAL | BITMAP, 0, 64)])
def test_dominant_key_probe(flags, window, block):
    """One key scores far above all others for every query: rows that see it return its V row
    (bf16-exact), rows that do not return the plain average of what they see.  Checks mask edges
    (diagonal, window edge i - j = W - 1 vs W, bitmap bit order) at token resolution."""
    S, D, H_ = 1024, 128, 2
    w = inputs.Workload("dom", 1, H_, H_, S, D, block, flags, window=window, keep_prob=0.5)
    bitmap = inputs.block_bitmap(H_, S // block, S // block, 0.5, seed=3) if flags & BITMAP else None
    rng = np.random.default_rng(1)
    for jstar in (0, 127, 128, 300, 511, 640, 1023):
        q = np.zeros((1, H_, S, D), np.float32)
        k = np.zeros((1, H_, S, D), np.float32)
        q[..., 5] = 16.0
        k[0, :, jstar, 5] = 16.0                      # score 256 * scale on key j*, 0 elsewhere
        v = rng.standard_normal((1, H_, S, D)).astype(np.float32)
        data = {"q": inputs.f32_to_bf16_bits(q), "k": inputs.f32_to_bf16_bits(k),
                "v": inputs.f32_to_bf16_bits(v), "bitmap": bitmap}
        attn, o, lse = H.run_gpu(w, data, scale=1.0)
        vb = inputs.bf16_bits_to_f64(data["v"])
        og = o.float().cpu().numpy()
        for h in range(H_):
            i = np.arange(S)
            sees = i >= jstar if flags & CAUSAL else np.ones(S, bool)
            if flags & WINDOW:
                sees &= (i - jstar) < window
            if flags & BITMAP:
                sees &= np.array([inputs.bitmap_bit(bitmap, h, r // block, jstar // block) for r in i])
            assert np.array_equal(og[0, h, sees], np.broadcast_to(vb[0, h, jstar], (int(sees.sum()), D)).astype(np.float32))
            # rows that do not see j* : uniform average over their visible keys (oracle checks values)
        rows = np.array([(0, h, r) for h in range(H_) for r in (0, 1, 127, 128, 129, 255, 256, 400, 639, 640, 641, 1023)])
        H.assert_parity(w, data, o, lse, rows, scale=1.0)
        attn.close()


@pytest.mark.parametrize("direction", ["increasing", "decreasing", "spikes"])
def test_rescale_stress(direction):
    """Scores ramp with the key index so the running maximum grows at every tile (every step
    rescales O), shrinks at every tile (never rescales), or jumps by far more than the lazy
    threshold at scattered keys."""
    S, D = 2048, 128
    w = inputs.Workload("ramp", 1, 2, 1, S, D, 128, 0 if direction == "spikes" else CAUSAL)
    rng = np.random.default_rng(2)
    q = rng.standard_normal((1, 2, S, D)).astype(np.float32) * 0.1
    k = rng.standard_normal((1, 1, S, D)).astype(np.float32) * 0.1
    v = rng.standard_normal((1, 1, S, D)).astype(np.float32)
    q[..., 0] = 8.0
    ramp = np.arange(S, dtype=np.float32) / S * 12.0          # score ramp of about 96 * scale ... large
    if direction == "increasing":
        k[0, 0, :, 0] = ramp
    elif direction == "decreasing":
        k[0, 0, :, 0] = ramp[::-1]
    else:
        k[0, 0, rng.choice(S, 24, replace=False), 0] = rng.uniform(4.0, 16.0, 24).astype(np.float32)
    data = {"q": inputs.f32_to_bf16_bits(q), "k": inputs.f32_to_bf16_bits(k), "v": inputs.f32_to_bf16_bits(v),
            "bitmap": None}
    attn, o, lse = H.run_gpu(w, data, scale=1.0)
    H.assert_parity(w, data, o, lse, H.all_rows(w), scale=1.0)
    attn.close()


def test_rows_masked_in_their_first_tile():
    """Window mask whose far-left partial tile hides every key from the last rows of a query tile
    while their running maximum is still -inf: no NaN, parity holds (W a multiple of the tile)."""
    w = inputs.Workload("farleft", 1, 2, 2, 1024, 128, 128, CAUSAL | WINDOW, window=256)
    data = inputs.make_inputs(w, seed=77)
    attn, o, lse = H.run_gpu(w, data)
    assert not torch.isnan(o.float()).any() and not torch.isnan(lse).any()
    H.assert_parity(w, data, o, lse, H.all_rows(w))
    attn.close()
