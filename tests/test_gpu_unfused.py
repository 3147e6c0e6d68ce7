"""Fused kernel and layer-by-layer attention (the comparison baseline of the paper's Sec. "Attention
Implementation Benchmark": GEMM -> scale / mask -> softmax -> GEMM through device memory) on the
paper's BERT and Llama shapes, each asserted against the fp64 oracle -- not against each other."""
import numpy as np
import pytest
import torch

from paper_2607_09385_b200 import inputs, layer_by_layer, traffic_model

import helpers as H

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["bert_h12_d64_s512", "llama1b_h32_d64_s2048"])
def test_fused_and_layer_by_layer_against_the_oracle(name):
    w = inputs.workload(name)
    data = inputs.make_inputs(w, seed=77)
    attn, o, lse = H.run_gpu(w, data)
    rows = H.all_rows(w) if w.seq <= 512 else H.sampled_rows(w, range(0, w.heads_q, 4), 1, 512)
    H.assert_parity(w, data, o, lse, rows)

    q, k, v = (H.to_device(data[x]) for x in "qkv")
    o_lbl = layer_by_layer.layer_by_layer_attention(q, k, v, w.scale, bool(w.flags & inputs.MASK_CAUSAL))
    # the baseline has no LSE output: compare O only (its score matrix is rounded to bf16 on the way
    # through memory, which the stated O tolerances absorb)
    lse_oracle = torch.zeros_like(lse)
    import oracle
    p = H.oracle_problem(w, data["bitmap"])
    o_ref, _ = oracle.rows(p, data["q"], data["k"], data["v"], rows)
    idx = tuple(torch.from_numpy(rows[:, c]).cuda() for c in range(3))
    err = np.abs(o_lbl[idx].float().cpu().numpy().astype(np.float64) - o_ref)
    assert err.max() <= H.TOL_O_MAX and err.mean() <= H.TOL_O_MEAN, (name, err.max(), err.mean())

    # the traffic model's two sides for this shape: layer-by-layer moves A and P through memory
    st = attn.stats()
    fused = traffic_model.fused_bytes(w.batch, w.heads_q, w.heads_kv, w.seq, w.seq, w.head_dim, st["kv_tile_loads"])
    unfused = traffic_model.unfused_bytes(w.batch, w.heads_q, w.heads_kv, w.seq, w.seq, w.head_dim)
    assert unfused["total"] > 5 * fused["compulsory"]
    attn.close()
    del lse_oracle
