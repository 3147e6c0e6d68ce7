"""The HBM traffic model (this repository's own; the paper's formulas are not printed): closed-form
checks and the orderings it must respect."""
from paper_2607_09385_b200 import traffic_model as T


def test_fused_bounds_and_unfused_total():
    # 12 heads, S = 4096, d = 64 (the BERT shape of the paper's comparison)
    f = T.fused_bytes(1, 12, 12, 4096, 4096, 64, kv_tile_loads=12 * 32 * 32 // 2)
    q = 12 * 4096 * 64 * 2
    assert f["compulsory"] == 2 * q + 2 * q + 12 * 4096 * 4
    assert f["no_reuse"] == 2 * q + 12 * 4096 * 4 + (12 * 32 * 32 // 2) * 2 * 128 * 64 * 2
    assert f["compulsory"] < f["no_reuse"]
    u = T.unfused_bytes(1, 12, 12, 4096, 4096, 64)
    scores = 12 * 4096 * 4096
    assert u["total"] == (q + q + 2 * scores) + 4 * scores + (2 * scores + 2 * scores) + (2 * scores + q + q)
    assert u["total"] == sum(u[k] for k in ("gemm1", "scale_mask", "softmax", "gemm2"))
    # the score matrix dominates: traffic grows with S^2 for layer-by-layer, with S for fused
    u2 = T.unfused_bytes(1, 12, 12, 8192, 8192, 64)
    f2 = T.fused_bytes(1, 12, 12, 8192, 8192, 64)
    assert 3.9 < u2["total"] / u["total"] < 4.0 and f2["compulsory"] == 2 * f["compulsory"]
    assert 90 < u["total"] / f["compulsory"] < 100      # 2.44 GB against 25.4 MB at S = 4096
