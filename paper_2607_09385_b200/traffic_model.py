"""Off-chip (HBM) traffic model of fused block-sparse attention against layer-by-layer attention.

The paper compares the two with an analytic transfer-volume model (Sec. "Attention Implementation
Benchmark") whose formulas it does not print; this is this repository's own model, stated in full
here, for the B200 memory hierarchy (tiles staged in shared memory, reuse through L2).  All sizes
in bytes; bf16 tensors (2 bytes) unless said otherwise.

Fused kernel, per call:
    compulsory   Q + O once, K + V once per KV head, LSE once           (perfect reuse through L2)
    no_reuse     Q + O + LSE once, K + V once per K/V tile load         (no reuse at all)
The measured traffic lies between the two.

Layer-by-layer (GEMM -> scale/mask -> softmax -> GEMM, every intermediate through HBM), per call,
for dense scores of ``score_bytes`` per element:
    GEMM 1     reads Q, K                 writes A  [B, Hq, Sq, Skv]
    scale/mask reads A                    writes A
    softmax    reads A                    writes P  (bf16)
    GEMM 2     reads P, V                 writes O
"""
from __future__ import annotations


def tensor_bytes(batch: int, heads: int, seq: int, head_dim: int, elem: int = 2) -> int:
    return batch * heads * seq * head_dim * elem


def fused_bytes(batch, heads_q, heads_kv, seq_q, seq_kv, head_dim, kv_tile_loads=None, tile=128) -> dict:
    q = tensor_bytes(batch, heads_q, seq_q, head_dim)
    kv = 2 * tensor_bytes(batch, heads_kv, seq_kv, head_dim)
    lse = batch * heads_q * seq_q * 4
    out = {"compulsory": 2 * q + kv + lse}
    if kv_tile_loads is not None:
        out["no_reuse"] = 2 * q + lse + kv_tile_loads * 2 * tile * head_dim * 2
    return out


def unfused_bytes(batch, heads_q, heads_kv, seq_q, seq_kv, head_dim, score_bytes: int = 2) -> dict:
    q = tensor_bytes(batch, heads_q, seq_q, head_dim)
    k = tensor_bytes(batch, heads_kv, seq_kv, head_dim)
    scores = batch * heads_q * seq_q * seq_kv
    gemm1 = q + k + scores * score_bytes
    scale = 2 * scores * score_bytes
    softmax = scores * score_bytes + scores * 2
    gemm2 = scores * 2 + k + q
    return {"gemm1": gemm1, "scale_mask": scale, "softmax": softmax, "gemm2": gemm2,
            "total": gemm1 + scale + softmax + gemm2}
