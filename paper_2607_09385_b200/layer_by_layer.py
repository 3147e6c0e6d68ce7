"""Layer-by-layer attention: the comparison baseline of the paper's Sec. "Attention Implementation
Benchmark" (GEMM -> scale / mask -> softmax -> GEMM as separate operators, the score matrix A and the
probabilities P travelling through device memory between them).  Library operators only (torch); it
is not part of the fused path and exists to be timed and measured beside it."""
from __future__ import annotations


def layer_by_layer_attention(q, k, v, scale: float, causal: bool):
    """q [B, H, S, d], k / v [B, H, S, d] bf16 CUDA tensors (equal head counts) -> O [B, H, S, d] bf16."""
    import torch
    a = torch.matmul(q, k.transpose(-1, -2))            # A = Q K^T, written to memory in bf16
    a = a * scale                                       # scale operator
    if causal:
        s = q.shape[-2]
        a = a.masked_fill(torch.ones(s, s, dtype=torch.bool, device=q.device).triu(1), float("-inf"))
    p = torch.softmax(a, dim=-1, dtype=torch.float32).to(torch.bfloat16)   # softmax operator, P in bf16
    return torch.matmul(p, v)                           # O = P V


def profile_one_call(workload_name: str) -> None:
    """One warm-up call, then one call between cudaProfilerStart / Stop (for a counter capture of
    exactly the kernels of one layer-by-layer call), then the same for the fused kernel."""
    import numpy as np
    import torch
    from . import binding, inputs
    w = inputs.workload(workload_name)
    assert w.heads_q == w.heads_kv
    data = inputs.make_inputs(w, inputs.DEFAULT_SEED)
    q, k, v = (torch.from_numpy(data[x].view(np.int16)).cuda().view(torch.bfloat16) for x in "qkv")
    causal = bool(w.flags & inputs.MASK_CAUSAL)
    attn = binding.SteelAttention(w.batch, w.heads_q, w.heads_kv, w.seq, w.seq, w.head_dim, w.scale, w.flags,
                                  w.block, w.window, None)
    o = torch.empty_like(q)
    layer_by_layer_attention(q, k, v, w.scale, causal)
    attn.run(q, k, v, o, None, want_lse=False)
    torch.cuda.synchronize()
    flush = torch.zeros(64 << 20, dtype=torch.int32, device="cuda")   # 256 MiB: twice the L2
    flush.add_(1)
    torch.cuda.synchronize()
    torch.cuda.profiler.start()
    ref = layer_by_layer_attention(q, k, v, w.scale, causal)
    torch.cuda.synchronize()
    torch.cuda.profiler.stop()
    flush.add_(1)
    torch.cuda.synchronize()
    torch.cuda.profiler.start()
    attn.run(q, k, v, o, None, want_lse=False)
    torch.cuda.synchronize()
    torch.cuda.profiler.stop()
    print(f"{w.name}: max |layer-by-layer - fused| = {float((ref.float() - o.float()).abs().max()):.3e}")
    attn.close()


if __name__ == "__main__":
    import sys
    profile_one_call(sys.argv[1] if len(sys.argv) > 1 else "bert_h12_d64_s2048")
