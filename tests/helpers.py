"""Shared helpers for the GPU parity tests: device transfer, oracle comparison, row sampling."""
import numpy as np
import torch

import oracle
from paper_2607_09385_b200 import binding, inputs

TOL_O_MAX, TOL_O_MEAN, TOL_LSE = 2e-2, 2e-3, 1e-3  # stated tolerances: bf16 in, fp32 accumulate


def to_device(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def make_attention(w: inputs.Workload, bitmap=None, scale=None, policy=0, exp_emulation=0) -> binding.SteelAttention:
    return binding.SteelAttention(w.batch, w.heads_q, w.heads_kv, w.seq, w.seq, w.head_dim,
                                  w.scale if scale is None else scale, w.flags, w.block, w.window, bitmap,
                                  policy=policy, exp_emulation=exp_emulation)


def oracle_problem(w: inputs.Workload, bitmap=None, scale=None) -> oracle.OracleProblem:
    return oracle.OracleProblem(w.batch, w.heads_q, w.heads_kv, w.seq, w.seq, w.head_dim,
                                w.scale if scale is None else scale, w.flags, w.block, w.block, w.window, bitmap)


def run_gpu(w, data, scale=None, poison=True, policy=0, exp_emulation=0):
    """Run the CUDA path on workload `w`; outputs are pre-filled with NaN so unwritten rows show."""
    attn = make_attention(w, data["bitmap"], scale, policy, exp_emulation)
    q, k, v = (to_device(data[x]) for x in "qkv")
    o = torch.full_like(q, float("nan")) if poison else torch.empty_like(q)
    lse = torch.full((w.batch, w.heads_q, w.seq), float("nan"), dtype=torch.float32, device="cuda")
    attn.run(q, k, v, o, lse)
    assert attn.last_status() == binding.STEEL_OK
    return attn, o, lse


def compare_rows(w, data, o, lse, rows, scale=None):
    """Element-by-element comparison of the listed (b, h, i) rows against the oracle."""
    rows = np.asarray(rows, dtype=np.int64).reshape(-1, 3)
    p = oracle_problem(w, data["bitmap"], scale)
    o_ref, lse_ref = oracle.rows(p, data["q"], data["k"], data["v"], rows)
    idx = tuple(torch.from_numpy(rows[:, c]).cuda() for c in range(3))
    o_gpu = o[idx].float().cpu().numpy().astype(np.float64)
    lse_gpu = lse[idx].cpu().numpy().astype(np.float64)
    assert not np.isnan(o_gpu).any() and not np.isnan(lse_gpu).any(), "rows left unwritten"
    err_o = np.abs(o_gpu - o_ref)
    finite = np.isfinite(lse_ref)
    assert np.array_equal(np.isfinite(lse_gpu), finite)
    err_l = np.abs(lse_gpu[finite] - lse_ref[finite])
    return float(err_o.max()), float(err_o.mean()), float(err_l.max()) if err_l.size else 0.0


def assert_parity(w, data, o, lse, rows, scale=None):
    mx, mean, el = compare_rows(w, data, o, lse, rows, scale)
    assert mx <= TOL_O_MAX and mean <= TOL_O_MEAN and el <= TOL_LSE, (w.name, mx, mean, el)
    return mx, mean, el


def all_rows(w):
    b, h, i = np.meshgrid(np.arange(w.batch), np.arange(w.heads_q), np.arange(w.seq), indexing="ij")
    return np.stack([b.ravel(), h.ravel(), i.ravel()], axis=1)


def sampled_rows(w, per_block_heads, block_stride=1, extra=256, seed=0):
    """Boundary rows for every head, one seeded random row in every `block_stride`-th query block of
    the listed heads, and `extra` seeded random rows anywhere."""
    rng = np.random.default_rng(seed)
    S, bm, W = w.seq, w.block, w.window
    cand = [0, 1, bm - 1, bm, bm + 1, S - bm, S - 1]
    if W:
        cand += [W - 1, W, W + 1, W + bm - 1, W + bm, S - bm - 1]
    boundary = sorted({c for c in cand if 0 <= c < S})
    rows = [(0, h, i) for h in range(w.heads_q) for i in boundary]
    for h in per_block_heads:
        for blk in range(0, S // bm, block_stride):
            rows.append((0, h, blk * bm + int(rng.integers(0, bm))))
    for _ in range(extra):
        rows.append((0, int(rng.integers(0, w.heads_q)), int(rng.integers(0, S))))
    return np.array(sorted(set(rows)), dtype=np.int64)
