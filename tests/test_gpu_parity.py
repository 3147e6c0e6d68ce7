"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs, element by element.  Tolerances are the stated ones: max-abs 2e-2 and mean-abs
2e-3 on O, 1e-3 on LSE."""
import numpy as np
import pytest
import torch

from paper_2607_09385_b200 import binding, inputs

import helpers as H

pytestmark = pytest.mark.gpu
CAUSAL, WINDOW, BITMAP = inputs.MASK_CAUSAL, inputs.MASK_WINDOW, inputs.MASK_BITMAP


def test_config1_and_config2_all_rows():
    for name in ("c1", "c2"):
        w = inputs.workload(name)
        data = inputs.make_inputs(w)
        attn, o, lse = H.run_gpu(w, data)
        rows = H.all_rows(w) if name == "c1" else H.sampled_rows(w, range(0, w.heads_q, 5), 1, 2048)
        H.assert_parity(w, data, o, lse, rows)
        attn.close()


def test_config2_every_row_of_two_heads():
    w = inputs.workload("c2")
    data = inputs.make_inputs(w)
    attn, o, lse = H.run_gpu(w, data)
    rows = np.array([(0, h, i) for h in (0, 31) for i in range(w.seq)])
    H.assert_parity(w, data, o, lse, rows)
    attn.close()


@pytest.mark.parametrize("name,heads,stride,extra", [
    ("c3", range(0, 32, 4), 1, 512),   # one query head per KV group, every query block
    ("c4", range(16), 2, 512),         # every head, every other query block
])
def test_config3_config4_sampled_rows(name, heads, stride, extra):
    w = inputs.workload(name)
    data = inputs.make_inputs(w)
    attn, o, lse = H.run_gpu(w, data)
    stats = attn.stats()
    if name == "c3":
        assert (stats["kept_tiles"], stats["partial_tiles"]) == (118272, 7168)
    else:
        bits = sum(bin(int(x)).count("1") for x in data["bitmap"].ravel())
        assert stats["kept_tiles"] == bits and stats["partial_tiles"] == 16 * 256
    H.assert_parity(w, data, o, lse, H.sampled_rows(w, heads, stride, extra))
    attn.close()


def test_config5_sampled_rows():
    w = inputs.workload("c5")
    data = inputs.make_inputs(w)
    attn, o, lse = H.run_gpu(w, data, poison=False)
    assert attn.stats()["kept_tiles"] == 16793600
    rows = H.sampled_rows(w, range(0, 32, 4), 8, 256)
    H.assert_parity(w, data, o, lse, rows)
    assert not torch.isnan(lse).any()
    attn.close()


EDGE_CASES = [
    dict(name="dense", B=1, Hq=2, Hkv=1, S=384, D=128, flags=0),
    dict(name="batch2_gqa", B=2, Hq=4, Hkv=2, S=512, D=128, flags=CAUSAL),
    dict(name="odd_group", B=1, Hq=3, Hkv=1, S=640, D=128, flags=CAUSAL),
    dict(name="window_unaligned", B=1, Hq=2, Hkv=2, S=1024, D=128, flags=CAUSAL | WINDOW, window=300),
    dict(name="window_tiny", B=1, Hq=1, Hkv=1, S=512, D=64, flags=CAUSAL | WINDOW, window=1),
    dict(name="window_only", B=1, Hq=2, Hkv=2, S=768, D=128, flags=WINDOW, window=200),
    # a window far beyond 32 bits hides nothing; with a ragged last key tile the kernel's column
    # arithmetic must not overflow
    dict(name="window_huge_ragged", B=1, Hq=2, Hkv=1, S=1000, D=128, flags=WINDOW, window=1 << 40),
    dict(name="bitmap128", B=1, Hq=4, Hkv=4, S=2048, D=128, flags=CAUSAL | BITMAP, keep=0.3),
    dict(name="bitmap64_d64", B=1, Hq=2, Hkv=2, S=1024, D=64, flags=CAUSAL | BITMAP, block=64, keep=0.4),
    dict(name="bitmap_gqa", B=2, Hq=4, Hkv=2, S=1024, D=128, flags=CAUSAL | BITMAP, keep=0.5),
    dict(name="ragged_1000", B=1, Hq=2, Hkv=2, S=1000, D=128, flags=CAUSAL),
    dict(name="ragged_77_d64", B=1, Hq=2, Hkv=1, S=77, D=64, flags=CAUSAL | WINDOW, window=50),
    dict(name="single_row", B=1, Hq=1, Hkv=1, S=1, D=64, flags=CAUSAL),
    dict(name="one_tile_dense", B=1, Hq=1, Hkv=1, S=128, D=128, flags=0),
]


@pytest.mark.parametrize("emu", [0, 3], ids=["hw_exp", "half_poly_exp"])
@pytest.mark.parametrize("case", EDGE_CASES, ids=[c["name"] for c in EDGE_CASES])
def test_edge_cases_all_rows(case, emu):
    """Every edge shape on the shipped kernel builds at both ends of the software-exponent range."""
    w = inputs.Workload(case["name"], case["B"], case["Hq"], case["Hkv"], case["S"], case["D"],
                        case.get("block", 128), case["flags"], window=case.get("window", 0),
                        keep_prob=case.get("keep", 0.0))
    data = inputs.make_inputs(w, seed=0xABC + len(case["name"]))
    if w.flags & BITMAP:
        t = -(-w.seq // w.block)
        data["bitmap"] = inputs.block_bitmap(w.heads_q, t, t, w.keep_prob, seed=5)
    attn, o, lse = H.run_gpu(w, data, exp_emulation=emu)
    H.assert_parity(w, data, o, lse, H.all_rows(w))
    attn.close()


@pytest.mark.parametrize("name", ["bert_h12_d64_s512", "llama1b_h32_d64_s2048"])
def test_paper_shapes_head_dim_64(name):
    """The paper's own attention shapes (BERT bidirectional, Llama-3.1-1B causal; head_dim 64)."""
    w = inputs.workload(name)
    data = inputs.make_inputs(w, seed=64)
    attn, o, lse = H.run_gpu(w, data)
    rows = H.all_rows(w) if w.seq <= 512 else H.sampled_rows(w, range(0, w.heads_q, 3), 1, 512)
    H.assert_parity(w, data, o, lse, rows)
    attn.close()


def test_seq_q_differs_from_seq_kv():
    """Bottom-right aligned causal mask with more keys than queries, and the reverse (rows with no
    visible key give O = 0, LSE = -inf)."""
    import oracle
    rng = np.random.default_rng(3)
    for sq, skv in ((200, 456), (456, 200)):
        D, Hq, Hkv = 128, 2, 1
        q = inputs.f32_to_bf16_bits(rng.standard_normal((1, Hq, sq, D)).astype(np.float32))
        k = inputs.f32_to_bf16_bits(rng.standard_normal((1, Hkv, skv, D)).astype(np.float32))
        v = inputs.f32_to_bf16_bits(rng.standard_normal((1, Hkv, skv, D)).astype(np.float32))
        attn = binding.SteelAttention(1, Hq, Hkv, sq, skv, D, 0.1, CAUSAL)
        o, lse = attn.run(H.to_device(q), H.to_device(k), H.to_device(v))
        assert attn.last_status() == binding.STEEL_OK
        p = oracle.OracleProblem(1, Hq, Hkv, sq, skv, D, 0.1, CAUSAL)
        o_ref, lse_ref = oracle.rows(p, q, k, v, oracle.steel_oracle.all_rows(p))
        og, lg = o.float().cpu().numpy().reshape(-1, D), lse.cpu().numpy().reshape(-1)
        fin = np.isfinite(lse_ref)
        assert np.array_equal(np.isfinite(lg), fin) and np.all(np.isneginf(lg[~fin]))
        assert np.abs(og - o_ref).max() <= H.TOL_O_MAX and np.abs(lg[fin] - lse_ref[fin]).max() <= H.TOL_LSE
        assert np.all(og[~fin] == 0)
        attn.close()


RECT_CASES = [
    # name, seq_q, seq_kv, head_dim, heads_q, heads_kv, flags, window, scale
    ("decode_like_one_query", 1, 3000, 128, 4, 2, CAUSAL, 0, 0.09),
    ("decode_like_window", 5, 2000, 64, 2, 2, CAUSAL | WINDOW, 700, 0.125),
    ("cross_attention_dense", 300, 1000, 128, 2, 1, 0, 0, 0.09),
    ("window_longer_than_sequence", 640, 640, 128, 2, 2, CAUSAL | WINDOW, 100000, 0.09),
    ("large_scale", 384, 384, 64, 2, 2, CAUSAL, 0, 1.5),
]


@pytest.mark.parametrize("case", RECT_CASES, ids=[c[0] for c in RECT_CASES])
def test_rectangular_and_degenerate_shapes(case):
    """Few queries against many keys (bottom-right aligned masks), unmasked cross attention, a window
    that never cuts, and a softmax scale that makes the exponents large: every row against the oracle."""
    import oracle
    name, sq, skv, D, Hq, Hkv, flags, window, scale = case
    rng = np.random.default_rng(len(name))
    q = inputs.f32_to_bf16_bits(rng.standard_normal((1, Hq, sq, D)).astype(np.float32))
    k = inputs.f32_to_bf16_bits(rng.standard_normal((1, Hkv, skv, D)).astype(np.float32))
    v = inputs.f32_to_bf16_bits(rng.standard_normal((1, Hkv, skv, D)).astype(np.float32))
    attn = binding.SteelAttention(1, Hq, Hkv, sq, skv, D, scale, flags, window=window)
    o, lse = attn.run(H.to_device(q), H.to_device(k), H.to_device(v))
    assert attn.last_status() == binding.STEEL_OK
    p = oracle.OracleProblem(1, Hq, Hkv, sq, skv, D, scale, flags, 128, 128, window)
    o_ref, lse_ref = oracle.rows(p, q, k, v, oracle.steel_oracle.all_rows(p))
    og, lg = o.float().cpu().numpy().reshape(-1, D), lse.cpu().numpy().reshape(-1)
    assert np.isfinite(lse_ref).all() and np.isfinite(lg).all()
    err = np.abs(og - o_ref)
    assert err.max() <= H.TOL_O_MAX and err.mean() <= H.TOL_O_MEAN and np.abs(lg - lse_ref).max() <= H.TOL_LSE
    attn.close()


def test_bitmap_with_empty_row_blocks():
    """Rows whose bitmap row-block is empty: O = 0 and LSE = -inf, neighbours unaffected."""
    w = inputs.Workload("empty_rows", 1, 2, 2, 512, 128, 128, BITMAP)
    data = inputs.make_inputs(w, seed=11)
    bitmap = np.zeros((2, 4, 1), dtype=np.uint32)
    bitmap[0, 0, 0], bitmap[0, 2, 0], bitmap[1, 3, 0] = 0b0101, 0b1000, 0b0001
    data["bitmap"] = bitmap
    attn, o, lse = H.run_gpu(w, data)
    H.assert_parity(w, data, o, lse, H.all_rows(w))
    assert torch.all(o[0, 0, 128:256] == 0) and torch.all(torch.isneginf(lse[0, 1, :384]))
    attn.close()


def test_determinism_and_handle_reuse():
    w = inputs.Workload("det", 1, 4, 2, 2048, 128, 128, CAUSAL | BITMAP, keep_prob=0.4)
    data = inputs.make_inputs(w, seed=21)
    attn, o1, lse1 = H.run_gpu(w, data)
    q, k, v = (H.to_device(data[x]) for x in "qkv")
    o2, lse2 = attn.run(q, k, v)
    torch.cuda.synchronize()
    assert torch.equal(o1.view(torch.int16), o2.view(torch.int16)) and torch.equal(lse1, lse2)
    # same handle, other tensors
    data2 = inputs.make_inputs(w, seed=22)
    data2["bitmap"] = data["bitmap"]
    o3, lse3 = attn.run(*(H.to_device(data2[x]) for x in "qkv"))
    assert attn.last_status() == binding.STEEL_OK
    H.assert_parity(w, data2, o3, lse3, H.sampled_rows(w, range(4), 1, 64))
    attn.close()


@pytest.mark.parametrize("policy", [1, 2])
def test_other_placement_policies_match(policy):
    """Uniform (contiguous) and interleaved placement compute the same result as the default."""
    w = inputs.Workload("policy", 1, 4, 4, 2048, 128, 128, CAUSAL)
    data = inputs.make_inputs(w, seed=31)
    attn0, o0, lse0 = H.run_gpu(w, data)
    attn1, o1, lse1 = H.run_gpu(w, data, policy=policy)
    H.assert_parity(w, data, o1, lse1, H.sampled_rows(w, range(4), 1, 64))
    assert (o0.float() - o1.float()).abs().max() <= 2e-2
    attn0.close()
    attn1.close()


def test_run_rejects_bad_arguments():
    w = inputs.workload("c1")
    data = inputs.make_inputs(w)
    attn = H.make_attention(w)
    q, k, v = (H.to_device(data[x]) for x in "qkv")
    o = torch.empty_like(q)
    lib = binding.load_library()
    s = torch.cuda.current_stream().cuda_stream
    assert lib.steel_attn_run(attn.handle, None, k.data_ptr(), v.data_ptr(), o.data_ptr(), None, s) == binding.STEEL_ERR_INVALID_ARG
    assert lib.steel_attn_run(attn.handle, q.data_ptr() + 2, k.data_ptr(), v.data_ptr(), o.data_ptr(), None, s) == binding.STEEL_ERR_INVALID_ARG
    assert lib.steel_attn_run(None, q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), None, s) == binding.STEEL_ERR_INVALID_ARG
    o2, _ = attn.run(q, k, v, want_lse=False)   # LSE may be omitted
    assert attn.last_status() == binding.STEEL_OK and not torch.isnan(o2.float()).any()
    attn.close()
