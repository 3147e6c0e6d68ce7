"""Host-side input generator: known splitmix64 vectors, moments, bf16 rounding, bitmap."""
import numpy as np
import torch

from paper_2607_09385_b200 import inputs


def test_splitmix64_reference_vectors():
    # First three outputs of the published splitmix64 generator seeded with 0.
    g = 0x9E3779B97F4A7C15
    states = np.array([0, g, (2 * g) & (2**64 - 1)], dtype=np.uint64)
    out = inputs.splitmix64(states)
    assert [int(x) for x in out] == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]


def test_normal_moments_and_independence_of_chunking():
    e = np.arange(1 << 20, dtype=np.uint64)
    z = inputs.normal(123, inputs.STREAM_Q, e)
    assert abs(z.mean()) < 5e-3 and abs(z.std() - 1.0) < 5e-3
    assert abs(np.mean(z**4) - 3.0) < 0.05
    a = inputs.normal_bf16(7, inputs.STREAM_K, (1, 2, 1 << 21, 2), threads=4)
    b = inputs.normal_bf16(7, inputs.STREAM_K, (1, 2, 1 << 21, 2), threads=1)
    assert np.array_equal(a, b)


def test_bf16_rounding_matches_torch():
    x = np.random.default_rng(0).standard_normal(100000).astype(np.float32)
    x[:4] = [1.00390625, 1.01171875, -0.0, 3.3895314e38]
    bits = inputs.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, ref)
    back = inputs.bf16_bits_to_f64(bits)
    assert np.array_equal(back, torch.from_numpy(x).to(torch.bfloat16).double().numpy())


def test_bitmap_structure_and_density():
    t = 64
    bm = inputs.block_bitmap(4, t, t, 0.25, seed=99)
    assert bm.shape == (4, t, 2) and bm.dtype == np.uint32
    dense = np.array([[[inputs.bitmap_bit(bm, h, i, j) for j in range(t)] for i in range(t)]
                      for h in range(4)])
    for i in range(t):
        assert dense[:, i, i].all() and dense[:, i, 0].all()
        assert not dense[:, i, i + 1:].any()
    free = np.array([dense[h, i, j] for h in range(4) for i in range(t) for j in range(1, i)])
    assert abs(free.mean() - 0.25) < 0.03
    assert not np.array_equal(dense[0], dense[1])


def test_workload_table_and_head_scale():
    assert [w.seq for w in inputs.WORKLOADS] == [256, 4096, 16384, 32768, 131072]
    w = inputs.workload("c1")
    d = inputs.make_inputs(w)
    assert d["q"].shape == (1, 1, 256, 64) and d["bitmap"] is None
    small = inputs.Workload("t", 1, 4, 2, 64, 16, 16, inputs.MASK_CAUSAL, sigma=0.5,
                            head_query_scale=True)
    d = inputs.make_inputs(small)
    s = d["head_scale"]
    assert s.shape == (4,) and (s >= 0.5).all() and (s <= 2.0).all()
    qs = inputs.bf16_bits_to_f64(d["q"])[0].reshape(4, -1).std(axis=1)
    assert np.allclose(qs, 0.5 * s, rtol=0.15)
