"""Pins for the CPU oracle: each test ties it to something other than itself.

Sources of truth used here: a brute-force dense softmax built with numpy broadcasting,
closed forms (Q = 0, one visible key, constant V), invariances of softmax attention, a
library routine (torch scaled_dot_product_attention in fp64 with a boolean mask) and the
closed-form tile counts stored under tests/golden/.
"""
import itertools
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2607_09385_b200 import inputs

CAUSAL, WINDOW, BITMAP = inputs.MASK_CAUSAL, inputs.MASK_WINDOW, inputs.MASK_BITMAP


def rand_bits(rng, shape, sigma=1.0):
    return inputs.f32_to_bf16_bits((rng.standard_normal(shape) * sigma).astype(np.float32))


def dense_mask(flags, sq, skv, block_q, block_kv, window, bitmap, heads):
    """Boolean [heads, sq, skv] visibility, by numpy broadcasting (independent of the C code)."""
    i = np.arange(sq)[:, None] + (skv - sq)
    j = np.arange(skv)[None, :]
    m = np.ones((heads, sq, skv), dtype=bool)
    if flags & CAUSAL:
        m &= (j <= i)[None]
    if flags & WINDOW:
        m &= (i - j < window)[None]
    if flags & BITMAP:
        tq, tkv = -(-sq // block_q), -(-skv // block_kv)
        blk = np.zeros((heads, tq, tkv), dtype=bool)
        for h, a, b in itertools.product(range(heads), range(tq), range(tkv)):
            blk[h, a, b] = (int(bitmap[h, a, b >> 5]) >> (b & 31)) & 1
        m &= np.repeat(np.repeat(blk, block_q, axis=1), block_kv, axis=2)[:, :sq, :skv]
    return m


def brute_force(qb, kb, vb, scale, mask):
    """softmax(Q K^T * scale + M) V with materialised [S_q, S_kv] matrices, fp64."""
    q, k, v = (inputs.bf16_bits_to_f64(x) for x in (qb, kb, vb))
    B, Hq, Sq, D = q.shape
    G = Hq // k.shape[1]
    o = np.zeros((B, Hq, Sq, D))
    lse = np.zeros((B, Hq, Sq))
    for b in range(B):
        for h in range(Hq):
            a = (q[b, h] @ k[b, h // G].T) * scale
            a = np.where(mask[h], a, -np.inf)
            with np.errstate(invalid="ignore"):
                mx = a.max(axis=1, keepdims=True)
                mx = np.where(np.isfinite(mx), mx, 0.0)
                e = np.exp(a - mx)
            s = e.sum(axis=1, keepdims=True)
            with np.errstate(divide="ignore", invalid="ignore"):
                p = np.where(s > 0, e / s, 0.0)
                lse[b, h] = np.where(s[:, 0] > 0, np.log(s[:, 0]) + mx[:, 0], -np.inf)
            o[b, h] = p @ v[b, h // G]
    return o, lse


def make_problem(B, Hq, Hkv, Sq, Skv, D, flags, blk=8, window=0, bitmap=None, scale=None):
    scale = 1.0 / np.sqrt(D) if scale is None else scale
    return oracle.OracleProblem(B, Hq, Hkv, Sq, Skv, D, scale, flags, blk, blk, window, bitmap)


def random_bitmap(rng, heads, tq, tkv, p=0.5, diagonal=True):
    bits = rng.random((heads, tq, tkv)) < p
    if diagonal:
        for t in range(min(tq, tkv)):
            bits[:, t, t] = True
    words = np.zeros((heads, tq, (tkv + 31) // 32), dtype=np.uint32)
    for h, a, b in itertools.product(range(heads), range(tq), range(tkv)):
        if bits[h, a, b]:
            words[h, a, b >> 5] |= np.uint32(1 << (b & 31))
    return words


CASES = [
    dict(B=1, Hq=1, Hkv=1, Sq=16, Skv=16, D=8, flags=0),
    dict(B=2, Hq=4, Hkv=2, Sq=32, Skv=32, D=16, flags=CAUSAL),
    dict(B=1, Hq=2, Hkv=1, Sq=48, Skv=48, D=8, flags=CAUSAL | WINDOW, window=16),
    dict(B=1, Hq=2, Hkv=2, Sq=40, Skv=40, D=8, flags=CAUSAL | WINDOW, window=11),
    dict(B=1, Hq=3, Hkv=1, Sq=64, Skv=64, D=8, flags=BITMAP),
    dict(B=1, Hq=4, Hkv=2, Sq=64, Skv=64, D=16, flags=CAUSAL | BITMAP),
    dict(B=1, Hq=2, Hkv=2, Sq=24, Skv=56, D=8, flags=CAUSAL),            # S_q != S_kv
    dict(B=1, Hq=2, Hkv=1, Sq=20, Skv=52, D=8, flags=CAUSAL | WINDOW, window=9),
    dict(B=1, Hq=1, Hkv=1, Sq=37, Skv=37, D=8, flags=CAUSAL),            # ragged last block
]


@pytest.mark.parametrize("case", CASES)
def test_rows_equal_brute_force_and_probabilities(case):
    rng = np.random.default_rng(hash(tuple(sorted(case.items()))) % 2**32)
    c = dict(case)
    B, Hq, Hkv, Sq, Skv, D = (c[x] for x in ("B", "Hq", "Hkv", "Sq", "Skv", "D"))
    blk = 8
    bitmap = None
    if c["flags"] & BITMAP:
        bitmap = random_bitmap(rng, Hq, -(-Sq // blk), -(-Skv // blk), 0.4,
                               diagonal=bool(c["flags"] & CAUSAL))
    p = make_problem(B, Hq, Hkv, Sq, Skv, D, c["flags"], blk, c.get("window", 0), bitmap)
    q, k, v = rand_bits(rng, (B, Hq, Sq, D)), rand_bits(rng, (B, Hkv, Skv, D)), rand_bits(rng, (B, Hkv, Skv, D))
    mask = dense_mask(c["flags"], Sq, Skv, blk, blk, c.get("window", 0), bitmap, Hq)
    o_ref, lse_ref = brute_force(q, k, v, p.c.scale, mask)
    rows = oracle.steel_oracle.all_rows(p)
    o, lse, probs = oracle.rows(p, q, k, v, rows, want_probs=True)
    o = o.reshape(B, Hq, Sq, D)
    lse = lse.reshape(B, Hq, Sq)
    probs = probs.reshape(B, Hq, Sq, Skv)
    assert np.allclose(o, o_ref, rtol=0, atol=1e-12)
    finite = np.isfinite(lse_ref)
    assert np.array_equal(np.isfinite(lse), finite)
    assert np.allclose(lse[finite], lse_ref[finite], rtol=0, atol=1e-12)
    # rows of P sum to one (or to zero for a row with no visible key); P = 0 where masked
    sums = probs.sum(axis=-1)
    assert np.allclose(sums[finite], 1.0, atol=1e-12) and np.all(sums[~finite] == 0.0)
    for b in range(B):
        assert np.all(probs[b][~mask] == 0.0)
        assert np.all(probs[b][mask & finite[b][..., None]] > 0.0)
    # the predicate itself, element by element
    for h in range(Hq):
        for i, j in itertools.product(range(0, Sq, 3), range(0, Skv, 5)):
            assert oracle.allowed(p, h, i, j) == bool(mask[h, i, j])


def test_empty_rows_without_causal_bitmap():
    """A bitmap whose row-block is empty leaves rows with no visible key: O = 0, LSE = -inf."""
    rng = np.random.default_rng(5)
    bitmap = np.zeros((1, 4, 1), dtype=np.uint32)
    bitmap[0, 0, 0] = 0b0011
    bitmap[0, 2, 0] = 0b1000
    p = make_problem(1, 1, 1, 32, 32, 8, BITMAP, 8, 0, bitmap)
    q, k, v = (rand_bits(rng, (1, 1, 32, 8)) for _ in range(3))
    o, lse = oracle.rows(p, q, k, v, oracle.steel_oracle.all_rows(p))
    empty = np.r_[8:16, 24:32]
    assert np.all(o[empty] == 0.0) and np.all(np.isneginf(lse[empty]))
    assert np.all(np.isfinite(lse[np.r_[0:8, 16:24]]))


def test_alg1_equals_dense_exhaustive_small_grids():
    """Algorithm 1 over kept tiles == dense masked attention, for every bitmap on a 3x3 grid
    (with and without causal) and a sample of 4x4 grids."""
    rng = np.random.default_rng(11)
    blk, D = 4, 8
    for T, flag_set, masks in (
        (3, (BITMAP, BITMAP | CAUSAL), range(1 << 9)),
        (4, (BITMAP | CAUSAL,), [int(x) for x in rng.integers(0, 1 << 16, 150)]),
    ):
        S = T * blk
        q, k, v = (rand_bits(rng, (1, 1, S, D), 2.0) for _ in range(3))
        for flags in flag_set:
            for code in masks:
                bitmap = np.zeros((1, T, 1), dtype=np.uint32)
                for a in range(T):
                    bitmap[0, a, 0] = (code >> (a * T)) & ((1 << T) - 1)
                p = make_problem(1, 1, 1, S, S, D, flags, blk, 0, bitmap)
                blocks = [(0, 0, a) for a in range(T)]
                o1, lse1, executed = oracle.alg1_blocks(p, q, k, v, blocks)
                o2, lse2 = oracle.rows(p, q, k, v, oracle.steel_oracle.all_rows(p))
                assert np.allclose(o1.reshape(S, D), o2, atol=1e-12)
                fin = np.isfinite(lse2)
                assert np.array_equal(np.isfinite(lse1.ravel()), fin)
                assert np.allclose(lse1.ravel()[fin], lse2[fin], atol=1e-12)
                kept = [sum(oracle.classify(p, 0, a, b) != 0 for b in range(T)) for a in range(T)]
                assert list(executed) == kept


@pytest.mark.parametrize("flags,window", [(CAUSAL, 0), (CAUSAL | WINDOW, 24), (0, 0),
                                          (CAUSAL | WINDOW, 13)])
def test_alg1_equals_dense_causal_window(flags, window):
    rng = np.random.default_rng(3)
    S, D, blk = 96, 16, 8
    p = make_problem(1, 4, 2, S, S, D, flags, blk, window)
    q, k, v = rand_bits(rng, (1, 4, S, D), 3.0), rand_bits(rng, (1, 2, S, D)), rand_bits(rng, (1, 2, S, D))
    blocks = [(0, h, a) for h in range(4) for a in range(S // blk)]
    o1, lse1, executed = oracle.alg1_blocks(p, q, k, v, blocks)
    o2, lse2 = oracle.rows(p, q, k, v, oracle.steel_oracle.all_rows(p))
    assert np.allclose(o1.reshape(-1, D), o2, atol=1e-12)
    assert np.allclose(lse1.ravel(), lse2, atol=1e-12)
    # a partial far-left window tile masks whole rows while the running max is still -inf
    if flags & WINDOW and window % blk == 0:
        w = window // blk
        assert oracle.classify(p, 0, w + 1, 1) == 2 and not oracle.allowed(p, 0, (w + 1) * blk + blk - 1, blk + blk - 1)


def test_one_visible_key_returns_v_exactly():
    rng = np.random.default_rng(4)
    S, D = 32, 16
    p = make_problem(1, 2, 1, S, S, D, CAUSAL, 8)
    q, k, v = rand_bits(rng, (1, 2, S, D)), rand_bits(rng, (1, 1, S, D)), rand_bits(rng, (1, 1, S, D))
    o, lse = oracle.rows(p, q, k, v, [(0, 0, 0), (0, 1, 0)])
    vf, qf, kf = (inputs.bf16_bits_to_f64(x) for x in (v, q, k))
    for r, h in enumerate((0, 1)):
        assert np.array_equal(o[r], vf[0, 0, 0])
        assert lse[r] == pytest.approx(p.c.scale * float(qf[0, h, 0] @ kf[0, 0, 0]), abs=1e-13)
    # one key with a dominating score: O -> V_j, LSE -> s_ij
    u = np.zeros(D, dtype=np.float32)
    u[3] = 1.0
    kk = np.zeros((1, 1, S, D), dtype=np.float32)
    kk[0, 0, 17] = 64.0 * u
    qq = np.broadcast_to(64.0 * u, (1, 1, S, D)).copy()
    p1 = make_problem(1, 1, 1, S, S, D, 0, 8, scale=1.0)
    o, lse = oracle.rows(p1, inputs.f32_to_bf16_bits(qq), inputs.f32_to_bf16_bits(kk), v,
                         oracle.steel_oracle.all_rows(p1))
    assert np.allclose(o, vf[0, 0, 17][None, :], atol=1e-300, rtol=1e-15)
    assert np.allclose(lse, 4096.0, atol=1e-9)


@pytest.mark.parametrize("flags,window,blk", [(CAUSAL, 0, 8), (CAUSAL | WINDOW, 16, 8),
                                              (CAUSAL | WINDOW, 5, 8), (CAUSAL | BITMAP, 0, 8)])
def test_zero_queries_give_uniform_average(flags, window, blk):
    """Q = 0 => P uniform over visible keys: O_i = mean of visible V rows, LSE_i = ln n_i,
    with n_i = i + 1 (causal), min(i + 1, W) (window), a popcount-derived count (bitmap)."""
    rng = np.random.default_rng(8)
    S, D, H = 64, 8, 2
    T = S // blk
    bitmap = random_bitmap(rng, H, T, T, 0.5) if flags & BITMAP else None
    p = make_problem(1, H, H, S, S, D, flags, blk, window, bitmap)
    q = np.zeros((1, H, S, D), dtype=np.uint16)
    k, v = rand_bits(rng, (1, H, S, D)), rand_bits(rng, (1, H, S, D))
    vf = inputs.bf16_bits_to_f64(v)
    o, lse = oracle.rows(p, q, k, v, oracle.steel_oracle.all_rows(p))
    o, lse = o.reshape(H, S, D), lse.reshape(H, S)
    for h in range(H):
        for i in range(S):
            if flags & BITMAP:
                vis = [j for j in range(i + 1)
                       if (int(bitmap[h, i // blk, (j // blk) >> 5]) >> ((j // blk) & 31)) & 1]
                full_blocks = bin(int(bitmap[h, i // blk, 0]) & ((1 << (i // blk)) - 1)).count("1")
                assert len(vis) == full_blocks * blk + (i % blk) + 1
            elif flags & WINDOW:
                vis = list(range(max(0, i - window + 1), i + 1))
                assert len(vis) == min(i + 1, window)
            else:
                vis = list(range(i + 1))
            assert lse[h, i] == pytest.approx(np.log(len(vis)), abs=1e-12)
            assert np.allclose(o[h, i], vf[0, h, vis].mean(axis=0), atol=1e-12)


def test_invariances():
    rng = np.random.default_rng(9)
    S, D = 40, 16
    p = make_problem(1, 2, 2, S, S, D, CAUSAL, 8)
    q, k, v = (rand_bits(rng, (1, 2, S, D)) for _ in range(3))
    rows = oracle.steel_oracle.all_rows(p)
    o, lse = oracle.rows(p, q, k, v, rows)
    # constant V => constant O
    vc = np.broadcast_to(inputs.f32_to_bf16_bits(np.float32([1.5])), v.shape).copy()
    oc, _ = oracle.rows(p, q, k, vc, rows)
    assert np.allclose(oc, 1.5, atol=1e-13)
    # adding a vector u to every key leaves O unchanged and shifts LSE by scale * q.u
    kf = inputs.bf16_bits_to_f64(k)
    u = np.zeros(D)
    u[:4] = [2.0, -4.0, 8.0, 1.0]          # exactly representable, keeps k + u in bf16 range
    ku = kf.copy()
    ku = np.round(ku * 8) / 8 + u          # keys on a 1/8 grid stay exact after the shift
    k8 = inputs.f32_to_bf16_bits((np.round(kf * 8) / 8).astype(np.float32))
    kus = inputs.f32_to_bf16_bits(ku.astype(np.float32))
    assert np.array_equal(inputs.bf16_bits_to_f64(kus), ku)
    o8, lse8 = oracle.rows(p, q, k8, v, rows)
    ou, lseu = oracle.rows(p, q, kus, v, rows)
    qf = inputs.bf16_bits_to_f64(q).reshape(-1, D)
    assert np.allclose(ou, o8, atol=1e-11)
    assert np.allclose(lseu - lse8, p.c.scale * (qf @ u), atol=1e-11)
    # scaling Q by a power of two == scaling `scale`
    q2 = inputs.f32_to_bf16_bits((inputs.bf16_bits_to_f64(q) * 2.0).astype(np.float32))
    p2 = make_problem(1, 2, 2, S, S, D, CAUSAL, 8, scale=p.c.scale * 2.0)
    oa, la = oracle.rows(p, q2, k, v, rows)
    ob, lb = oracle.rows(p2, q, k, v, rows)
    assert np.allclose(oa, ob, atol=1e-13) and np.allclose(la, lb, atol=1e-12)
    # dense mask: a joint permutation of (K, V) rows leaves O and LSE unchanged
    pd = make_problem(1, 2, 2, S, S, D, 0, 8)
    perm = rng.permutation(S)
    o0, l0 = oracle.rows(pd, q, k, v, rows)
    o1, l1 = oracle.rows(pd, q, k[:, :, perm], v[:, :, perm], rows)
    assert np.allclose(o0, o1, atol=1e-13) and np.allclose(l0, l1, atol=1e-12)
    assert not np.allclose(o, o0)


def test_gqa_equals_repeated_mha():
    rng = np.random.default_rng(10)
    S, D = 32, 8
    q, k, v = rand_bits(rng, (2, 8, S, D)), rand_bits(rng, (2, 2, S, D)), rand_bits(rng, (2, 2, S, D))
    pg = make_problem(2, 8, 2, S, S, D, CAUSAL | WINDOW, 8, 12)
    pm = make_problem(2, 8, 8, S, S, D, CAUSAL | WINDOW, 8, 12)
    og, lg = oracle.rows(pg, q, k, v, oracle.steel_oracle.all_rows(pg))
    om, lm = oracle.rows(pm, q, np.repeat(k, 4, axis=1), np.repeat(v, 4, axis=1),
                         oracle.steel_oracle.all_rows(pm))
    assert np.array_equal(og, om) and np.array_equal(lg, lm)


@pytest.mark.parametrize("flags,window", [(0, 0), (CAUSAL, 0), (CAUSAL | WINDOW, 24),
                                          (CAUSAL | BITMAP, 0)])
def test_against_torch_sdpa_fp64(flags, window):
    """Library cross-check: torch's scaled_dot_product_attention in fp64 with a boolean mask."""
    rng = np.random.default_rng(12)
    B, Hq, Hkv, S, D, blk = 2, 4, 2, 64, 32, 16
    bitmap = random_bitmap(rng, Hq, S // blk, S // blk, 0.5) if flags & BITMAP else None
    p = make_problem(B, Hq, Hkv, S, S, D, flags, blk, window, bitmap, scale=0.2)
    q, k, v = rand_bits(rng, (B, Hq, S, D)), rand_bits(rng, (B, Hkv, S, D)), rand_bits(rng, (B, Hkv, S, D))
    mask = torch.from_numpy(dense_mask(flags, S, S, blk, blk, window, bitmap, Hq))
    tq, tk, tv = (torch.from_numpy(inputs.bf16_bits_to_f64(x)) for x in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(
        tq, tk.repeat_interleave(Hq // Hkv, 1), tv.repeat_interleave(Hq // Hkv, 1),
        attn_mask=mask[None], scale=0.2)
    o, _ = oracle.rows(p, q, k, v, oracle.steel_oracle.all_rows(p))
    assert np.allclose(o.reshape(B, Hq, S, D), ref.numpy(), atol=1e-12)


def _golden_tile_counts():
    path = os.path.join(os.path.dirname(__file__), "golden", "tile_counts.txt")
    out = {}
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        name, heads, t, wb, kept, partial = line.split()
        out[name] = tuple(int(x) for x in (heads, t, wb, kept, partial))
    return out


def test_classification_against_closed_form_counts():
    """Brute-force tile classes reproduce the closed-form counts of the graded workloads
    (small blocks stand in for 128-token blocks: the counts depend only on T and W/block)."""
    golden = _golden_tile_counts()
    for name, (heads, t, wb, kept, partial) in golden.items():
        w = inputs.workload(name)
        assert (w.heads_q, w.tiles) == (heads, t)
        assert kept == heads * sum(min(i, wb if wb else i) + 1 for i in range(t))
        if t > 128:
            continue
        blk = 4
        p = oracle.OracleProblem(1, 1, 1, t * blk, t * blk, 8, 1.0, w.flags, blk, blk, wb * blk)
        counts = oracle.count_tiles(p)
        assert counts[0, 0] * heads == kept and counts[0, 1] * heads == partial


def test_classify_cases_causal_and_window():
    blk, T = 8, 10
    p = make_problem(1, 1, 1, T * blk, T * blk, 8, CAUSAL | WINDOW, blk, 3 * blk)
    for I, J in itertools.product(range(T), range(T)):
        c = oracle.classify(p, 0, I, J)
        expect = 0 if (J > I or J < I - 3) else (2 if J in (I, I - 3) else 1)
        assert c == expect
    # a window that is not a multiple of the block: one more partial tile on the left
    p = make_problem(1, 1, 1, T * blk, T * blk, 8, CAUSAL | WINDOW, blk, 3 * blk + 1)
    assert oracle.classify(p, 0, 6, 3) == 2 and oracle.classify(p, 0, 6, 4) == 1
    assert oracle.classify(p, 0, 6, 2) == 0
