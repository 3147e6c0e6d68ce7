"""Host planner (tile classification, work lists, CTA assignment) against the oracle's brute-force
three-case classification and the closed-form tile counts.  CPU only."""
import itertools
import os

import numpy as np
import pytest

import oracle
from paper_2607_09385_b200 import binding as B
from paper_2607_09385_b200 import inputs

CAUSAL, WINDOW, BITMAP = inputs.MASK_CAUSAL, inputs.MASK_WINDOW, inputs.MASK_BITMAP


def host_plan(batch, hq, hkv, sq, skv, d, flags, block=128, window=0, bitmap=None, tiles=True, policy=0):
    p, keep = B.make_params(batch, hq, hkv, sq, skv, d, 0.1, flags, block, block, window, bitmap, policy)
    st, stats, recs = B.steel_attn_plan_host(p, want_tiles=tiles)
    assert st == B.STEEL_OK
    return stats, recs


def golden():
    path = os.path.join(os.path.dirname(__file__), "golden", "tile_counts.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    return {r[0]: tuple(int(x) for x in r[1:]) for r in rows}


def test_tile_counts_of_the_graded_workloads():
    g = golden()
    for name, (heads, t, wb, kept, partial) in g.items():
        w = inputs.workload(name)
        stats, _ = host_plan(w.batch, w.heads_q, w.heads_kv, w.seq, w.seq, w.head_dim, w.flags, w.block,
                             w.window, None, tiles=False)
        assert (stats["kept_tiles"], stats["partial_tiles"]) == (kept, partial), name
        assert stats["effective_flop"] == 4.0 * w.block * w.block * w.head_dim * kept
        if w.block == 128:
            assert stats["exec_tiles"] == kept and stats["exec_partial"] == partial
        # visible pairs in closed form: causal sum_i (i+1); window sum_i min(i+1, W)
        n = sum(min(i + 1, w.window) if w.window else i + 1 for i in range(w.seq)) if w.seq <= 16384 else \
            w.seq * (w.seq + 1) // 2
        assert stats["useful_flop"] == 4.0 * w.head_dim * n * w.heads_q
    w = inputs.workload("c4")
    bm = inputs.block_bitmap(w.heads_q, w.tiles, w.tiles, w.keep_prob)
    stats, _ = host_plan(1, w.heads_q, w.heads_kv, w.seq, w.seq, w.head_dim, w.flags, 128, 0, bm, tiles=False)
    bits = sum(bin(int(x)).count("1") for x in bm.ravel())
    assert stats["kept_tiles"] == bits == stats["exec_tiles"] and stats["partial_tiles"] == 16 * 256
    expected = 16 * (511 + 0.25 * 32385)
    assert abs(bits - expected) < 4 * np.sqrt(16 * 32385 * 0.1875)


CASES = [
    dict(hq=2, hkv=2, sq=640, skv=640, flags=CAUSAL),
    dict(hq=4, hkv=2, sq=640, skv=640, flags=CAUSAL),
    dict(hq=3, hkv=1, sq=512, skv=512, flags=0),
    dict(hq=2, hkv=1, sq=1024, skv=1024, flags=CAUSAL | WINDOW, window=256),
    dict(hq=1, hkv=1, sq=1024, skv=1024, flags=CAUSAL | WINDOW, window=300),
    dict(hq=1, hkv=1, sq=1024, skv=1024, flags=CAUSAL | WINDOW, window=1),
    dict(hq=2, hkv=2, sq=768, skv=768, flags=WINDOW, window=200),
    dict(hq=1, hkv=1, sq=1000, skv=1000, flags=CAUSAL),
    dict(hq=1, hkv=1, sq=200, skv=456, flags=CAUSAL),
    dict(hq=1, hkv=1, sq=456, skv=200, flags=CAUSAL),
    dict(hq=4, hkv=4, sq=1024, skv=1024, flags=CAUSAL | BITMAP, keep=0.3),
    dict(hq=4, hkv=2, sq=1024, skv=1024, flags=BITMAP, keep=0.5),
    dict(hq=2, hkv=2, sq=1024, skv=1024, flags=CAUSAL | BITMAP, block=64, keep=0.4),
    dict(hq=2, hkv=1, sq=960, skv=960, flags=BITMAP | WINDOW | CAUSAL, block=64, keep=0.6, window=130),
]


@pytest.mark.parametrize("case", CASES)
def test_plan_executes_exactly_the_unmasked_tiles(case):
    """Every (head, query tile, key tile) that the brute-force classification keeps appears exactly
    once in the plan with the right partial flag; skipped tiles never appear."""
    c = dict(case)
    block = c.get("block", 128)
    rng = np.random.default_rng(4)
    bitmap = None
    if c["flags"] & BITMAP:
        tq, tkv = -(-c["sq"] // block), -(-c["skv"] // block)
        bits = rng.random((c["hq"], tq, tkv)) < c["keep"]
        bitmap = np.zeros((c["hq"], tq, (tkv + 31) // 32), np.uint32)
        for h, a, b in zip(*np.nonzero(bits)):
            bitmap[h, a, b >> 5] |= np.uint32(1 << (b & 31))
    for batch in (1, 2):
        stats, recs = host_plan(batch, c["hq"], c["hkv"], c["sq"], c["skv"], 128, c["flags"], block,
                                c.get("window", 0), bitmap)
        assert stats["exec_tiles"] == len(recs)
        seen = {}
        for item, b, h, I, J, fl in recs:
            key = (b, h, I, J)
            assert key not in seen
            seen[key] = fl
        # the oracle classifies 128-token tiles by brute force over every (i, j) pair; with 64-token
        # bitmap blocks the predicate already carries the sub-block bits
        p128 = oracle.OracleProblem(1, c["hq"], c["hkv"], c["sq"], c["skv"], 8, 1.0, c["flags"], block, block,
                                    c.get("window", 0), bitmap)
        tq128, tkv128 = -(-c["sq"] // 128), -(-c["skv"] // 128)
        for h, I, J in itertools.product(range(c["hq"]), range(tq128), range(tkv128)):
            vis = tot = 0
            for i in range(I * 128, min(I * 128 + 128, c["sq"])):
                row = [oracle.allowed(p128, h, i, j) for j in range(J * 128, min(J * 128 + 128, c["skv"]))]
                vis += sum(row)
                tot += len(row)
            for b in range(batch):
                if vis == 0:
                    assert (b, h, I, J) not in seen
                else:
                    assert (b, h, I, J) in seen
                    partial = bool(seen[(b, h, I, J)] & 1)
                    ragged_keys = min(J * 128 + 128, c["skv"]) - J * 128 < 128
                    assert partial == (vis < tot or ragged_keys), (h, I, J, vis, tot)
        # block-granular statistics against the oracle's brute-force counts
        counts = oracle.count_tiles(p128)
        assert stats["kept_tiles"] == batch * counts[:, 0].sum()
        assert stats["partial_tiles"] == batch * counts[:, 1].sum()


def test_sub_block_bits_for_64_token_blocks():
    bitmap = np.zeros((1, 4, 1), np.uint32)
    bitmap[0, 0, 0] = 0b0001      # block row 0: key block 0
    bitmap[0, 1, 0] = 0b0010      # block row 1: key block 1
    bitmap[0, 2, 0] = 0b0100      # block row 2: key block 2
    bitmap[0, 3, 0] = 0b0011      # block row 3: key blocks 0, 1
    stats, recs = host_plan(1, 1, 1, 256, 256, 128, BITMAP, 64, 0, bitmap)
    by_tile = {(I, J): fl for _, _, _, I, J, fl in recs}
    assert set(by_tile) == {(0, 0), (1, 0), (1, 1)}
    assert by_tile[(0, 0)] >> 4 == 0b1001 and by_tile[(0, 0)] & 1      # TL and BR enabled
    assert by_tile[(1, 1)] >> 4 == 0b0001 and by_tile[(1, 0)] >> 4 == 0b1100
    assert stats["kept_tiles"] == 5 and stats["exec_tiles"] == 3


def test_shared_loads_and_item_structure():
    # MHA causal: adjacent query tiles share every key tile but the last
    stats, recs = host_plan(1, 1, 1, 1024, 1024, 128, CAUSAL)
    assert stats["work_items"] == 4 and stats["exec_tiles"] == 36
    assert stats["kv_tile_loads"] == 36 - (1 + 3 + 5 + 7)
    shared = [r for r in recs if r[5] & 2]
    assert all(r[3] % 2 == 1 for r in shared)           # the shared flag sits on the second slot
    # GQA: two heads of a group walk identical ranges, everything is shared
    stats, _ = host_plan(1, 4, 2, 1024, 1024, 128, CAUSAL)
    assert stats["kv_tile_loads"] * 2 == stats["exec_tiles"]
    assert stats["steps"] == stats["kv_tile_loads"]


def test_balance_and_policies():
    w = inputs.workload("c2")
    stats, recs0 = host_plan(1, w.heads_q, w.heads_kv, w.seq, w.seq, 128, w.flags, tiles=True)
    assert stats["grid"] == 148
    assert stats["max_cta_steps"] <= 1.08 * stats["steps"] / 148 + 2
    key = lambda r: {tuple(x[1:5]) for x in r}
    by_policy = {0: stats}
    for policy in (1, 2):
        by_policy[policy], recs = host_plan(1, w.heads_q, w.heads_kv, w.seq, w.seq, 128, w.flags, tiles=True,
                                            policy=policy)
        assert key(recs0) == key(recs) and by_policy[policy]["exec_tiles"] == stats["exec_tiles"]
    # contiguous chunks (uniform placement) are the most unbalanced under a causal mask, dealing
    # consecutive tiles round-robin (sparsity-aware placement) is better, longest-first is best
    assert by_policy[1]["max_cta_steps"] > by_policy[2]["max_cta_steps"] > by_policy[0]["max_cta_steps"]
    bad, _ = B.make_params(1, 2, 2, 256, 256, 128, 0.1, w.flags, policy=3)
    assert B.steel_attn_plan_host(bad)[0] == B.STEEL_ERR_INVALID_ARG


def test_makespan_model_of_uniform_vs_interleaved_placement():
    """With P synchronised pipelines and causal rows of i + 1 tiles, contiguous chunks cost
    sum over waves of the slowest pipeline; interleaving consecutive rows equalises them.  The
    ratio tends to P / (2P - 1): an upper bound consistent with the 38 % the paper reports for
    its sparsity-aware placement."""
    for P, T in ((5, 100), (10, 200), (10, 1000)):
        chunk = T // P
        uniform = sum(max(p * chunk + r + 1 for p in range(P)) for r in range(chunk))
        interleaved = sum(max(wv * P + p + 1 for p in range(P)) for wv in range(chunk))
        assert uniform == chunk * (P - 1) * chunk + chunk * (chunk + 1) // 2
        assert interleaved == P * chunk * (chunk + 1) // 2
        assert abs(interleaved / uniform - P / (2 * P - 1)) < 0.03
