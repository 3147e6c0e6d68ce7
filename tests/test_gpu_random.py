"""Seeded random problem shapes (batch, GQA group, ragged lengths, every mask kind, both head
dimensions, both block sizes, every placement policy and software-exponent share) through the C ABI
against the oracle, all rows."""
import numpy as np
import pytest

from paper_2607_09385_b200 import inputs

import helpers as H

pytestmark = pytest.mark.gpu
CAUSAL, WINDOW, BITMAP = inputs.MASK_CAUSAL, inputs.MASK_WINDOW, inputs.MASK_BITMAP


def random_cases(n, seed):
    rng = np.random.default_rng(seed)
    cases = []
    for k in range(n):
        hkv = int(rng.integers(1, 4))
        group = int(rng.choice([1, 2, 3, 4]))
        d = int(rng.choice([64, 128]))
        block = int(rng.choice([64, 128]))
        flags = int(rng.choice([0, CAUSAL, CAUSAL | WINDOW, WINDOW, CAUSAL | BITMAP, BITMAP]))
        seq = int(rng.integers(1, 1400))
        cases.append(dict(id=f"r{k}", B=int(rng.integers(1, 3)), Hq=hkv * group, Hkv=hkv, S=seq, D=d, block=block,
                          flags=flags, window=int(rng.integers(1, max(2, seq))), keep=float(rng.uniform(0.1, 0.9)),
                          policy=int(rng.integers(0, 3)), emu=int(rng.integers(0, 4)), seed=int(rng.integers(1, 1 << 30))))
    return cases


CASES = random_cases(24, seed=20250)


@pytest.mark.parametrize("case", CASES, ids=[c["id"] for c in CASES])
def test_random_shape_matches_oracle(case):
    w = inputs.Workload(case["id"], case["B"], case["Hq"], case["Hkv"], case["S"], case["D"], case["block"],
                        case["flags"], window=case["window"] if case["flags"] & WINDOW else 0, keep_prob=case["keep"])
    data = inputs.make_inputs(w, seed=case["seed"])
    if w.flags & BITMAP:
        t = -(-w.seq // w.block)
        # without a causal term the bitmap may have empty rows of blocks: those query rows see no key
        rng = np.random.default_rng(case["seed"])
        bits = rng.random((w.heads_q, t, ((t + 31) // 32) * 32)) < case["keep"]
        bits[:, :, t:] = False
        if w.flags & CAUSAL:
            bits[:, np.arange(t), np.arange(t)] = True
        data["bitmap"] = (bits.reshape(w.heads_q, t, -1, 32).astype(np.uint32) << np.arange(32, dtype=np.uint32)).sum(
            axis=3, dtype=np.uint32)
    attn, o, lse = H.run_gpu(w, data, policy=case["policy"], exp_emulation=case["emu"])
    H.assert_parity(w, data, o, lse, H.all_rows(w))
    attn.close()
