"""The benchmark's two arms describe the workload with the same `config` object: the CPU-oracle arm
derives the kept-tile count from the mask's definition alone (closed forms, the bitmap's population
count or the oracle's brute-force count), the CUDA arm from the planner.  Both must agree."""
import importlib.util
import os

import numpy as np
import pytest

from paper_2607_09385_b200 import binding as B
from paper_2607_09385_b200 import inputs


@pytest.fixture(scope="module")
def bench(repo_root):
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(repo_root, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def planner_counts(w, bitmap):
    p, keep = B.make_params(w.batch, w.heads_q, w.heads_kv, w.seq, w.seq, w.head_dim, w.scale, w.flags,
                            w.block, w.block, w.window, bitmap)
    st, stats, _ = B.steel_attn_plan_host(p)
    assert st == B.STEEL_OK
    return stats["kept_tiles"], stats["partial_tiles"], stats["effective_flop"]


@pytest.mark.parametrize("name", ["c1", "c2", "c3", "c4", "c5", "bert_h12_d64_s512", "llama1b_h32_d64_s2048"])
def test_definition_counts_match_the_planner(bench, name):
    w = inputs.workload(name)
    bitmap = inputs.block_bitmap(w.heads_q, w.tiles, w.tiles, w.keep_prob) if w.flags & inputs.MASK_BITMAP else None
    kept, partial = bench.tile_counts_from_definition(w, bitmap)
    kept_p, partial_p, flop_p = planner_counts(w, bitmap)
    assert (kept, partial) == (kept_p, partial_p)
    cfg = bench.make_config(w, kept, partial, 1)
    assert cfg["effective_flop"] == flop_p and cfg["kept_tiles"] == kept_p


def test_definition_counts_fall_back_to_the_oracle_on_unaligned_shapes(bench):
    w = inputs.Workload("ragged", 1, 2, 1, 1000, 64, 64, inputs.MASK_CAUSAL | inputs.MASK_WINDOW, window=300)
    kept, partial = bench.tile_counts_from_definition(w, None)
    assert (kept, partial) == planner_counts(w, None)[:2]
    # a bitmap with bits above the diagonal under a causal mask: the population count would over-count
    w = inputs.Workload("bitmap_dense", 1, 2, 2, 512, 64, 64, inputs.MASK_CAUSAL | inputs.MASK_BITMAP)
    bitmap = np.full((2, 8, 1), 0xFF, dtype=np.uint32)
    kept, partial = bench.tile_counts_from_definition(w, bitmap)
    assert (kept, partial) == planner_counts(w, bitmap)[:2] == (2 * 36, 2 * 8)
