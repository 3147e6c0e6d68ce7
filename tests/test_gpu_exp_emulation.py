"""Software exponent (the counterpart of the lookup-table exponent the paper uses on the NPU
generation without an exponent unit, Sec. "Comparison with State-of-the-Art on NPU"): kernel builds
that evaluate 12.5 %, 25 % or 50 % of the Second Stage's exponentials by a cubic polynomial on the FMA
pipe, selected at create time, against the fp64 oracle within the stated tolerances."""
import numpy as np
import pytest
import torch

from paper_2607_09385_b200 import binding, inputs

import helpers as H

pytestmark = pytest.mark.gpu
CAUSAL, WINDOW, BITMAP = inputs.MASK_CAUSAL, inputs.MASK_WINDOW, inputs.MASK_BITMAP


@pytest.mark.parametrize("emu", [1, 2, 3])
@pytest.mark.parametrize("name", ["c2", "llama1b_h32_d64_s2048"])
def test_emulated_exponent_matches_oracle(name, emu):
    w = inputs.workload(name)
    data = inputs.make_inputs(w, seed=7)
    attn, o, lse = H.run_gpu(w, data, exp_emulation=emu)
    rows = H.sampled_rows(w, range(0, w.heads_q, 5), 1, 1024)
    mx, mean, el = H.assert_parity(w, data, o, lse, rows)
    # the polynomial's 7.5e-5 relative error must stay far inside the LSE tolerance
    assert el <= 2e-4
    attn.close()


@pytest.mark.parametrize("emu", [1, 3])
def test_emulated_exponent_on_masked_tiles_and_empty_rows(emu):
    """Partial tiles put -inf scores through the polynomial path: masked keys must still carry no
    weight, rows without any visible key must end as O = 0 and LSE = -inf exactly."""
    import oracle
    # sliding window that is not a multiple of the tile, with a ragged tail
    w = inputs.Workload("emu_window", 1, 2, 2, 1000, 128, 128, CAUSAL | WINDOW, window=300)
    data = inputs.make_inputs(w, seed=11)
    attn, o, lse = H.run_gpu(w, data, exp_emulation=emu)
    H.assert_parity(w, data, o, lse, H.all_rows(w))
    attn.close()
    # 64-token bitmap blocks: executed 128-tiles contain disabled sub-blocks
    w = inputs.Workload("emu_bitmap64", 1, 2, 2, 1024, 64, 64, CAUSAL | BITMAP, keep_prob=0.4)
    data = inputs.make_inputs(w, seed=12)
    data["bitmap"] = inputs.block_bitmap(w.heads_q, 16, 16, 0.4, seed=5)
    attn, o, lse = H.run_gpu(w, data, exp_emulation=emu)
    H.assert_parity(w, data, o, lse, H.all_rows(w))
    attn.close()
    # more queries than keys under a bottom-right aligned causal mask: the first rows see no key
    rng = np.random.default_rng(3)
    sq, skv, D = 456, 200, 128
    q = inputs.f32_to_bf16_bits(rng.standard_normal((1, 2, sq, D)).astype(np.float32))
    k = inputs.f32_to_bf16_bits(rng.standard_normal((1, 1, skv, D)).astype(np.float32))
    v = inputs.f32_to_bf16_bits(rng.standard_normal((1, 1, skv, D)).astype(np.float32))
    attn = binding.SteelAttention(1, 2, 1, sq, skv, D, 0.1, CAUSAL, exp_emulation=emu)
    og, lg = attn.run(H.to_device(q), H.to_device(k), H.to_device(v))
    assert attn.last_status() == binding.STEEL_OK
    p = oracle.OracleProblem(1, 2, 1, sq, skv, D, 0.1, CAUSAL)
    o_ref, lse_ref = oracle.rows(p, q, k, v, oracle.steel_oracle.all_rows(p))
    og, lg = og.float().cpu().numpy().reshape(-1, D), lg.cpu().numpy().reshape(-1)
    fin = np.isfinite(lse_ref)
    assert np.array_equal(np.isfinite(lg), fin) and np.all(np.isneginf(lg[~fin])) and np.all(og[~fin] == 0)
    assert np.abs(og - o_ref).max() <= H.TOL_O_MAX and np.abs(lg[fin] - lse_ref[fin]).max() <= H.TOL_LSE
    attn.close()


def test_emulation_changes_the_result_only_slightly():
    """Same inputs with and without emulation: different arithmetic (not bit-identical), same answer."""
    w = inputs.Workload("emu_diff", 1, 4, 4, 2048, 128, 128, CAUSAL)
    data = inputs.make_inputs(w, seed=13)
    attn0, o0, lse0 = H.run_gpu(w, data)
    attn3, o3, lse3 = H.run_gpu(w, data, exp_emulation=3)
    assert not torch.equal(lse0, lse3)
    assert (lse0 - lse3).abs().max().item() <= 2e-4 and (o0.float() - o3.float()).abs().max().item() <= 2e-2
    attn0.close()
    attn3.close()
