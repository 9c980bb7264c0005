"""SimScore (Sec. 3.2, Eq. 1) through the C ABI against the oracle's definition."""
import numpy as np
import pytest
import torch

import synthetic_inputs as S
from oracle import swiftkv_oracle as O
from helpers import oracle_config, oracle_weights, to_np

pytestmark = pytest.mark.gpu

MID = S.ModelShape(1024, 512, 4, 8, 2, 128, 1024, 500000.0, 1e-5, "mid")
SIX = S.ModelShape(512, 256, 6, 8, 2, 32, 688, 10000.0, 1e-5, "tiny-6-layers")


@pytest.mark.parametrize("shape,dtype,bar", [(S.TINY, torch.float32, 1e-5), (SIX, torch.float32, 1e-5), (MID, torch.bfloat16, 2e-3)])
def test_simscore_against_oracle(shape, dtype, bar):
    import paper_2410_03960_b200 as P
    seed, lens = 31, [150, 1, 77]
    w = S.make_weights(shape, seed, dtype, "cuda")
    tok = S.make_prompts(seed, lens, shape.vocab)
    model = P.SwiftKVModel(shape, w, dtype, sum(lens), len(lens), shape.n_layers, 1)
    score, sim = model.simscore(tok, lens)
    model.status()
    xs = O.layer_inputs(oracle_config(shape), oracle_weights(w), tok.numpy(), lens)
    want = O.simscore(xs)
    assert np.max(np.abs(to_np(score) - want)) <= bar, (to_np(score), want)
    L = shape.n_layers
    sim = to_np(sim)
    for a in range(L):
        for b in range(L):
            ref = 1.0 if a == b else O.similarity(xs[a], xs[b])
            assert abs(sim[a, b] - ref) <= bar, (a, b)
    # the full-depth prefill ran as a side effect: its logits are those of the unmodified model
    base = O.baseline(oracle_config(shape), oracle_weights(w), tok.numpy(), lens)
    assert np.max(np.abs(to_np(model.first_logits()) - base["logits"])) <= (1e-3 if dtype == torch.float32 else 0.1)
    model.close()


def test_simscore_is_one_when_every_layer_is_the_identity():
    """W_O = W_down = 0: all layer inputs are equal, so every SimScore is exactly 1 (the paper's premise made exact)."""
    import paper_2410_03960_b200 as P
    shape, lens = S.TINY, [40, 9]
    w = S.make_weights(shape, 5, torch.float32, "cuda")
    for lw in w.layers:
        lw["wo"].zero_()
        lw["w_down"].zero_()
    model = P.SwiftKVModel(shape, w, torch.float32, sum(lens), len(lens), shape.n_layers, 1)
    score, sim = model.simscore(S.make_prompts(5, lens, shape.vocab), lens)
    assert torch.allclose(score, torch.ones_like(score), atol=1e-6) and torch.allclose(sim, torch.ones_like(sim), atol=1e-6)
    model.close()
