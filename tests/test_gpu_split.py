"""The half-pair activation format (SWIFTKV_ACT_F16_SPLIT): operands carried as hi + lo IEEE halves, multiplied in extra
tensor-core passes.  Operator level against exact fp64 products / the oracle's attention, then the whole prefill."""
import numpy as np
import pytest
import torch

import synthetic_inputs as S
from oracle import swiftkv_oracle as O
from helpers import check_prefill_against_oracle, oracle_config, oracle_weights, rel_l2, to_np

pytestmark = pytest.mark.gpu

MID = S.ModelShape(1024, 512, 4, 8, 2, 128, 1024, 500000.0, 1e-5, "mid")


@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (300, 512, 4096), (1000, 384, 1024)])
def test_gemm_with_a_half_pair_operand(M, N, K):
    """A as hi + lo halves, B as exact halves: the product keeps ~22 bits of A, so it matches the fp64 product of the
    fp32 A to ~1e-5 (what the fp32 accumulation over a long K leaves), where the single-half A gives ~1.5e-4."""
    import paper_2410_03960_b200 as P
    a = S.matrix(11, 1, M, K, torch.float32, "cuda", std=1.0)
    b = S.matrix(11, 2, N, K, torch.float16, "cuda", std=1.0)
    got = P.gemm_tc_split(a, b)
    torch.cuda.synchronize()
    ref = a.double().cpu().numpy() @ b.double().cpu().numpy().T
    single = a.half().double().cpu().numpy() @ b.double().cpu().numpy().T
    e_pair, e_single = rel_l2(to_np(got), ref), rel_l2(single, ref)
    assert e_pair < 3e-5, e_pair      # (fp32 accumulation inside the tensor core over K = 4096 leaves ~1e-5)
    assert e_single > 5 * e_pair


@pytest.mark.parametrize("lens,n_q,n_kv", [([1, 127, 129, 300], 4, 2), ([1000, 260], 8, 2)])
@pytest.mark.parametrize("out_split", [False, True])
def test_attention_with_half_pair_scores(lens, n_q, n_kv, out_split):
    """q and K scaled so that the softmax is sharp (score std ~4): with single halves the 2^-12 rounding of q and K
    moves the probabilities by ~1e-3; the three-pass scores remove that, and the pair output removes the output
    rounding as well.  Reference: the oracle's causal attention on the exact fp32 q, K and the half V."""
    import paper_2410_03960_b200 as P
    hd, T = 128, sum(lens)
    q = S.matrix(12, 1, T, n_q * hd, torch.float32, "cuda", std=2.0).view(T, n_q, hd)
    k = S.matrix(12, 2, T, n_kv * hd, torch.float32, "cuda", std=2.0).view(T, n_kv, hd)
    v = S.matrix(12, 3, T, n_kv * hd, torch.float16, "cuda", std=1.0).view(T, n_kv, hd)
    got = P.attention_prefill_split(q, k, v, lens, out_split=out_split)
    plain = P.attention_prefill(q.half(), k.half(), v, lens, use_tensor_cores=True)
    torch.cuda.synchronize()
    assert torch.isfinite(got).all()
    off, e_pair, e_plain = 0, 0.0, 0.0
    for n in lens:
        ref = O.causal_attention(to_np(q[off:off + n]), to_np(k[off:off + n]), to_np(v[off:off + n]))
        e_pair = max(e_pair, rel_l2(to_np(got[off:off + n]), ref))
        e_plain = max(e_plain, rel_l2(to_np(plain[off:off + n]), ref))
        off += n
    print("attention rel-L2 against the oracle: half pairs", e_pair, "plain halves", e_plain)
    # what is left: P as a half (2^-12, averaged over the keys) and -- without the pair output -- the output's own rounding
    assert e_pair < (2.5e-4 if out_split else 4e-4), (e_pair, e_plain)      # measured 1.0e-4 .. 2.6e-4; plain halves 6.5e-4
    assert e_plain > 2 * e_pair, (e_pair, e_plain)


@pytest.mark.parametrize("mask", [1, 2, 4, 8, 16, 7, 31])
def test_prefill_with_half_pairs_every_operand(mask):
    """The whole prefill with each operand class as half pairs, alone and together: same bars as every bf16 model, and never
    worse than plain halves by more than noise."""
    import paper_2410_03960_b200 as P
    lens, l, g = [300, 77, 129, 1], 2, 1
    w = S.make_weights(MID, 2, torch.bfloat16, "cuda")
    tok = S.make_prompts(2, lens, MID.vocab)
    ref = O.swiftkv(oracle_config(MID), oracle_weights(w), tok.numpy(), lens, l, g)
    model = P.SwiftKVModel(MID, w, torch.bfloat16, sum(lens), len(lens), l, g)
    model.set_activation_format(P.ACT_F16_SPLIT)
    model.set_split_mask(mask)
    model.prefill(tok, lens, l, g)
    model.status()
    res = check_prefill_against_oracle(model, ref, MID.n_layers, 2e-2, 2e-2, 0.1)
    print("split mask", mask, res)
    model.close()
