"""End-to-end parity of the CUDA prefill (through the C ABI) with the CPU oracle: every layer's K / V cache and
the first-token logits, element by element, on the same seeded inputs.

Bars: fp32 model -- rel-L2 <= 1e-4 on every tensor; bf16 model -- rel-L2 <= 2e-2 per tensor and max-abs logit
error <= 0.1 (bf16 storage between kernels, fp32 accumulation and fp32 residual stream).
"""
import os

import numpy as np
import pytest
import torch

import synthetic_inputs as S
from oracle import swiftkv_oracle as O
from helpers import check_prefill_against_oracle, oracle_config, oracle_weights, rel_l2, to_np

pytestmark = pytest.mark.gpu

# a shape every tensor-core kernel tiles (K % 64 == 0, N % 256 == 0, head_dim 128) yet small enough for the oracle
MID = S.ModelShape(1024, 512, 4, 8, 2, 128, 1024, 500000.0, 1e-5, "mid")
# Llama-3.1-8B widths with a reduced depth (the oracle stays within a minute)
W8B_4L = S.ModelShape(128256, 4096, 4, 32, 8, 128, 14336, 500000.0, 1e-5, "8b-width-4-layers")


def _run(shape, dtype, seed, lens, l, g, max_tokens=None, kernel_mask=None, act_format=None):
    import paper_2410_03960_b200 as P
    w = S.make_weights(shape, seed, dtype, "cuda")
    tok = S.make_prompts(seed, lens, shape.vocab)
    model = P.SwiftKVModel(shape, w, dtype, max_tokens or sum(lens), len(lens), l, g)
    if kernel_mask is not None:
        model.set_kernel_mask(kernel_mask)
    if act_format is not None:
        model.set_activation_format(act_format)
    model.prefill(tok, lens, l, g)
    model.status()
    ref = O.swiftkv(oracle_config(shape), oracle_weights(w), tok.numpy(), lens, l, g)
    return model, ref, w, tok


@pytest.mark.parametrize("l,g", [(2, 1), (4, 1), (1, 1), (1, 2), (2, 2), (3, 1), (1, 3)])
def test_config1_fp32(l, g):
    """Config 1: tiny Llama-style decoder, fp32 weights, prompts of 128 and 96 tokens (l = 2, g = 1 is the
    named point; l = 4 is the unmodified model; the rest cover AcrossKV incl. a short last group)."""
    model, ref, _, _ = _run(S.TINY, torch.float32, 0, [128, 96], l, g)
    check_prefill_against_oracle(model, ref, S.TINY.n_layers, 1e-4, 1e-4, 1e-3)


@pytest.mark.parametrize("act", [0, 1])
@pytest.mark.parametrize("l,g", [(2, 1), (4, 1), (1, 2)])
def test_config1_bf16(l, g, act):
    model, ref, _, _ = _run(S.TINY, torch.bfloat16, 0, [128, 96], l, g, act_format=act)
    check_prefill_against_oracle(model, ref, S.TINY.n_layers, 2e-2, 2e-2, 0.1)


@pytest.mark.parametrize("lens", [[1], [1, 1, 1], [257, 1, 31, 128, 3]])
def test_degenerate_and_ragged_batches_fp32(lens):
    model, ref, _, _ = _run(S.TINY, torch.float32, 7, lens, 2, 1)
    check_prefill_against_oracle(model, ref, S.TINY.n_layers, 1e-4, 1e-4, 1e-3)


def test_more_prompts_than_one_tail_pass():
    lens = [3, 9, 1, 17, 5, 2, 8, 11, 4, 6, 7]       # 11 prompts: the last-token path runs in two passes of <= 8 rows
    model, ref, _, _ = _run(S.TINY, torch.float32, 8, lens, 2, 2)
    check_prefill_against_oracle(model, ref, S.TINY.n_layers, 1e-4, 1e-4, 1e-3)


@pytest.mark.parametrize("l,g", [(2, 1), (4, 1), (1, 2), (2, 2)])
@pytest.mark.parametrize("mask,act", [(83, 1), (83, 0), (64, 1), (19, 1), (19, 0), (3, 1), (3, 0), (0, 1), (0, 0), (1, 1), (2, 1)])
def test_mid_shape_bf16_tensor_core_and_simt_paths(l, g, mask, act):
    """The same model through the tcgen05 kernels (mask 3; mask 19: attention as persistent CTAs walking a host-balanced
    work list; mask 83: plus the last-token path as one persistent launch, mask 64: that launch after SIMT kernels), the SIMT
    kernels (mask 0) and the two mixtures, with
    half (act 1) and bfloat16 (act 0) activations; several row tiles and a ragged tail (T = 507), prompts of 1 and
    129 tokens included."""
    lens = [300, 77, 129, 1]
    model, ref, _, _ = _run(MID, torch.bfloat16, 2, lens, l, g, kernel_mask=mask, act_format=act)
    check_prefill_against_oracle(model, ref, MID.n_layers, 2e-2, 2e-2, 0.1)


def test_reusing_a_model_across_l_g_and_batches():
    """One model object, several prefills: a smaller later batch must not see stale state, and switching (l, g)
    re-folds the SingleInputKV weight."""
    import paper_2410_03960_b200 as P
    shape, dtype = S.TINY, torch.float32
    w = S.make_weights(shape, 4, dtype, "cuda")
    model = P.SwiftKVModel(shape, w, dtype, 300, 4, 1, 1)
    cfg, ow = oracle_config(shape), oracle_weights(w)
    for lens, l, g in [([200, 100], 2, 1), ([50], 1, 3), ([10, 20, 30, 40], 3, 1), ([64, 64], 4, 1), ([64, 64], 2, 2)]:
        tok = S.make_prompts(4 + l, lens, shape.vocab)
        model.prefill(tok, lens, l, g)
        model.status()
        ref = O.swiftkv(cfg, ow, tok.numpy(), lens, l, g)
        check_prefill_against_oracle(model, ref, shape.n_layers, 1e-4, 1e-4, 1e-3)
        # layers of one AcrossKV group alias one cache slot
        for j in range(l, shape.n_layers):
            kj, _, owner = model.kv_cache_view(j)
            assert owner == l + ((j - l) // g) * g
            assert kj.data_ptr() == model.kv_cache_view(owner)[0].data_ptr()


def test_device_resident_tokens_match_host_tokens():
    import paper_2410_03960_b200 as P
    shape, dtype, lens = S.TINY, torch.float32, [40, 25]
    w = S.make_weights(shape, 5, dtype, "cuda")
    tok = S.make_prompts(5, lens, shape.vocab)
    model = P.SwiftKVModel(shape, w, dtype, 65, 2, 2, 1)
    model.prefill(tok, lens, 2, 1)
    model.status()
    a = model.first_logits().clone()
    model.prefill_device_tokens(tok.cuda(), lens, 2, 1)
    model.status()
    assert torch.equal(a, model.first_logits())
    bad = tok.clone()
    bad[3] = shape.vocab + 5
    with pytest.raises(P.SwiftKVError) as e:
        model.prefill(bad, lens, 2, 1)
    assert e.value.code == -1
    model.prefill_device_tokens(bad.cuda(), lens, 2, 1)
    with pytest.raises(P.SwiftKVError) as e:
        model.status()
    assert e.value.code == -6
    with pytest.raises(P.SwiftKVError):
        model.prefill(tok, [40, 26], 2, 1)            # more tokens than max_tokens


def test_llama8b_width_reduced_depth():
    """Llama-3.1-8B widths (hidden 4096, 32/8 heads of 128, FFN 14336, vocab 128256), 4 layers, l = 2:
    the real GEMM / attention shapes, ragged prompts spanning several 128-row tiles."""
    lens = [333, 128, 1, 200]
    model, ref, _, _ = _run(W8B_4L, torch.bfloat16, 1, lens, 2, 1)
    res = check_prefill_against_oracle(model, ref, W8B_4L.n_layers, 2e-2, 2e-2, 0.1)
    print("8b-width parity:", res)


W70B_2L = S.ModelShape(128256, 8192, 2, 64, 8, 128, 28672, 500000.0, 1e-5, "70b-width-2-layers")


def test_llama70b_width_reduced_depth():
    """Llama-3.1-70B widths (hidden 8192, 64/8 heads of 128 -- 8 query heads per KV head --, FFN 28672), 2 layers,
    l = 1: the config-4 GEMM / attention / last-token shapes at a size the oracle finishes in seconds."""
    lens = [200, 1, 140]
    model, ref, _, _ = _run(W70B_2L, torch.bfloat16, 3, lens, 1, 1)
    res = check_prefill_against_oracle(model, ref, W70B_2L.n_layers, 2e-2, 2e-2, 0.1)
    print("70b-width parity:", res)


def _truncated(lens, factor):
    return [max(1, n // factor) for n in lens]


@pytest.mark.parametrize("cfg_name,seed,full_lens,l,g,factor", [
    ("config2", 1, S.uniform_lengths(1, 8, 2048, 8192), 16, 1, 32),      # 8 prompts U[2048, 8192], l = 16
    ("config3", 2, [16384] * 4, 24, 2, 64),                               # 4 x 16384, l = 24, AcrossKV 2
])
def test_llama8b_full_depth_truncated_prompts(cfg_name, seed, full_lens, l, g, factor):
    """The full 32-layer Llama-3.1-8B shape with the named seeds, l and g, prompts cut to their first n/factor
    tokens (ragged lengths survive): every layer's cache and the first-token logits against the oracle."""
    lens = _truncated(full_lens, factor)
    model, ref, _, _ = _run(S.LLAMA31_8B, torch.bfloat16, seed, lens, l, g)
    res = check_prefill_against_oracle(model, ref, 32, 2e-2, 2e-2, 0.1)
    print(cfg_name, "truncated parity:", lens, res)


def test_config2_full_size_prefix_parity_and_determinism():
    """The benchmark's configuration at full size (41123 tokens, l = 16): by causality the cache rows of the first P
    tokens of every prompt equal those of the truncated prompts, which the oracle can afford; the logits of the
    full-length run are checked for run-to-run bitwise determinism and finiteness."""
    import paper_2410_03960_b200 as P
    shape, seed, l, g, prefix = S.LLAMA31_8B, 1, 16, 1, 24
    lens = S.uniform_lengths(seed, 8, 2048, 8192)
    assert sum(lens) == 41123
    w = S.make_weights(shape, seed, torch.bfloat16, "cuda")
    tok = S.make_prompts(seed, lens, shape.vocab)
    model = P.SwiftKVModel(shape, w, torch.bfloat16, sum(lens), len(lens), l, g)
    model.prefill(tok, lens, l, g)
    model.status()
    logits1 = model.first_logits().clone()
    assert torch.isfinite(logits1).all()
    # the oracle on the first `prefix` tokens of every prompt
    short = [prefix] * len(lens)
    tok_short = S.make_prompts(seed, short, shape.vocab)
    ref = O.swiftkv(oracle_config(shape), oracle_weights(w), tok_short.numpy(), short, l, g)
    offs = np.concatenate([[0], np.cumsum(lens)])[:-1]
    rows = np.concatenate([np.arange(o, o + prefix) for o in offs])
    idx = torch.as_tensor(rows, device="cuda")
    for j in range(shape.n_layers):
        K, V, _ = model.kv_cache_view(j)
        assert rel_l2(to_np(K[idx]), ref["K"][j]) <= 2e-2, j
        assert rel_l2(to_np(V[idx]), ref["V"][j]) <= 2e-2, j
    model.prefill(tok, lens, l, g)
    model.status()
    assert torch.equal(logits1, model.first_logits())
    _check_full_size_samples(model, lens, to_np(logits1), "config2_full_sample.npz")


@pytest.mark.parametrize("name,seed,lens,l,g", [
    ("config3", 2, [16384] * 4, 24, 2),                 # config 3 at full size: 4 x 16384 tokens, l = 24, 2-way AcrossKV
    ("sweep-l24-g4", 4, [16384], 24, 4),                # a sweep point with 4-way AcrossKV
    ("sweep-l24-g2", 4, [16384], 24, 2),
])
def test_full_size_prefix_parity_and_determinism_with_acrosskv(name, seed, lens, l, g):
    """Full-size runs whose complete oracle evaluation is out of reach (hours of host time): by causality the cache rows of
    the first P tokens of every prompt equal those of the P-token prompts, which the oracle affords -- every layer, the
    shared AcrossKV slots included; the full-length logits must be finite and bitwise reproducible; layers of one group
    must return the same cache pointers."""
    import paper_2410_03960_b200 as P
    shape, prefix = S.LLAMA31_8B, 24
    w = S.make_weights(shape, seed, torch.bfloat16, "cuda")
    tok = S.make_prompts(seed, lens, shape.vocab)
    model = P.SwiftKVModel(shape, w, torch.bfloat16, sum(lens), len(lens), l, g)
    model.prefill(tok, lens, l, g)
    model.status()
    logits1 = model.first_logits().clone()
    assert torch.isfinite(logits1).all()
    short = [prefix] * len(lens)
    ref = O.swiftkv(oracle_config(shape), oracle_weights(w), S.make_prompts(seed, short, shape.vocab).numpy(), short, l, g)
    offs = np.concatenate([[0], np.cumsum(lens)])[:-1]
    idx = torch.as_tensor(np.concatenate([np.arange(o, o + prefix) for o in offs]), device="cuda")
    for j in range(shape.n_layers):
        K, V, owner = model.kv_cache_view(j)
        assert rel_l2(to_np(K[idx]), ref["K"][j]) <= 2e-2, (name, j)
        assert rel_l2(to_np(V[idx]), ref["V"][j]) <= 2e-2, (name, j)
        if j >= l:
            leader = l + ((j - l) // g) * g
            assert owner == leader and K.data_ptr() == model.kv_cache_view(leader)[0].data_ptr()
    model.prefill(tok, lens, l, g)
    model.status()
    assert torch.equal(logits1, model.first_logits())
    model.close()


def _check_full_size_samples(model, lens, logits, file):
    """Sampled outputs of the oracle's FULL-size run of the same workload (tests/golden/*_full_sample.npz, written by
    tests/golden/make_config2_full_sample.py from the oracle alone): first-token logits at 2048 vocabulary entries per
    prompt, the arg-max, and K / V rows of layers 1, 16, 17, 32 at four positions per prompt (first, last, two inside)
    -- the last positions and the logits depend on every token of the prompt."""
    path = os.path.join(os.path.dirname(__file__), "golden", file)
    if not os.path.exists(path):
        pytest.skip(f"tests/golden/{file} has not been generated (tests/golden/make_config2_full_sample.py)")
    gold = np.load(path)
    assert list(gold["lens"]) == list(lens)
    for b in range(len(lens)):
        got = logits[b][gold["vocab_idx"][b]]
        ref = gold["logits"][b].astype(np.float64)
        # (the norm of the sample against the sample: same 2e-2 bar as for a whole row)
        assert rel_l2(got, ref) <= 2e-2, (b, rel_l2(got, ref))
        assert np.max(np.abs(got - ref)) <= 0.1, (b, float(np.max(np.abs(got - ref))))
        # the oracle's arg-max entry: within the bar of the oracle's value, and no entry beats it by more than the bar
        assert abs(logits[b][gold["argmax"][b]] - gold["max"][b]) <= 0.1
        assert logits[b].max() <= gold["max"][b] + 0.1
        assert abs(np.linalg.norm(logits[b]) / gold["logits_norm"][b] - 1) <= 2e-2
    offs = np.concatenate([[0], np.cumsum(lens)])[:-1]
    rows = torch.as_tensor((offs[:, None] + gold["pos"]).reshape(-1), device="cuda")
    for j in (0, 15, 16, 31):
        K, V, _ = model.kv_cache_view(j)
        assert rel_l2(to_np(K[rows]), gold[f"K{j}"]) <= 2e-2, (j, rel_l2(to_np(K[rows]), gold[f"K{j}"]))
        assert rel_l2(to_np(V[rows]), gold[f"V{j}"]) <= 2e-2, (j, rel_l2(to_np(V[rows]), gold[f"V{j}"]))


def test_longest_sweep_point_65536_tokens_prefix_parity_and_determinism():
    """The largest single prompt of the sweep (65536 tokens: 512 query tiles, 64 key splits in the last-token attention):
    cache rows of the first tokens against the oracle's run of the truncated prompt (causality), finite logits,
    run-to-run bitwise determinism."""
    import paper_2410_03960_b200 as P
    shape, seed, l, g, n, prefix = S.LLAMA31_8B, 4, 16, 1, 65536, 24
    w = S.make_weights(shape, seed, torch.bfloat16, "cuda")
    tok = S.make_prompts(seed, [n], shape.vocab)
    model = P.SwiftKVModel(shape, w, torch.bfloat16, n, 1, l, g)
    model.prefill(tok, [n], l, g)
    model.status()
    logits1 = model.first_logits().clone()
    assert torch.isfinite(logits1).all()
    ref = O.swiftkv(oracle_config(shape), oracle_weights(w), tok[:prefix].numpy(), [prefix], l, g)
    for j in range(shape.n_layers):
        K, V, _ = model.kv_cache_view(j)
        assert K.shape[0] == n
        assert rel_l2(to_np(K[:prefix]), ref["K"][j]) <= 2e-2, j
        assert rel_l2(to_np(V[:prefix]), ref["V"][j]) <= 2e-2, j
        assert torch.isfinite(K[-128:].float()).all() and torch.isfinite(V[-128:].float()).all()
    model.prefill(tok, [n], l, g)
    model.status()
    assert torch.equal(logits1, model.first_logits())


@pytest.mark.parametrize("n", [4096, 16384])
def test_sweep_point_full_length_against_oracle_samples(n):
    """Points of the prompt-length sweep (one prompt of n tokens, seed 4, l = 16) at full length and depth."""
    import paper_2410_03960_b200 as P
    shape, seed, l, g, lens = S.LLAMA31_8B, 4, 16, 1, [n]
    w = S.make_weights(shape, seed, torch.bfloat16, "cuda")
    tok = S.make_prompts(seed, lens, shape.vocab)
    model = P.SwiftKVModel(shape, w, torch.bfloat16, sum(lens), len(lens), l, g)
    model.prefill(tok, lens, l, g)
    model.status()
    _check_full_size_samples(model, lens, to_np(model.first_logits()), f"sweep_n{n}_full_sample.npz")


def _check_config4_samples(model, lens, file):
    """tests/golden/config4_*_sample.npz (written by tests/golden/make_config4_sample.py from the oracle alone): the
    complete first-token logits of every prompt and K / V rows of ten layers at three positions per prompt."""
    path = os.path.join(os.path.dirname(__file__), "golden", file)
    if not os.path.exists(path):
        pytest.skip(f"tests/golden/{file} has not been generated (tests/golden/make_config4_sample.py)")
    gold = np.load(path)
    assert list(gold["lens"]) == list(lens)
    logits = to_np(model.first_logits())
    ref = gold["logits"].astype(np.float64)
    worst_rel = max(rel_l2(logits[b], ref[b]) for b in range(len(lens)))
    worst_abs = float(np.max(np.abs(logits - ref)))
    rows = torch.as_tensor(gold["rows"].astype(np.int64), device="cuda")
    worst_kv = 0.0
    for j in (0, 9, 19, 29, 39, 40, 49, 59, 69, 79):
        K, V, _ = model.kv_cache_view(j)
        ek, ev = rel_l2(to_np(K[rows]), gold[f"K{j}"]), rel_l2(to_np(V[rows]), gold[f"V{j}"])
        assert ek <= 2e-2 and ev <= 2e-2, (j, ek, ev)
        worst_kv = max(worst_kv, ek, ev)
    return {"logit_rel": worst_rel, "logit_abs": worst_abs, "kv": worst_kv}


def test_config4_llama70b_full_depth_truncated_prompts():
    """Config 4: the full 80-layer Llama-3.1-70B shape (141 GB of bf16 weights on one GPU), l = 40, the seed-3 varlen
    batch with every prompt cut to 1/64 of its length, against stored oracle outputs (all logits; sampled cache rows).
    This random-weight model has a very sharp softmax (score std 3.3), so the 2^-12 rounding of plain half operands in
    the normed hidden state, q and K grows to a max-abs logit error of 0.14 over its 80 layers; the model therefore runs
    with those operands as half pairs (SWIFTKV_ACT_F16_SPLIT), which is what the 2e-2 / 0.1 bars are asserted for."""
    import paper_2410_03960_b200 as P
    full_lens = S.lengths_to_total(3, 16384, 1024, 4096)
    lens = _truncated(full_lens, 64)
    shape, seed, l, g = S.LLAMA31_70B, 3, 40, 1
    w = S.make_weights(shape, seed, torch.bfloat16, "cuda")
    tok = S.make_prompts(seed, lens, shape.vocab)
    model = P.SwiftKVModel(shape, w, torch.bfloat16, sum(lens), len(lens), l, g)
    model.set_activation_format(P.ACT_F16_SPLIT)
    model.prefill(tok, lens, l, g)
    model.status()
    res = _check_config4_samples(model, lens, "config4_truncated_sample.npz")
    print("config4 truncated parity (half pairs):", lens, res)
    assert res["logit_rel"] <= 2e-2 and res["logit_abs"] <= 0.1, res
    # for the record: the same model with plain half operands (the default format) -- inside the relative bars, outside
    # the absolute one; printed, not asserted
    model.set_activation_format(P.ACT_F16)
    model.prefill(tok, lens, l, g)
    model.status()
    print("config4 truncated parity (plain halves):", _check_config4_samples(model, lens, "config4_truncated_sample.npz"))
    model.close()


def test_config4_full_size_against_oracle_samples():
    """Config 4 at FULL size -- the 80-layer 70B shape, the complete seed-3 batch of 7 prompts totalling 16384 tokens,
    l = 40 -- in the half-pair format, against stored outputs of the oracle's run of the same batch: all first-token
    logits of every prompt, and K / V rows of ten layers at the first, the last and an inner position of every prompt."""
    import paper_2410_03960_b200 as P
    if not os.path.exists(os.path.join(os.path.dirname(__file__), "golden", "config4_full_sample.npz")):
        pytest.skip("tests/golden/config4_full_sample.npz has not been generated (tests/golden/make_config4_sample.py --full)")
    lens = S.lengths_to_total(3, 16384, 1024, 4096)
    shape, seed, l, g = S.LLAMA31_70B, 3, 40, 1
    w = S.make_weights(shape, seed, torch.bfloat16, "cuda")
    tok = S.make_prompts(seed, lens, shape.vocab)
    model = P.SwiftKVModel(shape, w, torch.bfloat16, sum(lens), len(lens), l, g)
    model.set_activation_format(P.ACT_F16_SPLIT)
    model.prefill(tok, lens, l, g)
    model.status()
    res = _check_config4_samples(model, lens, "config4_full_sample.npz")
    print("config4 full-size parity (half pairs):", lens, res)
    assert res["logit_rel"] <= 2e-2 and res["logit_abs"] <= 0.1, res
    model.close()


def test_fused_last_token_launch_against_oracle_and_the_per_operator_path():
    """Kernel-mask bit 6: layers l+1..L and the lm_head of the continuing tokens in one persistent cooperative launch.
    Eleven prompts (two passes of at most 8 rows), ragged lengths incl. 1 token, AcrossKV groups with a short last group;
    against the oracle at the bf16 bars, against the per-operator path to fp32 summation-order noise, and bitwise
    reproducible."""
    import paper_2410_03960_b200 as P
    lens = [300, 1, 129, 77, 513, 128, 2, 255, 40, 700, 9]
    l, g = 1, 2
    w = S.make_weights(MID, 6, torch.bfloat16, "cuda")
    tok = S.make_prompts(6, lens, MID.vocab)
    ref = O.swiftkv(oracle_config(MID), oracle_weights(w), tok.numpy(), lens, l, g)
    out = {}
    for mask in (119, 55):
        model = P.SwiftKVModel(MID, w, torch.bfloat16, sum(lens), len(lens), l, g)
        assert model.set_kernel_mask(mask) == mask
        model.prefill(tok, lens, l, g)
        model.status()
        check_prefill_against_oracle(model, ref, MID.n_layers, 2e-2, 2e-2, 0.1)
        out[mask] = model.first_logits().clone()
        if mask == 119:
            n_fused = model.last_launch_count()
            model.prefill(tok, lens, l, g)
            model.status()
            assert torch.equal(out[119], model.first_logits())
        else:
            assert model.last_launch_count() > n_fused + 20          # the fused form really replaces ~10 launches per layer
        model.close()
    assert (out[119] - out[55]).abs().max().item() <= 2e-3


def test_fused_last_token_launch_repeats_bit_for_bit_at_8b_widths():
    """The fused launch streams weights through a shared-memory ring that a producer warp refills as soon as the MMA warps
    release a stage; a release that comes before every lane has read the stage shows up as a few wrong weight rows in a
    tile, rarely (one step in ~20 at these widths), so: 8 prompts (8 activation rows, the widest form), the 8B widths
    (down projection K = 14336, the stage that reads activations from L2 while it multiplies), 60 repeats, equal bits."""
    import paper_2410_03960_b200 as P
    shape = S.LLAMA31_8B
    lens = [700, 300, 512, 900, 411, 650, 1000, 257]
    l, g = 16, 1
    w = S.make_weights(shape, 1, torch.bfloat16, "cuda")
    tok = S.make_prompts(1, lens, shape.vocab).cuda()
    model = P.SwiftKVModel(shape, w, torch.bfloat16, sum(lens), len(lens), l, g)
    assert model.set_kernel_mask(119) == 119
    first = None
    for it in range(60):
        model.prefill_device_tokens(tok, lens, l, g)
        model.status()
        lg = model.first_logits()
        if first is None:
            first = lg.clone()
        else:
            assert torch.equal(lg, first), f"repeat {it}: max difference {(lg - first).abs().max().item():.3e}"
    model.set_kernel_mask(55)
    model.prefill_device_tokens(tok, lens, l, g)
    model.status()
    assert (model.first_logits() - first).abs().max().item() <= 2e-3
    model.close()


def test_persistent_attention_gives_the_same_bits():
    """Kernel-mask bit 4 only changes which CTA runs which (query tile, head pair) item and in what order: every item's
    arithmetic is the same, so logits and caches must match bit for bit -- many short prompts (fewer items than SMs is the
    other extreme, in the tests above), ragged tails, a one-token prompt, a prompt of several query tiles."""
    import paper_2410_03960_b200 as P
    lens = [700, 1, 129, 300, 77, 513, 128, 2, 255, 40]
    l, g = 3, 1
    w = S.make_weights(MID, 5, torch.bfloat16, "cuda")
    tok = S.make_prompts(5, lens, MID.vocab)
    out = {}
    for mask in (55, 39):
        model = P.SwiftKVModel(MID, w, torch.bfloat16, sum(lens), len(lens), l, g)
        assert model.set_kernel_mask(mask) == mask
        model.prefill(tok, lens, l, g)
        model.status()
        out[mask] = (model.first_logits().clone(), [t.clone() for j in range(MID.n_layers) for t in model.kv_cache_view(j)[:2]])
        model.close()
    assert torch.equal(out[55][0], out[39][0])
    for a, b in zip(out[55][1], out[39][1]):
        assert torch.equal(a, b)
