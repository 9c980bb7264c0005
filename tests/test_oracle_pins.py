"""Pins for the CPU oracle: facts the paper and the mathematics fix, independent of the oracle itself.

Each test is chosen so that a plausible mistake in the oracle (a dropped term, a wrong sign or index, a
transposed operand, a wrong mask) fails at least one of them.
"""
import math
import os

import numpy as np
import pytest
import torch

import synthetic_inputs as S
from oracle import swiftkv_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _cfg(shape: S.ModelShape) -> O.Config:
    return O.Config(shape.vocab, shape.hidden, shape.n_layers, shape.n_q_heads, shape.n_kv_heads,
                    shape.head_dim, shape.ffn, shape.rope_theta, shape.rms_eps)


def _weights(shape: S.ModelShape, seed=0, dtype=torch.float32, zero_out=False) -> O.Weights:
    w = S.make_weights(shape, seed, dtype)
    layers = []
    for lw in w.layers:
        d = {k: v.double().numpy() for k, v in lw.items()}
        if zero_out:
            d["wo"] = np.zeros_like(d["wo"])
            d["w_down"] = np.zeros_like(d["w_down"])
        layers.append(d)
    return O.Weights.from_arrays(w.embed.double().numpy(), w.final_norm.double().numpy(),
                                 w.lm_head.double().numpy(), layers)


SMALL = S.ModelShape(96, 64, 6, 4, 2, 16, 80, 10000.0, 1e-5, "small")
LENS = [13, 1, 7]


@pytest.fixture(scope="module")
def small():
    cfg = _cfg(SMALL)
    W = _weights(SMALL, seed=5)
    tok = S.make_prompts(5, LENS, SMALL.vocab).numpy()
    return cfg, W, tok


def rel_l2(a, b):
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


# ------------------------------------------------------------------ operators ---------------------
def test_attention_against_brute_force():
    """Explicit n x n scores, explicit mask, explicit loops -- on tiny inputs, including n = 1."""
    rng = np.random.default_rng(0)
    for n, nq, nkv, hd in [(1, 4, 2, 8), (5, 4, 1, 4), (17, 6, 3, 8), (33, 2, 2, 16)]:
        q = rng.standard_normal((n, nq, hd))
        K = rng.standard_normal((n, nkv, hd))
        V = rng.standard_normal((n, nkv, hd))
        got = O.causal_attention(q, K, V).reshape(n, nq, hd)
        for p in range(n):
            for h in range(nq):
                kv = h // (nq // nkv)
                w = [math.exp(sum(q[p, h, c] * K[t, kv, c] for c in range(hd)) / math.sqrt(hd)) for t in range(p + 1)]
                z = sum(w)
                ref = [sum(w[t] * V[t, kv, c] for t in range(p + 1)) / z for c in range(hd)]
                assert np.allclose(got[p, h], ref, rtol=1e-10, atol=1e-12)
        if n == 1:
            assert np.allclose(got[0], np.repeat(V[0], nq // nkv, axis=0))
        # the single-query form equals the last row of the causal form
        sq = O.single_query_attention(q[-1], K, V)
        assert np.allclose(sq, got[-1].reshape(-1), rtol=1e-12, atol=1e-14)


def test_attention_against_torch_sdpa():
    rng = np.random.default_rng(1)
    n, nq, nkv, hd = 40, 8, 2, 32
    q, K, V = (rng.standard_normal((n, h, hd)) for h in (nq, nkv, nkv))
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q).transpose(0, 1)[None], torch.from_numpy(K).transpose(0, 1)[None],
        torch.from_numpy(V).transpose(0, 1)[None], is_causal=True, enable_gqa=True)[0].transpose(0, 1)
    assert np.allclose(O.causal_attention(q, K, V), ref.reshape(n, -1).numpy(), rtol=1e-10, atol=1e-12)


def test_rope_identities():
    rng = np.random.default_rng(2)
    hd, theta = 16, 10000.0
    q = rng.standard_normal((1, 3, hd))
    k = rng.standard_normal((1, 3, hd))
    assert np.array_equal(O.rope(q, np.array([0]), theta), q)                    # position 0 is the identity
    for m, n in [(5, 3), (100, 7), (65535, 65000)]:
        qm = O.rope(q, np.array([m]), theta)
        kn = O.rope(k, np.array([n]), theta)
        assert np.allclose(np.linalg.norm(qm, axis=-1), np.linalg.norm(q, axis=-1))   # a rotation
        lhs = np.sum(qm * kn, axis=-1)
        rhs = np.sum(O.rope(q, np.array([m - n]), theta) * k, axis=-1)           # depends on m - n only
        assert np.allclose(lhs, rhs, rtol=1e-9, atol=1e-9)
    # complex-number formulation: pair (i, i + hd/2) times exp(i * p * theta^(-2i/hd))
    p = 11
    x = rng.standard_normal((1, 1, hd))
    z = (x[0, 0, :hd // 2] + 1j * x[0, 0, hd // 2:]) * np.exp(1j * p * theta ** (-2.0 * np.arange(hd // 2) / hd))
    assert np.allclose(O.rope(x, np.array([p]), theta)[0, 0], np.concatenate([z.real, z.imag]))
    # a hand-computed value: hd = 2, theta irrelevant (single frequency 1), 90-degree turn
    out = O.rope(np.array([[[1.0, 0.0]]]), np.array([1]), 10000.0)
    assert np.allclose(out[0, 0], [math.cos(1.0), math.sin(1.0)])


def test_rmsnorm_silu_softmax():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((5, 32)) * 3
    g = rng.standard_normal(32)
    eps = 1e-5
    y = O.rmsnorm(x, np.ones(32), eps)
    ms = np.mean(x * x, -1)
    assert np.allclose(np.mean(y * y, -1), ms / (ms + eps))
    assert np.allclose(O.rmsnorm(1000 * x, g, eps), O.rmsnorm(x, g, eps), rtol=1e-4)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (32,), torch.from_numpy(g), eps).numpy()
    assert np.allclose(O.rmsnorm(x, g, eps), ref, rtol=1e-12)
    assert np.allclose(O.unit_rms(x, eps) * g, O.rmsnorm(x, g, eps))
    assert O.silu(np.array([0.0]))[0] == 0.0
    assert np.allclose(O.silu(np.array([30.0, -30.0])), [30.0, 0.0], atol=1e-11)
    assert np.allclose(O.silu(x), torch.nn.functional.silu(torch.from_numpy(x)).numpy())
    sm = O.softmax_rows(x)
    assert np.allclose(sm.sum(-1), 1.0) and np.allclose(sm, torch.softmax(torch.from_numpy(x), -1).numpy())


# ------------------------------------------------------------------ library cross-check -----------
def _torch_llama_forward(shape, w, tokens, seq_lens):
    """An independent fp64 forward of the unmodified model from torch library routines
    (rms_norm, linear, scaled_dot_product_attention with GQA, silu) and complex-number RoPE."""
    F = torch.nn.functional
    dt = torch.float64
    hd, half = shape.head_dim, shape.head_dim // 2
    Ks, Vs, logits = [[] for _ in range(shape.n_layers)], [[] for _ in range(shape.n_layers)], []
    off = 0
    for n in seq_lens:
        ids = torch.as_tensor(tokens[off:off + n]).long()
        off += n
        x = w.embed.to(dt)[ids]
        rot = torch.polar(torch.ones(n, half, dtype=dt),
                          torch.arange(n, dtype=dt)[:, None] * shape.rope_theta ** (-2.0 * torch.arange(half, dtype=dt) / hd))

        def rope(t):
            z = torch.complex(t[..., :half], t[..., half:]) * rot[:, None, :]
            return torch.cat([z.real, z.imag], -1)
        for j, lw in enumerate(w.layers):
            lw = {k: v.to(dt) for k, v in lw.items()}
            h = F.rms_norm(x, (shape.hidden,), lw["in_norm"], shape.rms_eps)
            q = rope(F.linear(h, lw["wq"]).view(n, shape.n_q_heads, hd))
            k = rope(F.linear(h, lw["wk"]).view(n, shape.n_kv_heads, hd))
            v = F.linear(h, lw["wv"]).view(n, shape.n_kv_heads, hd)
            Ks[j].append(k)
            Vs[j].append(v)
            a = F.scaled_dot_product_attention(q.transpose(0, 1)[None], k.transpose(0, 1)[None],
                                               v.transpose(0, 1)[None], is_causal=True, enable_gqa=True)
            x = x + F.linear(a[0].transpose(0, 1).reshape(n, -1), lw["wo"])
            m = F.rms_norm(x, (shape.hidden,), lw["post_norm"], shape.rms_eps)
            x = x + F.linear(F.silu(F.linear(m, lw["w_gate"])) * F.linear(m, lw["w_up"]), lw["w_down"])
        logits.append(F.linear(F.rms_norm(x[-1], (shape.hidden,), w.final_norm.to(dt), shape.rms_eps), w.lm_head.to(dt)))
    return [torch.cat(k).numpy() for k in Ks], [torch.cat(v).numpy() for v in Vs], torch.stack(logits).numpy()


def test_baseline_against_torch_library_forward_on_config1():
    """Config 1 (tiny Llama-style decoder, prompts of 128 and 96 tokens): the oracle's unmodified model
    against a forward pass assembled from torch library routines."""
    shape = S.TINY
    lens = [128, 96]
    w = S.make_weights(shape, 0, torch.float32)
    tok = S.make_prompts(0, lens, shape.vocab).numpy()
    Kt, Vt, lt = _torch_llama_forward(shape, w, tok, lens)
    out = O.baseline(_cfg(shape), _weights(shape, 0), tok, lens)
    for j in range(shape.n_layers):
        assert rel_l2(out["K"][j], Kt[j]) < 1e-12 and rel_l2(out["V"][j], Vt[j]) < 1e-12
    assert rel_l2(out["logits"], lt) < 1e-12
    # and the SwiftKV model agrees with it on everything that does not depend on the re-wiring
    sk = O.swiftkv(_cfg(shape), _weights(shape, 0), tok, lens, 2, 1)
    for j in range(2):
        assert np.array_equal(sk["K"][j], out["K"][j]) and np.array_equal(sk["V"][j], out["V"][j])
    assert rel_l2(sk["logits"], out["logits"]) > 1e-3          # it IS a different model


def _torch_swiftkv_forward(shape, w, tokens, seq_lens, l, g):
    """An independent fp64 SwiftKV forward from torch library routines: layers 1..l as in the unmodified model,
    K/V of every later layer projected from the layer-l output with that group's leading layer's norm gain and
    W_K, W_V (Eq. 2, Sec. 3.3), and only the last token of each prompt carried through layers l+1..L
    (footnote of Sec. 3.2, Sec. 3.5) -- written per prompt with SDPA on a one-row query, no code shared with the oracle."""
    F = torch.nn.functional
    dt = torch.float64
    L, hd, half = shape.n_layers, shape.head_dim, shape.head_dim // 2
    inv = shape.rope_theta ** (-2.0 * torch.arange(half, dtype=dt) / hd)
    Ks, Vs, logits = [[] for _ in range(L)], [[] for _ in range(L)], []
    lay = [{k: v.to(dt) for k, v in lw.items()} for lw in w.layers]
    off = 0
    for n in seq_lens:
        ids = torch.as_tensor(tokens[off:off + n]).long()
        off += n
        x = w.embed.to(dt)[ids]
        rot = torch.polar(torch.ones(n, half, dtype=dt), torch.arange(n, dtype=dt)[:, None] * inv)

        def rope(t, r):
            z = torch.complex(t[..., :half], t[..., half:]) * r[:, None, :]
            return torch.cat([z.real, z.imag], -1)
        for j in range(l):
            lw = lay[j]
            h = F.rms_norm(x, (shape.hidden,), lw["in_norm"], shape.rms_eps)
            q = rope(F.linear(h, lw["wq"]).view(n, shape.n_q_heads, hd), rot)
            k = rope(F.linear(h, lw["wk"]).view(n, shape.n_kv_heads, hd), rot)
            v = F.linear(h, lw["wv"]).view(n, shape.n_kv_heads, hd)
            Ks[j].append(k)
            Vs[j].append(v)
            a = F.scaled_dot_product_attention(q.transpose(0, 1)[None], k.transpose(0, 1)[None],
                                               v.transpose(0, 1)[None], is_causal=True, enable_gqa=True)
            x = x + F.linear(a[0].transpose(0, 1).reshape(n, -1), lw["wo"])
            m = F.rms_norm(x, (shape.hidden,), lw["post_norm"], shape.rms_eps)
            x = x + F.linear(F.silu(F.linear(m, lw["w_gate"])) * F.linear(m, lw["w_up"]), lw["w_down"])
        s = x
        cache = {}
        for j in range(l, L):
            r = l + ((j - l) // g) * g                      # 0-based first layer of j's group
            if r not in cache:
                h = F.rms_norm(s, (shape.hidden,), lay[r]["in_norm"], shape.rms_eps)
                cache[r] = (rope(F.linear(h, lay[r]["wk"]).view(n, shape.n_kv_heads, hd), rot),
                            F.linear(h, lay[r]["wv"]).view(n, shape.n_kv_heads, hd))
            Ks[j].append(cache[r][0])
            Vs[j].append(cache[r][1])
        y = s[n - 1:n]                                      # [1, d]: the continuing token, position n - 1
        for j in range(l, L):
            lw = lay[j]
            k, v = cache[l + ((j - l) // g) * g]
            h = F.rms_norm(y, (shape.hidden,), lw["in_norm"], shape.rms_eps)
            q = rope(F.linear(h, lw["wq"]).view(1, shape.n_q_heads, hd), rot[n - 1:n])
            # one query row against all n cached keys: no mask (every key is at or before position n - 1)
            a = F.scaled_dot_product_attention(q.transpose(0, 1)[None], k.transpose(0, 1)[None],
                                               v.transpose(0, 1)[None], is_causal=False, enable_gqa=True)
            y = y + F.linear(a[0].transpose(0, 1).reshape(1, -1), lw["wo"])
            m = F.rms_norm(y, (shape.hidden,), lw["post_norm"], shape.rms_eps)
            y = y + F.linear(F.silu(F.linear(m, lw["w_gate"])) * F.linear(m, lw["w_up"]), lw["w_down"])
        logits.append(F.linear(F.rms_norm(y[0], (shape.hidden,), w.final_norm.to(dt), shape.rms_eps), w.lm_head.to(dt)))
    return [torch.cat(k).numpy() for k in Ks], [torch.cat(v).numpy() for v in Vs], torch.stack(logits).numpy()


@pytest.mark.parametrize("l,g", [(2, 1), (1, 2), (1, 3), (3, 1)])
def test_swiftkv_against_torch_library_forward_on_config1(l, g):
    """Config 1 with the re-wiring on: every layer's cache and the first-token logits against a SwiftKV forward
    assembled from torch library routines.  This is what fixes the continuing token's path through layers l+1..L
    (its own hidden state through the layer's own input norm and W_Q, rotary position n - 1, all n cached keys,
    attention residual, post-attention norm, MLP residual)."""
    shape = S.TINY
    lens = [128, 96]
    w = S.make_weights(shape, 0, torch.float32)
    tok = S.make_prompts(0, lens, shape.vocab).numpy()
    Kt, Vt, lt = _torch_swiftkv_forward(shape, w, tok, lens, l, g)
    out = O.swiftkv(_cfg(shape), _weights(shape, 0), tok, lens, l, g)
    for j in range(shape.n_layers):
        assert rel_l2(out["K"][j], Kt[j]) < 1e-12 and rel_l2(out["V"][j], Vt[j]) < 1e-12
    assert rel_l2(out["logits"], lt) < 1e-12


@pytest.mark.parametrize("which", ["small", "config1"])
def test_tail_layer_is_the_last_row_of_a_causal_layer(which):
    """The last row of an unmodified causal layer depends only on that row's hidden state and on the layer's
    cache, so `tail_layer` fed with the baseline's own hidden state x_j[n-1] and its own K_j, V_j must return
    row n - 1 of `decoder_layer`'s output -- for every layer and prompt.  A wrong query position, a wrong norm
    gain, a dropped residual or a key-range slip in `tail_layer` breaks the identity."""
    if which == "small":
        shape, lens, seed = SMALL, LENS, 5
    else:
        shape, lens, seed = S.TINY, [128, 96], 0
    cfg, W = _cfg(shape), _weights(shape, seed)
    tok = S.make_prompts(seed, lens, shape.vocab).numpy()
    off = 0
    for n in lens:
        X = np.asarray(W.embed_rows(tok[off:off + n]), dtype=np.float64)
        off += n
        pos = np.arange(n)
        for j in range(cfg.n_layers):
            Xn, K, V = O.decoder_layer(cfg, W.layer(j), X, pos)
            y = O.tail_layer(cfg, W.layer(j), X[n - 1], n - 1, K, V)
            assert np.allclose(y, Xn[n - 1], rtol=1e-11, atol=1e-13)
            if n > 2:
                # an inner row p is the last row of the prefix 0..p: tail_layer must read keys 0..p only
                p = n // 2
                yp = O.tail_layer(cfg, W.layer(j), X[p], p, K, V)
                assert np.allclose(yp, Xn[p], rtol=1e-11, atol=1e-13)
            X = Xn


# ------------------------------------------------------------------ SwiftKV structure -------------
def test_layers_up_to_l_untouched_and_l_equal_L_is_baseline(small):
    cfg, W, tok = small
    base = O.baseline(cfg, W, tok, LENS)
    for l in (1, 3, 5):
        sk = O.swiftkv(cfg, W, tok, LENS, l, 2)
        for j in range(l):
            assert np.array_equal(sk["K"][j], base["K"][j]) and np.array_equal(sk["V"][j], base["V"][j])
    full = O.swiftkv(cfg, W, tok, LENS, cfg.n_layers, 3)
    for j in range(cfg.n_layers):
        assert np.array_equal(full["K"][j], base["K"][j]) and np.array_equal(full["V"][j], base["V"][j])
    assert np.array_equal(full["logits"], base["logits"])


def test_group1_equals_ungrouped_eq2(small):
    """AcrossKV with group 1 is SingleInputKV: compare with Eq. 2 written with no grouping code, fed with the
    hidden state after l unmodified layers."""
    cfg, W, tok = small
    l = 2
    s = O.hidden_after(cfg, W, tok, LENS, l)
    pos = np.concatenate([np.arange(n) for n in LENS])
    Ks, Vs = O.swiftkv_eq2_ungrouped(cfg, W, s, pos, l)
    sk = O.swiftkv(cfg, W, tok, LENS, l, 1)
    for j in range(l, cfg.n_layers):
        assert np.allclose(sk["K"][j], Ks[j], rtol=1e-13, atol=1e-15)
        assert np.allclose(sk["V"][j], Vs[j], rtol=1e-13, atol=1e-15)
    # Eq. 2 on V needs no RoPE: V_j = rmsnorm(s) W_V^T, re-derived here from library calls
    j = 4
    w = W.layer(j)
    v = torch.nn.functional.linear(
        torch.nn.functional.rms_norm(torch.from_numpy(s), (cfg.hidden,), torch.from_numpy(w["in_norm"]), cfg.rms_eps),
        torch.from_numpy(w["wv"])).numpy().reshape(-1, cfg.n_kv_heads, cfg.head_dim)
    assert np.allclose(sk["V"][j], v, rtol=1e-12, atol=1e-14)


def test_acrosskv_grouping(small):
    """Fig. 1's example: L = 8, l = 4, 2-way AcrossKV -> layers 5,6 share layer 5's projection, 7,8 layer 7's."""
    assert [O.group_leader(4, 2, j) for j in (5, 6, 7, 8)] == [5, 5, 7, 7]
    assert [O.group_leader(2, 4, j) for j in (3, 4, 5, 6, 7)] == [3, 3, 3, 3, 7]
    cfg, W, tok = small
    l = 2
    one = O.swiftkv(cfg, W, tok, LENS, l, 1)
    for g in (2, 3, 4):
        sk = O.swiftkv(cfg, W, tok, LENS, l, g)
        distinct = {id(k) for k in sk["K"]}
        assert len(distinct) == l + -(-(cfg.n_layers - l) // g)
        for j1 in range(l + 1, cfg.n_layers + 1):
            r1 = O.group_leader(l, g, j1)
            assert sk["K"][j1 - 1] is sk["K"][r1 - 1] and sk["V"][j1 - 1] is sk["V"][r1 - 1]
            # the projection of s does not depend on g
            assert np.array_equal(sk["K"][r1 - 1], one["K"][r1 - 1])
            assert np.array_equal(sk["V"][r1 - 1], one["V"][r1 - 1])
        assert rel_l2(sk["logits"], one["logits"]) > 1e-6       # sharing changes the model


def test_folded_fused_projection_equals_norm_then_project(small):
    cfg, W, tok = small
    pos = np.concatenate([np.arange(n) for n in LENS])
    for l, g in [(2, 1), (2, 2), (1, 3)]:
        s = O.hidden_after(cfg, W, tok, LENS, l)
        Wt = O.folded_kv_weight(cfg, W, l, g)
        n_groups = -(-(cfg.n_layers - l) // g)
        assert Wt.shape == (n_groups * 2 * cfg.d_kv, cfg.hidden)
        Ks, Vs = O.fused_single_input_kv(cfg, Wt, s, pos)
        sk = O.swiftkv(cfg, W, tok, LENS, l, g)
        for i in range(n_groups):
            r = l + i * g
            assert rel_l2(Ks[i], sk["K"][r]) < 1e-12 and rel_l2(Vs[i], sk["V"][r]) < 1e-12


def test_identity_residual_special_case():
    """W_O = W_down = 0 makes every layer the identity on the residual stream, so x_j = x_1 for all j and the
    SwiftKV model (any l, g = 1) must reproduce the unmodified model exactly: the paper's premise
    x_j ~ x_{l+1} made exact."""
    cfg = _cfg(SMALL)
    W = _weights(SMALL, seed=9, zero_out=True)
    tok = S.make_prompts(9, LENS, SMALL.vocab).numpy()
    base = O.baseline(cfg, W, tok, LENS)
    for l in (1, 2, 4, 5):
        sk = O.swiftkv(cfg, W, tok, LENS, l, 1)
        for j in range(cfg.n_layers):
            assert np.allclose(sk["K"][j], base["K"][j], rtol=1e-12, atol=1e-14)
            assert np.allclose(sk["V"][j], base["V"][j], rtol=1e-12, atol=1e-14)
        assert np.allclose(sk["logits"], base["logits"], rtol=1e-11, atol=1e-13)


def test_constant_prompt_special_case():
    """All tokens of a prompt identical -> all V rows identical -> attention output is V whatever the scores ->
    hidden states are position-independent: logits(length n) = logits(length 1), K_j[p] = rope(K_j[0], p)."""
    cfg = _cfg(SMALL)
    W = _weights(SMALL, seed=3)
    for fn in (lambda t, ln: O.baseline(cfg, W, t, ln), lambda t, ln: O.swiftkv(cfg, W, t, ln, 3, 2)):
        a = fn(np.full(9, 17), [9])
        b = fn(np.full(1, 17), [1])
        assert np.allclose(a["logits"], b["logits"], rtol=1e-10, atol=1e-13)
        for j in range(cfg.n_layers):
            assert np.allclose(a["V"][j], np.broadcast_to(a["V"][j][0], a["V"][j].shape), rtol=1e-10, atol=1e-13)
            k0 = np.repeat(b["K"][j], 9, axis=0)
            assert np.allclose(a["K"][j], O.rope(k0, np.arange(9), cfg.rope_theta), rtol=1e-10, atol=1e-13)


def test_causality_and_batch_independence(small):
    cfg, W, tok = small
    for l, g in [(cfg.n_layers, 1), (3, 2)]:
        full = O.swiftkv(cfg, W, tok, LENS, l, g)
        # a prompt alone gives the same caches and logits as inside the batch
        off = 0
        for b, n in enumerate(LENS):
            alone = O.swiftkv(cfg, W, tok[off:off + n], [n], l, g)
            for j in range(cfg.n_layers):
                # (equal up to BLAS blocking: a [T, d] and an [n, d] product round in different orders)
                assert np.allclose(alone["K"][j], full["K"][j][off:off + n], rtol=1e-12, atol=1e-14)
                assert np.allclose(alone["V"][j], full["V"][j][off:off + n], rtol=1e-12, atol=1e-14)
            assert np.allclose(alone["logits"][0], full["logits"][b], rtol=1e-12, atol=1e-14)   # BLAS blocks [B,d] and [1,d] differently
            off += n
        # changing later tokens leaves earlier cache rows untouched
        t2 = tok.copy()
        t2[8:13] = (t2[8:13] + 1) % cfg.vocab
        ch = O.swiftkv(cfg, W, t2, LENS, l, g)
        for j in range(cfg.n_layers):
            assert np.array_equal(ch["K"][j][:8], full["K"][j][:8]) and np.array_equal(ch["V"][j][:8], full["V"][j][:8])
            assert not np.array_equal(ch["V"][j][8:13], full["V"][j][8:13])
        # a truncated prompt is a causal prefix
        tr = O.swiftkv(cfg, W, tok[:6], [6], l, g)
        for j in range(cfg.n_layers):
            assert np.allclose(tr["K"][j], full["K"][j][:6], rtol=1e-12, atol=1e-14)
            assert np.allclose(tr["V"][j], full["V"][j][:6], rtol=1e-12, atol=1e-14)


# ------------------------------------------------------------------ SimScore (Eq. 1) --------------
def test_simscore_definition():
    """Eq. 1: SimScore(x_l) = average over the later layers j of Similarity(x_l, x_j), Similarity = average over tokens
    of the cosine.  Hand values, a library routine, and the facts a cosine obeys."""
    e1, e2 = np.array([1.0, 0.0, 0.0]), np.array([0.0, 1.0, 0.0])
    d45 = np.array([1.0, 1.0, 0.0])
    # two tokens; x_1 = (e1, e1); x_2 = (e1, e2) -> cosines 1 and 0; x_3 = (d45, -e1) -> cosines 1/sqrt2 and -1
    x1, x2, x3 = np.stack([e1, e1]), np.stack([e1, e2]), np.stack([d45, -e1])
    assert O.similarity(x1, x2) == pytest.approx(0.5)
    assert O.similarity(x1, x3) == pytest.approx((1 / math.sqrt(2) - 1) / 2)
    s = O.simscore([x1, x2, x3])
    assert s.shape == (2,)
    assert s[0] == pytest.approx((0.5 + (1 / math.sqrt(2) - 1) / 2) / 2)       # layers 2 and 3 follow layer 1
    assert s[1] == pytest.approx((1 / math.sqrt(2) + 0.0) / 2)                 # only layer 3 follows layer 2: cos 1/sqrt2, 0
    rng = np.random.default_rng(4)
    xs = [rng.standard_normal((9, 16)) for _ in range(5)]
    got = O.simscore(xs)
    for l in range(1, 5):
        want = np.mean([torch.nn.functional.cosine_similarity(torch.from_numpy(xs[l - 1]), torch.from_numpy(xs[j - 1]), dim=-1).mean().item()
                        for j in range(l + 1, 6)])
        assert got[l - 1] == pytest.approx(want, rel=1e-12)
    # a cosine ignores positive per-token scales and is 1 between equal inputs
    scaled = [x * np.exp(rng.uniform(-3, 3, (9, 1))) for x in xs]
    assert np.allclose(O.simscore(scaled), got, rtol=1e-12)
    assert np.allclose(O.simscore([xs[0]] * 4), 1.0)
    assert np.allclose(O.simscore([xs[0], -xs[0]]), -1.0)


def test_simscore_of_the_identity_residual_model_is_one():
    """W_O = W_down = 0: every layer is the identity on the residual stream, all layer inputs are equal (the paper's
    premise "inputs of deeper layers are similar" made exact), so SimScore(x_l) = 1 for every l; with the ordinary
    random weights it lies strictly between 0 and 1 and the layer inputs are what `decoder_layer` chains."""
    cfg = _cfg(SMALL)
    tok = S.make_prompts(9, LENS, SMALL.vocab).numpy()
    xs = O.layer_inputs(cfg, _weights(SMALL, seed=9, zero_out=True), tok, LENS)
    assert len(xs) == cfg.n_layers and np.allclose(O.simscore(xs), 1.0, rtol=0, atol=1e-12)
    W = _weights(SMALL, seed=9)
    xs = O.layer_inputs(cfg, W, tok, LENS)
    assert np.array_equal(xs[0], W.embed_rows(tok))                             # x_1 is the embedding
    pos = np.concatenate([np.arange(n) for n in LENS])
    a, e = 0, LENS[0]
    assert np.allclose(O.decoder_layer(cfg, W.layer(2), xs[2][a:e], pos[a:e])[0], xs[3][a:e], rtol=1e-12, atol=1e-14)
    s = O.simscore(xs)
    assert ((s > 0) & (s < 1)).all()


# ------------------------------------------------------------------ closed forms the paper prints --
def _rows(name):
    with open(os.path.join(GOLD, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def test_table1_flop_breakdown():
    cfg = _cfg(S.LLAMA31_70B)
    rows = _rows("table1_gflops_per_token.txt")
    # the context length behind the attention column is not printed; fix it from the baseline row only
    base_attn = float(rows[0][6])
    context = base_attn * 1e9 / (cfg.n_layers * 4 * cfg.d_q) * 2
    base_total = None
    for frac, g, vocab, kv, qo, mlp, attn, total, rel in rows:
        l = round(cfg.n_layers * (1 - float(frac)))
        got = O.table1_gflops_per_token(cfg, l, int(g), context)
        assert abs(got["vocab"] - float(vocab)) < 0.11
        assert abs(got["kv"] - float(kv)) < 0.1
        assert abs(got["qo"] - float(qo)) < 0.6
        assert abs(got["mlp"] - float(mlp)) < 0.6
        assert abs(got["attn"] - float(attn)) < 0.6
        assert abs(got["total"] - float(total)) < 1.5
        base_total = base_total or got["total"]
        assert abs(100 * got["total"] / base_total - float(rel)) < 0.15


def test_kv_cache_reduction_percentages():
    for g, pct in _rows("kv_cache_reduction.txt"):
        assert abs(100 * O.kv_cache_reduction(32, 16, int(g)) - float(pct)) < 1e-9
        if 40 % int(g) == 0:      # the printed figures assume whole groups; a short last group saves less
            assert abs(100 * O.kv_cache_reduction(80, 40, int(g)) - float(pct)) < 1e-9
    assert O.kv_cache_reduction(32, 32, 4) == 0.0 and O.kv_cache_reduction(32, 16, 1) == 0.0


def test_normalized_throughput_arithmetic():
    """tokens/s x 2 x parameter count of the baseline model reproduces the paper's TFLOPS/GPU figures."""
    shapes = {"llama-3.1-70b": S.LLAMA31_70B, "llama-3.1-8b": S.LLAMA31_8B}
    for name, tps, n_gpus, tflops in _rows("normalized_throughput.txt"):
        got = float(tps) * 2 * shapes[name].n_params() / int(n_gpus) / 1e12
        assert abs(got - float(tflops)) / float(tflops) < 0.01


# ---------------------------------------------------------------------------------------------------
# FP8 (e4m3) per-token cache quantization (appendix, KV quantization)
# ---------------------------------------------------------------------------------------------------
def test_e4m3_format_defining_values():
    """Values fixed by the format's definition: bias 7, 3 mantissa bits, no infinities, largest finite 448."""
    dec = O.e4m3_decode(np.arange(256))
    assert dec[0x00] == 0.0 and dec[0x80] == 0.0 and np.signbit(dec[0x80])
    assert dec[0x38] == 1.0 and dec[0x40] == 2.0 and dec[0x3C] == 1.5 and dec[0xB8] == -1.0
    assert dec[0x01] == 2.0 ** -9 and dec[0x07] == 7 * 2.0 ** -9 and dec[0x08] == 2.0 ** -6
    assert dec[0x7E] == 448.0 and dec[0xFE] == -448.0 and dec[0x77] == 240.0 and dec[0x78] == 256.0
    assert np.isnan(dec[0x7F]) and np.isnan(dec[0xFF]) and np.isfinite(np.delete(dec, [0x7F, 0xFF])).all()
    pos = dec[:0x7F]
    assert (np.diff(pos) > 0).all()                                # codes order like their values
    # library cross-check: torch's float8_e4m3fn reads the same 256 bit patterns
    lib = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    assert np.array_equal(np.isnan(dec), np.isnan(lib))
    assert np.array_equal(dec[~np.isnan(dec)], lib[~np.isnan(lib)])


def _nearest_code_by_search(y: float) -> int:
    """Brute force in plain Python: the finite code whose value is nearest to y; of two equally near values the one
    with the even code (even mantissa field); beyond the largest value, the largest value."""
    vals = [float(v) for v in O.e4m3_decode(np.arange(0x7F))]     # non-negative finite values, ascending
    a = abs(y)
    best, best_d = 0, None
    for c, v in enumerate(vals):
        d = abs(a - v)
        if best_d is None or d < best_d or (d == best_d and c % 2 == 0):
            best, best_d = c, d
    return best | (0x80 if math.copysign(1.0, y) < 0 else 0)


def test_e4m3_encode_against_search_and_library():
    vals = O.e4m3_decode(np.arange(0x7F))
    mid = (vals[:-1] + vals[1:]) / 2                               # every tie point (all exact in fp32)
    rng = np.random.default_rng(5)
    probe = np.concatenate([vals, mid, np.nextafter(mid.astype(np.float32), np.float32(0)),
                            np.nextafter(mid.astype(np.float32), np.float32(1e9)),
                            rng.uniform(0, 448, 300), rng.uniform(0, 2.0 ** -5, 100), [448.5, 463.9, 464.0, 1e6]])
    probe = np.concatenate([probe, -probe]).astype(np.float32)
    got = O.e4m3_encode(probe)
    want = np.array([_nearest_code_by_search(float(v)) for v in probe], dtype=np.uint8)
    assert np.array_equal(got, want)
    # every finite code is a fixed point
    codes = np.delete(np.arange(256), [0x7F, 0xFF]).astype(np.uint8)
    assert np.array_equal(O.e4m3_encode(O.e4m3_decode(codes)), codes)
    # library: torch's conversion rounds to nearest even as well (inside the finite range)
    big = np.concatenate([probe[np.abs(probe) <= 448], rng.standard_normal(200000).astype(np.float32) * 120]).astype(np.float32)
    big = big[np.abs(big) <= 448]
    lib = torch.from_numpy(big).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(O.e4m3_encode(big), lib)


def test_quantize_per_token_properties():
    rng = np.random.default_rng(9)
    x = (rng.standard_normal((37, 2, 32)) * np.exp(rng.uniform(-6, 6, (37, 1, 1)))).astype(np.float32)
    x[5] = 0.0                                                     # an all-zero row
    codes, scale, deq = O.quantize_per_token(x)
    assert codes.dtype == np.uint8 and codes.shape == x.shape and scale.dtype == np.float32 and scale.shape == (37,)
    flat, dflat, cflat = x.reshape(37, -1).astype(np.float64), deq.reshape(37, -1), codes.reshape(37, -1)
    amax = np.abs(flat).max(axis=1)
    # the scale maps the row maximum to 448 (one fp32 rounding), the maximum itself is stored as +-448
    nz = amax > 0
    assert np.allclose(scale[nz].astype(np.float64) * 448, amax[nz], rtol=2.0 ** -23, atol=0)
    assert ((cflat[nz] & 0x7F).max(axis=1) == 0x7E).all()
    assert (cflat[5] & 0x7F).max() == 0 and (dflat[5] == 0).all() and scale[5] == np.float32(2.0 ** -64 / 448)
    # error bound of round-to-nearest: half a step of the code's binade (3 mantissa bits), in units of the scale;
    # relative error at most 2^-4 for values in the normal range
    y = flat / scale.astype(np.float64)[:, None]
    step = np.where(np.abs(y) < 2.0 ** -6, 2.0 ** -9, 2.0 ** (np.floor(np.log2(np.maximum(np.abs(y), 2.0 ** -6))) - 3))
    err = np.abs(dflat - flat) / scale.astype(np.float64)[:, None]
    assert (err <= step / 2 * (1 + 1e-6) + 1e-12).all()
    normal = np.abs(y) >= 2.0 ** -6
    assert (np.abs(dflat - flat)[normal] <= np.abs(flat)[normal] * 2.0 ** -4 * (1 + 1e-6)).all()
    assert (np.sign(dflat) * np.sign(flat) >= 0).all()
    # rows are independent, and a power-of-two factor moves into the scale only
    c1, s1, _ = O.quantize_per_token(x[3:4])
    assert np.array_equal(c1[0], codes[3]) and s1[0] == scale[3]
    c2, s2, d2 = O.quantize_per_token(x * np.float32(8.0))
    assert np.array_equal(c2[nz], codes[nz]) and np.array_equal(s2[nz], scale[nz] * np.float32(8)) and np.array_equal(d2[nz], deq[nz] * 8)
    # sign symmetry
    c3, s3, _ = O.quantize_per_token(-x)
    assert np.array_equal(c3[nz] ^ 0x80, codes[nz]) and np.array_equal(s3, scale)


def test_round_to_bf16_against_library():
    rng = np.random.default_rng(2)
    x = np.concatenate([rng.standard_normal(100000).astype(np.float32) * 3,
                        np.float32([0.0, -0.0, 1.0, 1.00390625, 1.001953125, 1.005859375, 3.3895314e38, 1e-38])])
    want = torch.from_numpy(x).to(torch.bfloat16).float().numpy()
    assert np.array_equal(O.round_to_bf16(x), want)
    # ties go to the even significand: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert O.round_to_bf16(np.float32([1.00390625]))[0] == 1.0 and O.round_to_bf16(np.float32([1.01171875]))[0] == 1.015625
    c, s, _ = O.quantize_per_token(x[:64].reshape(2, 32), "bf16")
    c2, s2, _ = O.quantize_per_token(want[:64].reshape(2, 32))
    assert np.array_equal(c, c2) and np.array_equal(s, s2)


def test_kv_cache_reduction_with_fp8():
    for g, fp8, pct in _rows("kv_cache_reduction_fp8.txt"):
        got = 100 * O.kv_cache_reduction(32, 16, int(g), 0.5 if int(fp8) else 1.0)
        assert abs(got - float(pct)) < 1e-9


def test_swiftkv_with_fp8_cache_structure():
    """The quantized model: the stored rows are exactly the quantization of what the layer would have cached,
    everything downstream sees only them, and the structural facts of SwiftKV survive."""
    shape = S.TINY
    cfg, W = _cfg(shape), _weights(shape, seed=3)
    lens = [21, 9]
    tok = np.concatenate([S.token_ids(3, b, n, shape.vocab).numpy() for b, n in enumerate(lens)])
    ref = O.swiftkv(cfg, W, tok, lens, 2, 1)
    q = O.swiftkv(cfg, W, tok, lens, 2, 1, kv_fp8=True)
    # layer 1 sees the same input either way: its cache is the quantization of the unquantized run's cache
    for name in ("K", "V"):
        codes, scale, deq = O.quantize_per_token(ref[name][0])
        assert np.array_equal(q[name + "_codes"][0], codes) and np.array_equal(q[name + "_scale"][0], scale)
        assert np.array_equal(q[name][0], deq)
    # stored representation <-> values, every layer
    for j in range(shape.n_layers):
        for name in ("K", "V"):
            back = O.e4m3_decode(q[name + "_codes"][j]) * q[name + "_scale"][j].astype(np.float64)[:, None, None]
            assert np.allclose(back, q[name][j], rtol=2.0 ** -22, atol=0)
            assert 0.005 < rel_l2(q[name][j], ref[name][j]) < 0.06     # 3 mantissa bits: a few percent, not zero
    assert 0 < rel_l2(q["logits"], ref["logits"]) < 0.2
    # layer 2's attention read the quantized layer-2 cache: with the quantizer bypassed there, layer 3's input changes
    # (checked through the SingleInputKV rows, which are a function of the layer-2 output)
    assert not np.array_equal(q["K_codes"][2], O.quantize_per_token(ref["K"][2])[0])
    # AcrossKV aliasing and l = L (baseline) still hold
    q2 = O.swiftkv(cfg, W, tok, lens, 2, 2, kv_fp8=True)
    assert q2["K"][3] is q2["K"][2] and np.array_equal(q2["K_codes"][2], q["K_codes"][2])
    full = O.swiftkv(cfg, W, tok, lens, shape.n_layers, 1, kv_fp8=True)
    assert np.array_equal(full["K_codes"][0], q["K_codes"][0]) and np.array_equal(full["K_codes"][1], q["K_codes"][1])
    # a prompt alone equals the prompt inside the batch (per-token scales do not couple prompts)
    alone = O.swiftkv(cfg, W, tok[:21], [21], 2, 1, kv_fp8=True)
    assert np.array_equal(alone["K_codes"][3], q["K_codes"][3][:21]) and np.allclose(alone["logits"][0], q["logits"][0], rtol=1e-12)
    # constant prompt: all V rows equal, attention output = that row whatever the scores, so the logits do not
    # depend on the prompt length (the quantized rows are still identical to each other)
    c5 = O.swiftkv(cfg, W, np.full(5, 17), [5], 2, 1, kv_fp8=True)
    c1 = O.swiftkv(cfg, W, np.full(1, 17), [1], 2, 1, kv_fp8=True)
    assert np.allclose(c5["logits"], c1["logits"], rtol=1e-9, atol=1e-12)
