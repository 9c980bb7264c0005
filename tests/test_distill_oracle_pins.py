"""Pins of oracle/distill_oracle.py (Sec. 3.4, Eq. 3: distillation of the re-wired student from the unmodified teacher,
only W_Q, W_K, W_V of the layers > l trainable, temperature 2.0) against things other than itself: central finite
differences of the loss, torch autograd through a torch-assembled student and teacher (library softmax / KL / SDPA /
rms_norm), and the cases the mathematics fixes (no re-wiring: loss and gradients vanish; KL >= 0; only group leaders'
W_K / W_V get gradient)."""
import numpy as np
import pytest
import torch

import synthetic_inputs as S
from oracle import distill_oracle as D
from oracle import swiftkv_oracle as O

SMALL = S.ModelShape(96, 64, 6, 4, 2, 16, 80, 10000.0, 1e-5, "small")
LENS = [13, 1, 7]


def _cfg(shape):
    return O.Config(shape.vocab, shape.hidden, shape.n_layers, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.ffn,
                    shape.rope_theta, shape.rms_eps)


def _weights(shape, seed, scale=4.0):
    """Random weights, larger than the benchmark's N(0, 0.02) so that the re-wired student is clearly off the teacher."""
    w = S.make_weights(shape, seed, torch.float32)
    layers = [{k: (v.double().numpy() * (scale if v.ndim == 2 else 1.0)) for k, v in lw.items()} for lw in w.layers]
    return w, O.Weights.from_arrays(w.embed.double().numpy() * scale, w.final_norm.double().numpy(), w.lm_head.double().numpy() * scale, layers)


def _perturbed_student(cfg, W, l, seed):
    St = D.student_copies(cfg, W, l)
    rng = np.random.default_rng(seed)
    for name in St:
        for j in range(l, cfg.n_layers):
            St[name][j] = St[name][j] + 0.05 * rng.standard_normal(St[name][j].shape)
    return St


def _torch_loss(shape, W, St, tokens, seq_lens, l, g, tau):
    """Teacher and student logits at every position from torch library routines, the library's KL, autograd for the
    gradients -- no code shared with the oracle."""
    F = torch.nn.functional
    dt = torch.float64
    L, hd, half = shape.n_layers, shape.head_dim, shape.head_dim // 2
    inv = shape.rope_theta ** (-2.0 * torch.arange(half, dtype=dt) / hd)
    lay = [{k: torch.tensor(v, dtype=dt) for k, v in W.layer(j).items()} for j in range(L)]
    P = {name: [None if St[name][j] is None else torch.tensor(St[name][j], dtype=dt, requires_grad=True) for j in range(L)] for name in St}
    embed = torch.tensor(W.embed_rows(np.arange(shape.vocab)), dtype=dt)
    fin, head = torch.tensor(W.final_norm, dtype=dt), torch.tensor(W.lm_head(), dtype=dt)

    def run(ids, swift):
        n = len(ids)
        rot = torch.polar(torch.ones(n, half, dtype=dt), torch.arange(n, dtype=dt)[:, None] * inv)

        def rope(t):
            z = torch.complex(t[..., :half], t[..., half:]) * rot[:, None, :]
            return torch.cat([z.real, z.imag], -1)
        x = embed[ids]
        s = None
        for j in range(L):
            lw = lay[j]
            if j == l:
                s = x
            h = F.rms_norm(x, (shape.hidden,), lw["in_norm"], shape.rms_eps)
            if swift and j >= l:
                r = l + ((j - l) // g) * g
                hs = F.rms_norm(s, (shape.hidden,), lay[r]["in_norm"], shape.rms_eps)
                q = rope(F.linear(h, P["wq"][j]).view(n, shape.n_q_heads, hd))
                k = rope(F.linear(hs, P["wk"][r]).view(n, shape.n_kv_heads, hd))
                v = F.linear(hs, P["wv"][r]).view(n, shape.n_kv_heads, hd)
            else:
                q = rope(F.linear(h, lw["wq"]).view(n, shape.n_q_heads, hd))
                k = rope(F.linear(h, lw["wk"]).view(n, shape.n_kv_heads, hd))
                v = F.linear(h, lw["wv"]).view(n, shape.n_kv_heads, hd)
            a = F.scaled_dot_product_attention(q.transpose(0, 1)[None], k.transpose(0, 1)[None], v.transpose(0, 1)[None],
                                               is_causal=True, enable_gqa=True)
            x = x + F.linear(a[0].transpose(0, 1).reshape(n, -1), lw["wo"])
            m = F.rms_norm(x, (shape.hidden,), lw["post_norm"], shape.rms_eps)
            x = x + F.linear(F.silu(F.linear(m, lw["w_gate"])) * F.linear(m, lw["w_up"]), lw["w_down"])
        return F.linear(F.rms_norm(x, (shape.hidden,), fin, shape.rms_eps), head)

    yt, ys, off = [], [], 0
    for n in seq_lens:
        ids = torch.as_tensor(tokens[off:off + n]).long()
        off += n
        yt.append(run(ids, False).detach())
        ys.append(run(ids, True))
    yt, ys = torch.cat(yt), torch.cat(ys)
    loss = tau * tau * F.kl_div(F.log_softmax(ys / tau, -1), F.softmax(yt / tau, -1), reduction="batchmean")
    loss.backward()
    grads = {name: [None if p is None else (p.grad.numpy() if p.grad is not None else np.zeros(p.shape)) for p in P[name]] for name in P}
    return float(loss.detach()), grads


@pytest.mark.parametrize("l,g", [(3, 1), (2, 2), (1, 3)])
def test_loss_and_gradients_against_torch_autograd(l, g):
    cfg = _cfg(SMALL)
    _, W = _weights(SMALL, 3)
    tokens = S.make_prompts(3, LENS, SMALL.vocab).numpy()
    St = _perturbed_student(cfg, W, l, 7)
    loss, grads = D.distill_grads(cfg, W, St, tokens, LENS, l, g, 2.0)
    want_loss, want = _torch_loss(SMALL, W, St, tokens, LENS, l, g, 2.0)
    assert loss > 1e-4                                             # the re-wired student really differs from the teacher
    assert abs(loss - want_loss) <= 1e-10 * max(1.0, abs(want_loss))
    for name in ("wq", "wk", "wv"):
        for j in range(l, cfg.n_layers):
            a, b = grads[name][j], want[name][j]
            assert np.abs(a - b).max() <= 1e-9 * max(1.0, np.abs(b).max()), (name, j)
    # with AcrossKV only the first layer of a group projects K / V: the others' copies are never read
    for j in range(l, cfg.n_layers):
        leader = l + ((j - l) // g) * g
        for name in ("wk", "wv"):
            assert (np.abs(grads[name][j]).max() > 0) == (j == leader), (name, j)
    assert all(np.abs(grads["wq"][j]).max() > 0 for j in range(l, cfg.n_layers))


def test_gradients_against_central_differences():
    cfg = _cfg(SMALL)
    _, W = _weights(SMALL, 5)
    lens = [6, 3]
    tokens = S.make_prompts(5, lens, SMALL.vocab).numpy()
    l, g, tau = 3, 2, 2.0
    St = _perturbed_student(cfg, W, l, 11)
    _, grads = D.distill_grads(cfg, W, St, tokens, lens, l, g, tau)
    rng = np.random.default_rng(1)
    eps = 1e-5
    for name, layers in (("wq", [3, 4, 5]), ("wk", [3, 5]), ("wv", [3, 5])):
        for j in layers:
            for _ in range(3):
                i, k = rng.integers(St[name][j].shape[0]), rng.integers(St[name][j].shape[1])
                old = St[name][j][i, k]
                St[name][j][i, k] = old + eps
                up = D.distill_loss(cfg, W, St, tokens, lens, l, g, tau)
                St[name][j][i, k] = old - eps
                dn = D.distill_loss(cfg, W, St, tokens, lens, l, g, tau)
                St[name][j][i, k] = old
                fd = (up - dn) / (2 * eps)
                assert abs(fd - grads[name][j][i, k]) <= 1e-6 * max(1e-3, abs(fd)), (name, j, i, k, fd, grads[name][j][i, k])


def test_no_rewiring_means_no_loss_and_no_gradient():
    """l = L: the student is the teacher (Eq. 3 with identical modes); an unperturbed student at l < L is NOT."""
    cfg = _cfg(SMALL)
    _, W = _weights(SMALL, 2)
    tokens = S.make_prompts(2, LENS, SMALL.vocab).numpy()
    St = D.student_copies(cfg, W, cfg.n_layers)
    assert abs(D.distill_loss(cfg, W, St, tokens, LENS, cfg.n_layers, 1, 2.0)) <= 1e-14
    St = D.student_copies(cfg, W, 3)
    loss, grads = D.distill_grads(cfg, W, St, tokens, LENS, 3, 1, 2.0)
    assert loss > 0.0 and all(np.abs(grads["wk"][j]).max() > 0 for j in range(3, cfg.n_layers))
    # layer l + 1 itself reads x_{l+1}: its re-wired K / V equal the original ones, so with ONLY that layer re-wired
    # (l = L - 1) the student is again the teacher
    St = D.student_copies(cfg, W, cfg.n_layers - 1)
    loss, grads = D.distill_grads(cfg, W, St, tokens, LENS, cfg.n_layers - 1, 1, 2.0)
    assert loss <= 1e-24 and np.abs(grads["wq"][cfg.n_layers - 1]).max() <= 1e-12


def test_loss_definition_and_temperature():
    rng = np.random.default_rng(0)
    yt, ys = rng.standard_normal((5, 11)), rng.standard_normal((5, 11))
    for tau in (1.0, 2.0, 4.0):
        pt = np.exp(yt / tau) / np.exp(yt / tau).sum(-1, keepdims=True)
        ps = np.exp(ys / tau) / np.exp(ys / tau).sum(-1, keepdims=True)
        want = tau * tau * np.mean(np.sum(pt * np.log(pt / ps), -1))
        got = D.distill_loss_from_logits(yt, ys, tau)
        assert abs(got - want) <= 1e-12 and got > 0
        lib = tau * tau * torch.nn.functional.kl_div(torch.log_softmax(torch.tensor(ys) / tau, -1), torch.softmax(torch.tensor(yt) / tau, -1),
                                                     reduction="batchmean").item()
        assert abs(got - lib) <= 1e-12
    assert abs(D.distill_loss_from_logits(yt, yt, 2.0)) <= 1e-15
    assert abs(D.distill_loss_from_logits(yt, yt + 3.0, 2.0)) <= 1e-15          # logits are shift-invariant


def test_adamw_update_against_the_library():
    rng = np.random.default_rng(4)
    p0 = rng.standard_normal((7, 5))
    grads = [rng.standard_normal((7, 5)) * (10.0 ** -k) for k in range(4)]
    for wd in (0.05, 0.0):
        t = torch.tensor(p0, dtype=torch.float64, requires_grad=True)
        opt = torch.optim.AdamW([t], lr=3e-4, betas=(0.9, 0.999), eps=1e-8, weight_decay=wd)
        p, m, v = p0.copy(), np.zeros_like(p0), np.zeros_like(p0)
        for step, g in enumerate(grads, 1):
            t.grad = torch.tensor(g)
            opt.step()
            p, m, v = D.adamw_update(p, g, m, v, step, 3e-4, 0.9, 0.999, 1e-8, wd)
            assert np.abs(p - t.detach().numpy()).max() <= 1e-14
    # first step of a zero-decay run moves every weight by lr against the sign of its gradient (up to eps)
    p, _, _ = D.adamw_update(p0, grads[0], np.zeros_like(p0), np.zeros_like(p0), 1, 3e-4, weight_decay=0.0)
    assert np.allclose(p0 - p, 3e-4 * np.sign(grads[0]), rtol=1e-6)
