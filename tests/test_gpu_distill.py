"""The knowledge-recovery step (Sec. 3.4, Eq. 3) through the C ABI against the oracle: distillation loss at temperature 2
between the unmodified teacher and the re-wired student at every prompt position, and its gradients with respect to the
student's W_Q, W_K, W_V of the layers > l (AcrossKV groups included)."""
import numpy as np
import pytest
import torch

import synthetic_inputs as S
from oracle import distill_oracle as D
from helpers import oracle_config, oracle_weights, to_np

pytestmark = pytest.mark.gpu

MID = S.ModelShape(1024, 512, 4, 8, 2, 128, 1024, 500000.0, 1e-5, "mid")
SIX = S.ModelShape(512, 256, 6, 8, 2, 32, 688, 10000.0, 1e-5, "tiny-6-layers")
ODD = S.ModelShape(320, 192, 5, 6, 3, 48, 400, 10000.0, 1e-5, "odd-widths")          # head_dim 48: lanes past the head are idle
W8B_2L = S.ModelShape(2048, 4096, 2, 32, 8, 128, 14336, 500000.0, 1e-5, "8b-widths-2-layers")      # Llama-3.1-8B layer widths


def _scaled_weights(shape, seed, scale):
    """The benchmark's N(0, 0.02) weights leave teacher and student almost equal; larger matrices make the re-wiring matter."""
    w = S.make_weights(shape, seed, torch.float32, "cpu")
    for lw in w.layers:
        for name, t in lw.items():
            if t.ndim == 2:
                t.mul_(scale)
    w.embed.mul_(scale)
    w.lm_head.mul_(scale)
    return w


def _student(w, l, seed, noise):
    g = torch.Generator().manual_seed(seed)
    L = len(w.layers)
    return {name: [None if j < l else (w.layers[j][name] + noise * w.layers[j][name].std() * torch.randn(w.layers[j][name].shape, generator=g)).contiguous()
                   for j in range(L)] for name in ("wq", "wk", "wv")}


def _rel(a, b):
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-30))


@pytest.mark.parametrize("shape,lens,l,g,scale", [
    (SIX, [37, 1, 20], 3, 1, 3.0),
    (SIX, [37, 1, 20], 2, 2, 3.0),
    (SIX, [25, 14], 1, 3, 3.0),             # groups of 3 with a short last group (layers 2-4, 5-6)
    (ODD, [19, 30, 2], 2, 2, 3.0),
    (MID, [40, 9], 2, 1, 2.0),
    (MID, [130], 1, 2, 2.0),                # one prompt longer than a 128-row tile
    (W8B_2L, [48, 17], 1, 1, 1.5),          # the widths of the benchmark model (sums of 4096 and 14336 terms)
])
def test_loss_and_gradients_against_oracle(shape, lens, l, g, scale):
    import paper_2410_03960_b200 as P
    seed, tau = 17, 2.0
    w = _scaled_weights(shape, seed, scale)
    tok = S.make_prompts(seed, lens, shape.vocab)
    st = _student(w, l, seed + 1, 0.3)
    cfg, W = oracle_config(shape), oracle_weights(w)
    want_loss, want = D.distill_grads(cfg, W, {k: [None if t is None else t.double().numpy() for t in v] for k, v in st.items()},
                                      tok.numpy(), lens, l, g, tau)
    assert want_loss > 1e-3                                          # a real difference between the two modes

    wc = S.Weights(shape, torch.float32, w.embed.cuda(), w.final_norm.cuda(), w.lm_head.cuda(),
                   [{k: v.cuda() for k, v in lw.items()} for lw in w.layers])
    model = P.SwiftKVModel(shape, wc, torch.float32, sum(lens), len(lens), l, g)
    st_gpu = {k: [None if t is None else t.cuda() for t in v] for k, v in st.items()}
    loss, grads = model.distill_grads(tok, lens, l, g, tau, st_gpu)
    model.status()
    # fp32 arithmetic against fp64: rounding 6e-8 per operation, sums of up to a few thousand terms (x sqrt(n) ~ 50), about ten
    # dependent stages forward and backward -> a few 1e-5 at worst; measured 3e-6
    assert abs(float(loss) - want_loss) <= 2e-5 * want_loss, (float(loss), want_loss)
    worst = 0.0
    for name in ("wq", "wk", "wv"):
        for j in range(l, shape.n_layers):
            got, ref = to_np(grads[name][j]).astype(np.float64), want[name][j]
            if np.abs(ref).max() == 0.0:
                assert np.abs(got).max() == 0.0, (name, j)               # not a group leader: never read, zero gradient
                continue
            worst = max(worst, _rel(got, ref))
            assert _rel(got, ref) <= 5e-5, (name, j, _rel(got, ref))
    print(f"distill {shape.name} l={l} g={g}: loss {float(loss):.6f} (oracle {want_loss:.6f}), worst gradient rel-L2 {worst:.2e}")
    # bit-reproducible
    loss2, grads2 = model.distill_grads(tok, lens, l, g, tau, st_gpu)
    assert torch.equal(loss, loss2)
    assert all(torch.equal(a, b) for name in grads for a, b in zip(grads[name], grads2[name]) if a is not None)
    model.close()


@pytest.mark.parametrize("precision,loss_bar,grad_bar", [(1, 2e-5, 5e-5), (2, 5e-3, 2e-2)])
@pytest.mark.parametrize("shape,lens,l,g,scale", [(MID, [64, 32], 2, 1, 2.0), (MID, [96, 31, 1], 1, 2, 2.0), (W8B_2L, [64, 32], 1, 1, 1.5)])
def test_tensor_core_modes_against_oracle(precision, loss_bar, grad_bar, shape, lens, l, g, scale):
    """The GEMMs of the step on the tensor cores (tcgen05 kind::tf32).  Split operands (each an exact sum of two tf32 numbers,
    three products): the same bars as the fp32 mode.  Plain tf32 (operands cut to 10 mantissa bits, 2^-10 relative each,
    systematic because the hardware truncates): gradients to 2e-2.  MID's widths are multiples of 128, so every projection and
    data gradient runs on the tensor-core kernel; the weight gradients do when the token count is a multiple of 32 (96), and
    fall back to the CUDA-core kernel otherwise (128).  The case at the benchmark model's layer widths (inner dimensions 4096 and
    14336) is the one that shows how the tensor core accumulates: it cuts instead of rounding, so a long chain drifts; the split
    mode keeps its chains at 1024 and meets the fp32 bar there too (1.5e-4 with whole-K chains, 3e-5 with chunks)."""
    import paper_2410_03960_b200 as P
    seed, tau = 29, 2.0
    w = _scaled_weights(shape, seed, scale)
    tok = S.make_prompts(seed, lens, shape.vocab)
    st = _student(w, l, seed + 1, 0.3)
    want_loss, want = D.distill_grads(oracle_config(shape), oracle_weights(w),
                                      {k: [None if t is None else t.double().numpy() for t in v] for k, v in st.items()},
                                      tok.numpy(), lens, l, g, tau)
    wc = S.Weights(shape, torch.float32, w.embed.cuda(), w.final_norm.cuda(), w.lm_head.cuda(),
                   [{k: v.cuda() for k, v in lw.items()} for lw in w.layers])
    model = P.SwiftKVModel(shape, wc, torch.float32, sum(lens), len(lens), l, g)
    st_gpu = {k: [None if t is None else t.cuda() for t in v] for k, v in st.items()}
    loss, grads = model.distill_grads(tok, lens, l, g, tau, st_gpu, precision=precision)
    model.status()
    assert abs(float(loss) - want_loss) <= loss_bar * want_loss, (float(loss), want_loss)
    worst = 0.0
    for name in ("wq", "wk", "wv"):
        for j in range(l, shape.n_layers):
            got, ref = to_np(grads[name][j]).astype(np.float64), want[name][j]
            if np.abs(ref).max() == 0.0:
                assert np.abs(got).max() == 0.0
                continue
            worst = max(worst, _rel(got, ref))
            assert _rel(got, ref) <= grad_bar, (name, j, _rel(got, ref))
    print(f"distill {shape.name} precision {precision} lens {lens}: loss rel {abs(float(loss) - want_loss) / want_loss:.2e}, worst gradient rel-L2 {worst:.2e}")
    loss2, grads2 = model.distill_grads(tok, lens, l, g, tau, st_gpu, precision=precision)
    assert torch.equal(loss, loss2) and all(torch.equal(a, b) for n_ in grads for a, b in zip(grads[n_], grads2[n_]) if a is not None)
    model.close()


def test_unrewired_student_has_no_loss_and_a_gradient_step_lowers_the_loss():
    import paper_2410_03960_b200 as P
    shape, lens, tau = SIX, [30, 11], 2.0
    w = _scaled_weights(shape, 5, 3.0)
    wc = S.Weights(shape, torch.float32, w.embed.cuda(), w.final_norm.cuda(), w.lm_head.cuda(),
                   [{k: v.cuda() for k, v in lw.items()} for lw in w.layers])
    tok = S.make_prompts(5, lens, shape.vocab)
    model = P.SwiftKVModel(shape, wc, torch.float32, sum(lens), len(lens), 1, 1)
    # l = L - 1: the only re-wired layer reads x_{l+1} itself, so its K / V are the teacher's and the loss vanishes
    l = shape.n_layers - 1
    st = {name: [None if j < l else wc.layers[j][name].clone() for j in range(shape.n_layers)] for name in ("wq", "wk", "wv")}
    loss, grads = model.distill_grads(tok, lens, l, 1, tau, st)
    assert float(loss) <= 1e-9 and float(grads["wq"][l].abs().max()) <= 1e-6
    # l = 2, student initialised from the original weights (Sec. 3.4): plain gradient steps recover part of the gap
    l = 2
    st = {name: [None if j < l else wc.layers[j][name].clone() for j in range(shape.n_layers)] for name in ("wq", "wk", "wv")}
    loss0, grads = model.distill_grads(tok, lens, l, 1, tau, st)
    assert float(loss0) > 1e-3
    gnorm2 = sum(float((t.double() ** 2).sum()) for name in grads for t in grads[name] if t is not None)
    lr = 0.1 * float(loss0) / gnorm2                                   # a step that a linear model would turn into -10 %
    for name in st:
        for j in range(l, shape.n_layers):
            st[name][j] -= lr * grads[name][j]
    loss1, _ = model.distill_grads(tok, lens, l, 1, tau, st)
    assert float(loss1) < float(loss0) * 0.97, (float(loss0), float(loss1))
    model.close()


def test_bf16_model_with_fp32_student_copies():
    """A bf16 model's frozen weights are widened to fp32 inside the step (exactly), the student's copies and the gradients are
    fp32: same bars against the oracle run on the bf16 values."""
    import paper_2410_03960_b200 as P
    shape, lens, l, g, tau = MID, [33, 9, 70], 2, 2, 2.0
    w = _scaled_weights(shape, 23, 2.0)
    wb = S.Weights(shape, torch.bfloat16, w.embed.bfloat16(), w.final_norm.bfloat16(), w.lm_head.bfloat16(),
                   [{k: v.bfloat16() for k, v in lw.items()} for lw in w.layers])
    w32 = S.Weights(shape, torch.float32, wb.embed.float(), wb.final_norm.float(), wb.lm_head.float(),
                    [{k: v.float() for k, v in lw.items()} for lw in wb.layers])
    tok = S.make_prompts(23, lens, shape.vocab)
    st = _student(w32, l, 24, 0.3)
    want_loss, want = D.distill_grads(oracle_config(shape), oracle_weights(w32),
                                      {k: [None if t is None else t.double().numpy() for t in v] for k, v in st.items()},
                                      tok.numpy(), lens, l, g, tau)
    wc = S.Weights(shape, torch.bfloat16, wb.embed.cuda(), wb.final_norm.cuda(), wb.lm_head.cuda(),
                   [{k: v.cuda() for k, v in lw.items()} for lw in wb.layers])
    model = P.SwiftKVModel(shape, wc, torch.bfloat16, sum(lens), len(lens), l, g)
    loss, grads = model.distill_grads(tok, lens, l, g, tau, {k: [None if t is None else t.cuda() for t in v] for k, v in st.items()})
    model.status()
    assert abs(float(loss) - want_loss) <= 2e-5 * want_loss, (float(loss), want_loss)
    for name in ("wq", "wk", "wv"):
        for j in range(l, shape.n_layers):
            got, ref = to_np(grads[name][j]).astype(np.float64), want[name][j]
            if np.abs(ref).max() == 0.0:
                assert np.abs(got).max() == 0.0
            else:
                assert _rel(got, ref) <= 5e-5, (name, j, _rel(got, ref))
    # the prefill path of the same handle still works afterwards
    model.prefill(tok, lens, l, g)
    model.status()
    assert torch.isfinite(model.first_logits()).all()
    model.close()


def test_argument_checks():
    import paper_2410_03960_b200 as P
    shape, lens = S.TINY, [8]
    w = S.make_weights(shape, 1, torch.float32, "cuda")
    model = P.SwiftKVModel(shape, w, torch.float32, 8, 1, 2, 1)
    st = {name: [None, None] + [w.layers[j][name].clone() for j in range(2, shape.n_layers)] for name in ("wq", "wk", "wv")}
    tok = S.make_prompts(1, lens, shape.vocab)
    for bad in (dict(swift_layer=0), dict(swift_layer=shape.n_layers + 1), dict(acrosskv_group=0), dict(temperature=0.0)):
        args = dict(swift_layer=2, acrosskv_group=1, temperature=2.0)
        args.update(bad)
        with pytest.raises(P.SwiftKVError) as e:
            model.distill_grads(tok, lens, args["swift_layer"], args["acrosskv_group"], args["temperature"], st)
        assert e.value.code == -1, bad          # SWIFTKV_ERR_INVALID_ARG
    st["wk"][3] = None                          # a missing student matrix of a re-wired layer
    with pytest.raises((P.SwiftKVError, AssertionError)):
        model.distill_grads(tok, lens, 2, 1, 2.0, st)
    model.close()


def test_adamw_update_against_oracle_and_a_short_training_run():
    """The update that goes with the gradients (AdamW, the paper's lr 3e-4 / weight decay 0.05): elementwise parity with the
    oracle's formula over three steps, then eight distillation steps on one batch with the student initialised from the
    original weights -- the loss must fall steadily (knowledge recovery at toy scale, Sec. 3.4)."""
    import paper_2410_03960_b200 as P
    rng = np.random.default_rng(9)
    p0 = rng.standard_normal(10007).astype(np.float32)
    p, m, v = p0.astype(np.float64), np.zeros(10007), np.zeros(10007)
    tp, tm, tv = torch.tensor(p0).cuda(), torch.zeros(10007, device="cuda"), torch.zeros(10007, device="cuda")
    for step in range(1, 4):
        g = (rng.standard_normal(10007) * 10.0 ** -step).astype(np.float32)
        f32 = lambda x: float(np.float32(x))                           # the C ABI takes the hyper-parameters as floats  # noqa: E731
        p, m, v = D.adamw_update(p, g.astype(np.float64), m, v, step, f32(3e-4), f32(0.9), f32(0.999), f32(1e-8), f32(0.05))
        P.adamw_update(tp, torch.tensor(g).cuda(), tm, tv, step)
        assert np.abs(to_np(tp) - p).max() <= 2e-6 * np.abs(p).max()
        assert _rel(to_np(tm).astype(np.float64), m) <= 1e-6 and _rel(to_np(tv).astype(np.float64), v) <= 1e-6

    shape, lens, l, tau = SIX, [40, 23], 2, 2.0
    w = _scaled_weights(shape, 5, 3.0)
    wc = S.Weights(shape, torch.float32, w.embed.cuda(), w.final_norm.cuda(), w.lm_head.cuda(),
                   [{k: t.cuda() for k, t in lw.items()} for lw in w.layers])
    tok = S.make_prompts(5, lens, shape.vocab)
    model = P.SwiftKVModel(shape, wc, torch.float32, sum(lens), len(lens), l, 1)
    st = {name: [None if j < l else wc.layers[j][name].clone() for j in range(shape.n_layers)] for name in ("wq", "wk", "wv")}
    state = {name: [None if t is None else (torch.zeros_like(t), torch.zeros_like(t)) for t in st[name]] for name in st}
    losses = []
    for step in range(1, 9):
        loss, grads = model.distill_grads(tok, lens, l, 1, tau, st)
        losses.append(float(loss))
        for name in st:
            for j in range(l, shape.n_layers):
                P.adamw_update(st[name][j].view(-1), grads[name][j].view(-1), state[name][j][0].view(-1), state[name][j][1].view(-1),
                               step, lr=3e-3, weight_decay=0.05)
    torch.cuda.synchronize()
    assert all(b < a for a, b in zip(losses, losses[1:])), losses
    assert losses[-1] < 0.7 * losses[0], losses
    print("distillation losses over 8 AdamW steps:", [round(x, 5) for x in losses])
    model.close()
