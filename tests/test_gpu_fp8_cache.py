"""Per-token FP8 (e4m3) KV cache (the paper's appendix on KV quantization: SwiftKV / AcrossKV combined with a
per-token FP8 cache).  Three levels:
  1. the quantizing row pass alone: codes and scales are bit-exact functions of the fp32 input, compared with the
     oracle's quantizer on the same bits;
  2. single-query attention reading codes + scales, against the oracle's attention over the dequantized rows;
  3. the whole prefill / chunked steps with an FP8 cache against the oracle's quantized model.  The stored codes are
     integers decided by floating-point values that the two sides compute with different rounding, so a value that
     sits within that rounding of a decision boundary lands on a neighbouring code -- a 6-12 % jump of that cache
     entry, which the following layers see as input noise.  fp32 model: the inputs agree to ~1e-6 and the bars are
     tight absolute ones.  bf16 model: the oracle is run twice, with the rows quantized from bf16 (the precision the
     kernel decides in: the reference) and from fp32; the distance between these two oracle results measures how far
     a 2^-9 relative change of the quantizer's input moves this model, and the CUDA path -- whose arithmetic differs
     from fp64 by about that much -- must stay within 1.25 times that distance of the reference (rel-L2 of the
     dequantized rows; 1.5 times for the code-flip rate, twice for the scales and the logits), per layer and tensor.
     Whatever happened upstream, every stored row must be a valid representation: row maximum on the largest code,
     scale * 448 = that maximum, and re-quantizing the dequantized row with the oracle returns the stored codes."""
import numpy as np
import pytest
import torch

import synthetic_inputs as S
from oracle import swiftkv_oracle as O
from helpers import oracle_config, oracle_weights, rel_l2, to_np

pytestmark = pytest.mark.gpu

MID = S.ModelShape(1024, 512, 4, 8, 2, 128, 1024, 500000.0, 1e-5, "mid")


def test_quantizer_bit_exact_against_oracle():
    import paper_2410_03960_b200 as P
    g = torch.Generator().manual_seed(3)
    for rows, width in [(1, 8), (37, 64), (301, 1024), (5, 1000)]:
        x = torch.randn(rows, width, generator=g) * torch.exp(torch.empty(rows, 1).uniform_(-20, 20, generator=g))
        x[0, : min(width, 4)] = torch.tensor([0.0, -0.0, 1e-30, -3e38])[: min(width, 4)]
        if rows > 3:
            x[2] = 0.0                                          # all-zero row
            x[3] = torch.linspace(-1, 1, width)                 # many values on or near decision boundaries
        # exact ties: midpoints between neighbouring codes, in a row whose maximum is exactly 448 (scale 1)
        if rows > 4:
            vals = O.e4m3_decode(np.arange(0x7F))
            mid = ((vals[:-1] + vals[1:]) / 2)[: width - 1]
            x[4] = 0.0
            x[4, : len(mid)] = torch.from_numpy(mid.astype(np.float32))
            x[4, -1] = 448.0
        codes, scales, deq = P.quantize_rows_fp8(x.cuda())
        rc, rs, rd = O.quantize_per_token(x.numpy())
        assert np.array_equal(scales.cpu().numpy(), rs)
        assert np.array_equal(codes.cpu().numpy(), rc)
        assert np.allclose(to_np(deq), rd, rtol=2.0 ** -23, atol=0)


@pytest.mark.parametrize("n_q,n_kv,hd", [(8, 2, 128), (32, 8, 128), (4, 2, 32), (6, 3, 64)])
def test_tail_attention_over_fp8_rows(n_q, n_kv, hd):
    import paper_2410_03960_b200 as P
    g = torch.Generator().manual_seed(7)
    lens = [1, 700, 129, 2500]
    T = sum(lens)
    k = torch.randn(T, n_kv * hd, generator=g) * torch.exp(torch.empty(T, 1).uniform_(-2, 2, generator=g))
    v = torch.randn(T, n_kv * hd, generator=g) * torch.exp(torch.empty(T, 1).uniform_(-2, 2, generator=g))
    q = torch.randn(len(lens), n_q, hd, generator=g) * 0.3
    kc, ks, kd = O.quantize_per_token(k.numpy())
    vc, vs, vd = O.quantize_per_token(v.numpy())
    out = P.tail_attention_fp8(q.cuda(), torch.from_numpy(kc).cuda().view(T, n_kv, hd), torch.from_numpy(vc).cuda().view(T, n_kv, hd),
                               torch.from_numpy(ks).cuda(), torch.from_numpy(vs).cuda(), lens)
    off = 0
    for b, n in enumerate(lens):
        ref = O.single_query_attention(q[b].double().numpy(), kd[off:off + n].reshape(n, n_kv, hd), vd[off:off + n].reshape(n, n_kv, hd))
        assert rel_l2(to_np(out[b]), ref.reshape(-1)) <= 1e-4, b
        off += n


def _stats(codes, scales, ref, j, name, n):
    """(rel-L2 of the dequantized rows, fraction of differing codes among the large entries, largest elementwise gap
    beyond one code step in units of the row maximum, largest relative scale gap) against ref's layer j."""
    ref_c = ref[name + "_codes"][j][:n]
    ref_s = ref[name + "_scale"][j][:n].astype(np.float64)
    got_v, ref_v = O.e4m3_decode(codes), O.e4m3_decode(ref_c)            # in units of the row's scale (max 448)
    mag = np.maximum(np.abs(got_v), np.abs(ref_v))
    step = np.where(mag < 2.0 ** -6, 2.0 ** -9, 2.0 ** (np.floor(np.log2(np.maximum(mag, 2.0 ** -6))) - 3))
    excess = float(np.maximum(np.abs(got_v - ref_v) - step, 0).max() / 448)
    big = np.abs(ref_v) >= 448 / 16
    flips = float((codes[big] != ref_c[big]).mean())
    rel = rel_l2(got_v * scales[:, None, None], ref[name][j][:n])
    return rel, flips, excess, float(np.abs(scales / ref_s - 1).max())


def _gpu_layer(model, j, rows):
    Kc, Vc, Ks, Vs, _ = model.kv_cache_view_fp8(j)
    rows_t = torch.as_tensor(rows, device="cuda")
    return {"K": (Kc[rows_t].cpu().numpy(), to_np(Ks[rows_t])), "V": (Vc[rows_t].cpu().numpy(), to_np(Vs[rows_t]))}


# GPU-to-reference distance over oracle-to-oracle distance (see the module docstring).  Measured: rel-L2 ratios 0.27 .. 1.07,
# code-flip ratios 0.15 .. 1.30 (tiny, mid and 8B-width shapes, both activation formats)
RATIO_CAP, FLIP_CAP, LOOSE_CAP = 1.25, 1.5, 2.0
RATIOS = []          # (layer, tensor, measured ratio) of the last checks, for the record (printed with -s)


def _check_representation(codes, scales, tag):
    """What a stored FP8 row must satisfy whatever happened upstream (the oracle as checker of the representation): the
    row maximum sits on the largest code (+-448), every code is finite, and quantizing the dequantized row -- value(code)
    * scale, one fp32 multiply -- with the oracle's quantizer returns the stored codes bit for bit and the stored scale to
    one fp32 rounding."""
    flat = codes.reshape(codes.shape[0], -1)
    mag = flat & 0x7F
    assert (mag != 0x7F).all(), (tag, "a NaN code is stored")
    nonzero = mag.max(axis=1) > 0
    assert (mag[nonzero].max(axis=1) == 0x7E).all(), (tag, "a row's maximum is not on the largest code")
    assert np.isfinite(scales).all() and (scales > 0).all(), tag
    deq32 = (O.e4m3_decode(flat).astype(np.float32) * scales.astype(np.float32)[:, None]).astype(np.float32)
    c2, s2, _ = O.quantize_per_token(deq32)
    assert np.array_equal(c2[nonzero] & 0x7F, flat[nonzero] & 0x7F), (tag, "re-quantizing the stored row changes its codes")
    sign_matters = (flat & 0x7F) != 0                      # (+0 and -0 are the same value)
    assert np.array_equal((c2 & 0x80)[sign_matters & nonzero[:, None]], (flat & 0x80)[sign_matters & nonzero[:, None]]), tag
    assert np.allclose(s2[nonzero].astype(np.float64), scales[nonzero].astype(np.float64), rtol=2.0 ** -22, atol=0), tag
    assert np.allclose(np.abs(deq32[nonzero]).max(axis=1), 448.0 * scales[nonzero].astype(np.float64), rtol=2.0 ** -22, atol=0), \
        (tag, "scale * 448 is not the row maximum")


def _check_fp8_layer(model, ref, j, rows, n, other=None):
    """fp32 model (other is None): tight absolute bars.  bf16 model: within RATIO_CAP times the distance between the two
    oracle evaluations `ref` (rows quantized from bf16) and `other` (from fp32), plus a small floor.  Either way the stored
    representation is checked absolutely."""
    got = _gpu_layer(model, j, rows)
    for name in ("K", "V"):
        _check_representation(got[name][0], got[name][1], (name, j))
        rel, flips, excess, ds = _stats(got[name][0], got[name][1], ref, j, name, n)
        if other is None:
            assert rel <= 2e-3 and flips <= 1e-3 and excess <= 1e-4 and ds <= 1e-4, (name, j, rel, flips, excess, ds)
        else:
            o_rel, o_flips, o_excess, o_ds = _stats(other[name + "_codes"][j][:n], other[name + "_scale"][j][:n].astype(np.float64),
                                                    ref, j, name, n)
            RATIOS.append((j, name, round(rel / max(o_rel, 1e-12), 3), round(flips / max(o_flips, 1e-12), 3)))
            assert rel <= RATIO_CAP * o_rel + 5e-3, (name, j, rel, o_rel)
            assert flips <= FLIP_CAP * o_flips + 0.02, (name, j, flips, o_flips)
            assert excess <= LOOSE_CAP * o_excess + 0.01, (name, j, excess, o_excess)
            assert ds <= LOOSE_CAP * o_ds + 0.01, (name, j, ds, o_ds)


def _refs(cfg, ow, tok, lens, l, g, dtype):
    """(reference, second oracle evaluation for the sensitivity bars or None, logits bar)."""
    if dtype == torch.float32:
        return O.swiftkv(cfg, ow, tok, lens, l, g, kv_fp8=True), None, 5e-3
    ref = O.swiftkv(cfg, ow, tok, lens, l, g, kv_fp8=True, row_dtype="bf16")
    other = O.swiftkv(cfg, ow, tok, lens, l, g, kv_fp8=True)
    return ref, other, 2 * float(np.max(np.abs(other["logits"] - ref["logits"]))) + 0.02


@pytest.mark.parametrize("shape,dtype,act", [
    (S.TINY, torch.float32, None),
    (S.TINY, torch.bfloat16, 1),
    (MID, torch.bfloat16, 1),
    (MID, torch.bfloat16, 0),
])
@pytest.mark.parametrize("l,g", [(2, 1), (1, 2), (4, 1)])
def test_prefill_with_fp8_cache(shape, dtype, act, l, g):
    import paper_2410_03960_b200 as P
    seed, lens = 13, [300, 77, 129]
    w = S.make_weights(shape, seed, dtype, "cuda")
    cfg, ow = oracle_config(shape), oracle_weights(w)
    tok = S.make_prompts(seed, lens, shape.vocab)
    model = P.SwiftKVModel(shape, w, dtype, sum(lens), len(lens), l, g, kv_format=P.KV_FP8)
    if act is not None:
        model.set_activation_format(act)
    model.prefill(tok, lens, l, g)
    model.status()
    ref, other, lg_bar = _refs(cfg, ow, tok.numpy(), lens, l, g, dtype)
    n = sum(lens)
    for j in range(shape.n_layers):
        _check_fp8_layer(model, ref, j, np.arange(n), n, other)
    if other is not None:            # first layer: nothing upstream has been quantized, so absolute bars hold as well
        for name in ("K", "V"):
            rel, flips, _, _ = _stats(*_gpu_layer(model, 0, np.arange(n))[name], ref, 0, name, n)
            assert rel <= 2e-2 and flips <= 0.06, (name, rel, flips)
    lg = to_np(model.first_logits())
    print("fp8 prefill", shape.name, dtype, act, l, g, "GPU/oracle distance ratios (layer, tensor, rel-L2, flips):",
          RATIOS[-2 * shape.n_layers:] if other is not None else "n/a (fp32: absolute bars)",
          "logits", float(np.max(np.abs(lg - ref["logits"]))), "bar", lg_bar)
    assert np.max(np.abs(lg - ref["logits"])) <= lg_bar, (float(np.max(np.abs(lg - ref["logits"]))), lg_bar)
    # memory: codes + one fp32 scale per row and plane instead of 16-bit (32-bit) elements
    _, kv16 = P.workspace_bytes(shape, dtype, 4096, 4, l, g)
    _, kv8 = P.workspace_bytes(shape, dtype, 4096, 4, l, g, P.KV_FP8)
    d_kv = shape.n_kv_heads * shape.head_dim
    assert kv8 * (2 if dtype == torch.bfloat16 else 4) * d_kv == kv16 * (d_kv + 4)


@pytest.mark.parametrize("shape,dtype,act", [(S.TINY, torch.float32, None), (MID, torch.bfloat16, 1)])
@pytest.mark.parametrize("paged", [False, True])
def test_chunked_steps_with_fp8_cache(shape, dtype, act, paged):
    """Chunks and decode tokens read earlier rows back from the FP8 cache: still the oracle's one-shot quantized model."""
    import paper_2410_03960_b200 as P
    seed, lens, l, g, n_decode = 29, [260, 90], 2, 1, 2
    w = S.make_weights(shape, seed, dtype, "cuda")
    cfg, ow = oracle_config(shape), oracle_weights(w)
    toks = [S.token_ids(seed, b, n + n_decode, shape.vocab) for b, n in enumerate(lens)]
    pages = [[5, 1, 3], [4]]
    where = (lambda b: pages[b]) if paged else (lambda b: b * 384)
    model = P.SwiftKVModel(shape, w, dtype, 768, 2, l, g, kv_format=P.KV_FP8)
    if act is not None:
        model.set_activation_format(act)
    cut = 100
    model.step(torch.cat([toks[0][:cut], toks[1][:lens[1]]]), [(cut, 0, where(0), 0), (lens[1], 0, where(1), 1)], l, g)
    model.step(toks[0][cut:lens[0]], [(lens[0] - cut, cut, where(0), 1)], l, g)
    for t in range(n_decode):
        model.step(torch.stack([toks[b][n + t] for b, n in enumerate(lens)]),
                   [(1, n + t, where(b), 1) for b, n in enumerate(lens)], l, g)
    model.status()
    lg = to_np(model.first_logits())
    for b, n in enumerate(lens):
        m = n + n_decode
        ref, other, lg_bar = _refs(cfg, ow, toks[b][:m].numpy(), [m], l, g, dtype)
        p = np.arange(m)
        rows = (np.asarray(pages[b])[p // 128] * 128 + p % 128) if paged else b * 384 + p
        for j in range(shape.n_layers):
            _check_fp8_layer(model, ref, j, rows, m, other)
        assert np.max(np.abs(lg[b] - ref["logits"][0])) <= lg_bar, b


def test_fp8_cache_at_8b_widths():
    """Llama-3.1-8B layer widths (4 layers): tcgen05 GEMMs and attention, vectorized row pass, group-by-group
    SingleInputKV projection with 2-way AcrossKV."""
    import paper_2410_03960_b200 as P
    shape = S.ModelShape(128256, 4096, 4, 32, 8, 128, 14336, 500000.0, 1e-5, "8b-width-4-layers")
    seed, lens, l, g = 2, [257, 130], 2, 2
    w = S.make_weights(shape, seed, torch.bfloat16, "cuda")
    cfg, ow = oracle_config(shape), oracle_weights(w)
    tok = S.make_prompts(seed, lens, shape.vocab)
    model = P.SwiftKVModel(shape, w, torch.bfloat16, sum(lens), len(lens), l, g, kv_format=P.KV_FP8)
    model.prefill(tok, lens, l, g)
    model.status()
    ref, other, lg_bar = _refs(cfg, ow, tok.numpy(), lens, l, g, torch.bfloat16)
    n = sum(lens)
    for j in range(shape.n_layers):
        _check_fp8_layer(model, ref, j, np.arange(n), n, other)
    for name in ("K", "V"):
        rel, flips, _, _ = _stats(*_gpu_layer(model, 0, np.arange(n))[name], ref, 0, name, n)
        assert rel <= 2e-2 and flips <= 0.06, (name, rel, flips)
    assert model.kv_cache_view_fp8(3)[4] == 2 and model.kv_cache_view_fp8(2)[0].data_ptr() == model.kv_cache_view_fp8(3)[0].data_ptr()
    err = float(np.max(np.abs(to_np(model.first_logits()) - ref["logits"])))
    print("fp8 at 8B widths: GPU/oracle distance ratios (layer, tensor, rel-L2, flips):", RATIOS[-2 * shape.n_layers:], "logits", err, "bar", lg_bar)
    assert err <= lg_bar, (err, lg_bar)
