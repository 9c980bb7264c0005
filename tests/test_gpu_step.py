"""Chunked prefill and decode steps (the paper's Sec. 3.5 deployment: minibatches that mix chunks of prefill tokens and
decode tokens; after layer l the later layers' caches are filled and only the tokens that must produce output go
on).  Feeding a sequence in chunks, or one token at a time, is an exact reformulation: the caches and logits must
equal the oracle's one-shot SwiftKV prefill of the same token sequence."""
import numpy as np
import pytest
import torch

import synthetic_inputs as S
from oracle import swiftkv_oracle as O
from helpers import oracle_config, oracle_weights, rel_l2, to_np

pytestmark = pytest.mark.gpu

MID = S.ModelShape(1024, 512, 4, 8, 2, 128, 1024, 500000.0, 1e-5, "mid")


def _check_seq(model, shape, ref, row0, n, kv_bar):
    for j in range(shape.n_layers):
        K, V, _ = model.kv_cache_view(j)
        assert rel_l2(to_np(K[row0:row0 + n]), ref["K"][j][:n]) <= kv_bar, j
        assert rel_l2(to_np(V[row0:row0 + n]), ref["V"][j][:n]) <= kv_bar, j


@pytest.mark.parametrize("shape,dtype,act,kv_bar,lg_bar", [
    (S.TINY, torch.float32, None, 1e-4, 1e-3),
    (S.TINY, torch.bfloat16, 1, 2e-2, 0.1),
    (MID, torch.bfloat16, 1, 2e-2, 0.1),        # tensor-core kernels, half activations (gathered half K / V copies)
    (MID, torch.bfloat16, 0, 2e-2, 0.1),        # tensor-core kernels reading the bf16 cache in place
])
@pytest.mark.parametrize("l,g", [(2, 1), (1, 2), (4, 1)])
def test_chunked_prefill_then_decode(shape, dtype, act, kv_bar, lg_bar, l, g):
    import paper_2410_03960_b200 as P
    seed = 11
    lens = [300, 77, 129]                      # prompt lengths
    n_decode = 3
    cap = 512                                  # cache rows reserved per sequence
    w = S.make_weights(shape, seed, dtype, "cuda")
    cfg, ow = oracle_config(shape), oracle_weights(w)
    toks = [S.token_ids(seed, b, n + n_decode, shape.vocab) for b, n in enumerate(lens)]   # prompt + "generated" tokens
    model = P.SwiftKVModel(shape, w, dtype, cap * len(lens), len(lens), min(l, 1), 1)
    if act is not None:
        model.set_activation_format(act)

    # ---- chunked prefill: 100-token chunks, all sequences that still have prompt left share a minibatch
    chunk = 100
    done = [0] * len(lens)
    last_logits = {}
    while any(d < n for d, n in zip(done, lens)):
        seqs, packed, emitting = [], [], []
        for b, n in enumerate(lens):
            if done[b] >= n:
                continue
            k = min(chunk, n - done[b])
            emit = int(done[b] + k == n)
            seqs.append((k, done[b], b * cap, emit))
            packed.append(toks[b][done[b]:done[b] + k])
            if emit:
                emitting.append(b)
            done[b] += k
        model.step(torch.cat(packed), seqs, l, g)     # (steps in which nobody emits only fill caches)
        model.status()
        lg = model.first_logits().clone()
        assert lg.shape[0] == len(emitting)
        for i, b in enumerate(emitting):
            last_logits[b] = lg[i]
    for b, n in enumerate(lens):
        ref = O.swiftkv(cfg, ow, toks[b][:n].numpy(), [n], l, g)
        _check_seq(model, shape, ref, b * cap, n, kv_bar)
        assert np.max(np.abs(to_np(last_logits[b]) - ref["logits"][0])) <= lg_bar, b

    # ---- decode: every sequence appends one token per step (a minibatch of decode tokens)
    for t in range(n_decode):
        seqs = [(1, n + t, b * cap, 1) for b, n in enumerate(lens)]
        model.step(torch.stack([toks[b][n + t] for b, n in enumerate(lens)]), seqs, l, g)
        model.status()
        lg = to_np(model.first_logits())
        for b, n in enumerate(lens):
            ref = O.swiftkv(cfg, ow, toks[b][:n + t + 1].numpy(), [n + t + 1], l, g)
            assert np.max(np.abs(lg[b] - ref["logits"][0])) <= lg_bar, (t, b)
            if t == n_decode - 1:
                _check_seq(model, shape, ref, b * cap, n + t + 1, kv_bar)


@pytest.mark.parametrize("shape,dtype,bar", [(S.TINY, torch.float32, 1e-3), (MID, torch.bfloat16, 0.1)])
def test_decode_minibatch_on_both_paths(shape, dtype, bar):
    """A decode-only minibatch of at most 8 sequences runs every layer on the weight-streaming kernels (kernel-mask
    bit 5); with the bit cleared it takes the general path (128-row GEMM tiles, gathered attention operands).  Both must
    give the oracle's logits and caches."""
    import paper_2410_03960_b200 as P
    seed, lens, l, g, cap = 17, [140, 33, 260], 2, 2, 384
    w = S.make_weights(shape, seed, dtype, "cuda")
    cfg, ow = oracle_config(shape), oracle_weights(w)
    toks = [S.token_ids(seed, b, n + 2, shape.vocab) for b, n in enumerate(lens)]
    out = {}
    for mask in (55, 39, 7):
        model = P.SwiftKVModel(shape, w, dtype, cap * len(lens), len(lens), l, g)
        assert model.set_kernel_mask(mask) == mask
        model.step(torch.cat([t[:n] for t, n in zip(toks, lens)]), [(n, 0, b * cap, 1) for b, n in enumerate(lens)], l, g)
        for t in range(2):
            model.step(torch.stack([toks[b][n + t] for b, n in enumerate(lens)]),
                       [(1, n + t, b * cap, 1) for b, n in enumerate(lens)], l, g)
        model.status()
        out[mask] = to_np(model.first_logits())
        for b, n in enumerate(lens):
            ref = O.swiftkv(cfg, ow, toks[b][:n + 2].numpy(), [n + 2], l, g)
            assert np.max(np.abs(out[mask][b] - ref["logits"][0])) <= bar, (mask, b)
            _check_seq(model, shape, ref, b * cap, n + 2, 1e-4 if dtype == torch.float32 else 2e-2)
    assert np.max(np.abs(out[39] - out[7])) <= 2 * bar


def test_mixed_minibatch_of_prefill_chunk_and_decode_token():
    """One step carries a decode token of sequence 0 and a prefill chunk of sequence 1; only sequence 0 emits."""
    import paper_2410_03960_b200 as P
    shape, dtype, l, g, cap = MID, torch.bfloat16, 2, 1, 512
    w = S.make_weights(shape, 5, dtype, "cuda")
    cfg, ow = oracle_config(shape), oracle_weights(w)
    t0, t1 = S.token_ids(5, 0, 141, shape.vocab), S.token_ids(5, 1, 260, shape.vocab)
    model = P.SwiftKVModel(shape, w, dtype, 2 * cap, 2, l, g)
    model.step(t0[:140], [(140, 0, 0, 1)], l, g)                                     # prompt of sequence 0
    model.step(torch.cat([t0[140:141], t1[:130]]), [(1, 140, 0, 1), (130, 0, cap, 0)], l, g)   # decode + first chunk
    model.status()
    lg = to_np(model.first_logits())
    assert lg.shape[0] == 1
    ref0 = O.swiftkv(cfg, ow, t0.numpy(), [141], l, g)
    assert np.max(np.abs(lg[0] - ref0["logits"][0])) <= 0.1
    model.step(t1[130:], [(130, 130, cap, 1)], l, g)                                 # second chunk of sequence 1
    model.status()
    ref1 = O.swiftkv(cfg, ow, t1.numpy(), [260], l, g)
    assert np.max(np.abs(to_np(model.first_logits())[0] - ref1["logits"][0])) <= 0.1
    _check_seq(model, shape, ref0, 0, 141, 2e-2)
    _check_seq(model, shape, ref1, cap, 260, 2e-2)


def test_step_argument_checks():
    import paper_2410_03960_b200 as P
    shape = S.TINY
    w = S.make_weights(shape, 0, torch.float32, "cuda")
    model = P.SwiftKVModel(shape, w, torch.float32, 256, 2, 2, 1)
    tok = S.token_ids(0, 0, 40, shape.vocab)
    for bad in ([(40, 0, 250, 1)],                      # runs past max_tokens
                [(20, 0, 0, 1), (20, 0, 10, 1)],        # overlapping regions
                [(0, 0, 0, 1)]):                        # empty chunk
        n = sum(s[0] for s in bad)
        with pytest.raises(P.SwiftKVError) as e:
            model.step(tok[:max(n, 1)] if n else tok[:0], bad, 2, 1)
        assert e.value.code == -1


def _paged_rows(pages, n):
    """Cache rows of tokens 0..n-1 of a sequence that owns `pages` (128-row pages)."""
    p = np.arange(n)
    return np.asarray(pages)[p // 128] * 128 + p % 128


@pytest.mark.parametrize("shape,dtype,act,kv_bar,lg_bar", [
    (S.TINY, torch.float32, None, 1e-4, 1e-3),  # SIMT kernels follow the block tables
    (MID, torch.bfloat16, 1, 2e-2, 0.1),        # half copies gathered through the block tables
    (MID, torch.bfloat16, 0, 2e-2, 0.1),        # tcgen05 attention fetches K / V tiles page by page
])
@pytest.mark.parametrize("l,g", [(2, 1), (1, 2)])
def test_paged_cache_chunks_and_decode(shape, dtype, act, kv_bar, lg_bar, l, g):
    """Sequences own scattered, interleaved 128-row pages instead of contiguous regions; results are unchanged."""
    import paper_2410_03960_b200 as P
    seed, lens, n_decode = 23, [300, 77, 129], 2
    n_pages = 12
    perm = [7, 2, 10, 0, 5, 11, 3, 8, 1, 9, 4, 6]                 # page numbers handed out round-robin
    pages = [perm[0:9:3], perm[1:4:3], perm[2:9:3][:2]]           # 3, 1, 2 pages: [7,0,3], [2], [10,11]
    w = S.make_weights(shape, seed, dtype, "cuda")
    cfg, ow = oracle_config(shape), oracle_weights(w)
    toks = [S.token_ids(seed, b, n + n_decode, shape.vocab) for b, n in enumerate(lens)]
    model = P.SwiftKVModel(shape, w, dtype, n_pages * 128, len(lens), min(l, 1), 1)
    if act is not None:
        model.set_activation_format(act)
    # two prefill steps (first 60 tokens, then the rest), then decode steps
    cut = 60
    model.step(torch.cat([t[:cut] for t in toks]), [(cut, 0, pages[b], int(b == 0)) for b in range(3)], l, g)
    model.step(torch.cat([toks[b][cut:n] for b, n in enumerate(lens)]),
               [(n - cut, cut, pages[b], 1) for b, n in enumerate(lens)], l, g)
    model.status()
    lg = to_np(model.first_logits())

    def check(n_extra, lg):
        for b, n in enumerate(lens):
            m = n + n_extra
            ref = O.swiftkv(cfg, ow, toks[b][:m].numpy(), [m], l, g)
            assert np.max(np.abs(lg[b] - ref["logits"][0])) <= lg_bar, (n_extra, b)
            rows = torch.as_tensor(_paged_rows(pages[b], m), device="cuda")
            for j in range(shape.n_layers):
                K, V, _ = model.kv_cache_view(j)
                assert rel_l2(to_np(K[rows]), ref["K"][j][:m]) <= kv_bar, (b, j)
                assert rel_l2(to_np(V[rows]), ref["V"][j][:m]) <= kv_bar, (b, j)

    check(0, lg)
    for t in range(n_decode):
        if t == 1:
            pages[2] = pages[2] + [4]          # a fresh page may join a table at any step (unused until needed)
        model.step(torch.stack([toks[b][n + t] for b, n in enumerate(lens)]),
                   [(1, n + t, pages[b], 1) for b, n in enumerate(lens)], l, g)
        model.status()
        check(t + 1, to_np(model.first_logits()))


def test_paged_argument_checks():
    import paper_2410_03960_b200 as P
    shape = S.TINY
    w = S.make_weights(shape, 0, torch.float32, "cuda")
    model = P.SwiftKVModel(shape, w, torch.float32, 512, 2, 2, 1)      # 4 pages
    tok = S.token_ids(0, 0, 300, shape.vocab)
    for bad, n in (([(200, 0, [0], 1)], 200),                       # 2 pages needed, 1 listed
                   ([(100, 0, [4], 1)], 100),                       # page outside the cache
                   ([(100, 0, [1], 1), (100, 0, [1], 1)], 200),     # page listed twice
                   ([(100, 0, [1], 1), (100, 0, 0, 1)], 200)):      # paged and contiguous sequences mixed
        with pytest.raises(P.SwiftKVError) as e:
            model.step(tok[:n], bad, 2, 1)
        assert e.value.code == -1


W8B_4L = S.ModelShape(128256, 4096, 4, 32, 8, 128, 14336, 500000.0, 1e-5, "8b-width-4-layers")


@pytest.mark.parametrize("act,paged", [(1, False), (1, True), (0, False)])
def test_chunked_prefill_and_decode_at_8b_widths(act, paged):
    """The deployment path at the real Llama-3.1-8B widths (hidden 4096, 32 / 8 heads, FFN 14336; 4 layers, l = 2):
    chunks that are not multiples of the 128-row tiles and attend to a cached prefix, then three decode steps on the
    fused persistent launch (kernel-mask bits 5 and 6, the default), on the per-operator weight-streaming kernels (bit 5) and on
    the general path, each on a model of its own -- contiguous regions and
    scattered pages, both activation formats -- against the oracle's one-shot prefill of the same token sequences."""
    import paper_2410_03960_b200 as P
    shape, dtype, seed, l, g = W8B_4L, torch.bfloat16, 13, 2, 1
    # The 2e-2 / 0.1 bars hold for the default half activations.  With bfloat16 activations (act 0) four layers of these
    # widths sit at that format's own floor -- every stored activation rounds at 2^-9; measured max-abs 0.100 here, 0.089
    # in the one-shot prefill -- so that format is held to 0.15: what is checked for it is the wiring, not the format.
    abs_bar = 0.1 if act == 1 else 0.15
    lens, n_decode, chunk = [333, 128, 1, 200], 3, 150          # chunks of 150: 333 = 150 + 150 + 33
    cap_pages = 3                                                # 384 cache rows per sequence
    w = S.make_weights(shape, seed, dtype, "cuda")
    cfg, ow = oracle_config(shape), oracle_weights(w)
    toks = [S.token_ids(seed, b, n + n_decode, shape.vocab) for b, n in enumerate(lens)]
    refs = {}

    def ref_of(b, m):
        if (b, m) not in refs:
            refs[(b, m)] = O.swiftkv(cfg, ow, toks[b][:m].numpy(), [m], l, g)
        return refs[(b, m)]

    # scattered, interleaved pages for the paged variant; contiguous regions otherwise
    perm = [5, 0, 9, 2, 11, 7, 1, 10, 4, 8, 3, 6]
    pages = [perm[b::4][:cap_pages] for b in range(4)]
    where = (lambda b: pages[b]) if paged else (lambda b: b * cap_pages * 128)

    def rows_of(b, m):
        if paged:
            return torch.as_tensor(_paged_rows(pages[b], m), device="cuda")
        return torch.arange(b * cap_pages * 128, b * cap_pages * 128 + m, device="cuda")

    # decode steps on the fused persistent launch (the default: one launch per layer, K / V of the new token from the same
    # launch as Q, rows handed over pre-split between its stages), on the per-operator weight-streaming kernels, and on the
    # general path
    for mask in (119, 55, 23):
        model = P.SwiftKVModel(shape, w, dtype, 4 * cap_pages * 128, len(lens), l, g)
        model.set_kernel_mask(mask)
        model.set_activation_format(act)
        done, last = [0] * len(lens), {}
        while any(d < n for d, n in zip(done, lens)):
            seqs, packed, emitting = [], [], []
            for b, n in enumerate(lens):
                if done[b] >= n:
                    continue
                k = min(chunk, n - done[b])
                emit = int(done[b] + k == n)
                seqs.append((k, done[b], where(b), emit))
                packed.append(toks[b][done[b]:done[b] + k])
                if emit:
                    emitting.append(b)
                done[b] += k
            model.step(torch.cat(packed), seqs, l, g)
            model.status()
            lg = model.first_logits().clone()
            for i, b in enumerate(emitting):
                last[b] = lg[i]
        for b, n in enumerate(lens):
            assert np.max(np.abs(to_np(last[b]) - ref_of(b, n)["logits"][0])) <= abs_bar, (mask, b)
        for t in range(n_decode):
            model.step(torch.stack([toks[b][n + t] for b, n in enumerate(lens)]),
                       [(1, n + t, where(b), 1) for b, n in enumerate(lens)], l, g)
            model.status()
            lg = to_np(model.first_logits())
            for b, n in enumerate(lens):
                ref = ref_of(b, n + t + 1)
                assert rel_l2(lg[b], ref["logits"][0]) <= 2e-2, (mask, t, b)
                assert np.max(np.abs(lg[b] - ref["logits"][0])) <= abs_bar, (mask, t, b)
        for b, n in enumerate(lens):
            m = n + n_decode
            rows = rows_of(b, m)
            for j in range(shape.n_layers):
                K, V, _ = model.kv_cache_view(j)
                assert rel_l2(to_np(K[rows]), ref_of(b, m)["K"][j]) <= 2e-2, (mask, b, j)
                assert rel_l2(to_np(V[rows]), ref_of(b, m)["V"][j]) <= 2e-2, (mask, b, j)
        model.close()


def test_half_weight_cache_gives_the_same_bits_and_follows_weight_updates():
    """swiftkv_set_half_weight_cache: the half copies of the first layers' matrices made once and kept, instead of once per
    step.  Same conversion kernel, same GEMMs: logits and caches of chunked steps and of a one-shot prefill are bit-identical
    with and without it; a cache too small for the step's l falls back to per-step copies; after the caller changes a weight
    and sets the cache again, the result follows the new weight (and differs from the stale one)."""
    import paper_2410_03960_b200 as P
    shape, l, g, seed = MID, 3, 1, 23
    lens, cap, chunk = [300, 130], 384, 128
    w = S.make_weights(shape, seed, torch.bfloat16, "cuda")
    toks = [S.token_ids(seed, b, n, shape.vocab) for b, n in enumerate(lens)]

    def run(model):
        done = [0] * len(lens)
        while any(d < n for d, n in zip(done, lens)):
            seqs, packed = [], []
            for b, n in enumerate(lens):
                if done[b] < n:
                    k = min(chunk, n - done[b])
                    seqs.append((k, done[b], b * cap, int(done[b] + k == n)))
                    packed.append(toks[b][done[b]:done[b] + k])
                    done[b] += k
            model.step(torch.cat(packed), seqs, l, g)
        model.status()
        out = [model.first_logits().clone()]
        for j in range(shape.n_layers):
            K, V, _ = model.kv_cache_view(j)
            out += [K.clone(), V.clone()]
        return out

    model = P.SwiftKVModel(shape, w, torch.bfloat16, cap * len(lens), len(lens), l, g)
    plain = run(model)
    launches_plain = model.last_launch_count()
    assert model.set_half_weight_cache(l) == 2 * l * (2 * shape.hidden * shape.n_q_heads * shape.head_dim +
                                                      2 * shape.hidden * shape.n_kv_heads * shape.head_dim + 3 * shape.hidden * shape.ffn)
    first = run(model)          # makes the copies
    again = run(model)          # reuses them
    assert model.last_launch_count() == launches_plain - 7 * l          # the last step no longer copies 7 matrices per layer
    for a, b_, c in zip(plain, first, again):
        assert torch.equal(a, b_) and torch.equal(a, c)
    model.set_half_weight_cache(l - 1)                                   # too small for l: per-step copies again
    for a, b_ in zip(plain, run(model)):
        assert torch.equal(a, b_)
    assert model.last_launch_count() == launches_plain
    # a weight update: stale copies until the cache is set again
    model.set_half_weight_cache(l)
    run(model)
    w.layers[0]["w_down"].mul_(0.5)
    stale = run(model)
    assert all(torch.equal(a, b_) for a, b_ in zip(plain, stale))        # (documented: the library cannot see the change)
    model.set_half_weight_cache(l)
    fresh = run(model)
    model.set_half_weight_cache(0)
    uncached = run(model)
    assert not torch.equal(fresh[0], plain[0])
    for a, b_ in zip(fresh, uncached):
        assert torch.equal(a, b_)
    with pytest.raises(P.SwiftKVError):
        P.binding._check(model.lib.swiftkv_set_half_weight_cache(model._h, None, 256))
    model.close()
