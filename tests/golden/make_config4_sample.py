"""Writes tests/golden/config4_truncated_sample.npz: outputs of the CPU oracle for config 4 (Llama-3.1-70B shape, 80
layers, bf16-valued weights, SwiftKV l = 40, g = 1, the seed-3 varlen batch of prompts U[1024, 4096] totalling 16384
tokens) with every prompt cut to its first n/64 tokens -- a causal prefix of the real prompt, so ragged lengths
survive.  With `--full` it writes config4_full_sample.npz from the complete 16384-token batch instead (hours).

Calls only the oracle and the seeded input generators; the 141 GB model never exists at once: a layer's tensors are
generated when the oracle first reads them and dropped with the layer (peak host memory ~25 GB).  On host cores alone
nearly all of the time goes into the integer weight generator (hours); `--device cuda` lets the generator -- which
gives the same bits on either device and holds none of the method's arithmetic -- run its integer ops on a GPU, the
oracle itself stays on the host cores either way (a few minutes for the truncated batch):
    python tests/golden/make_config4_sample.py [--device cuda] [--full]
Stored (float32): the complete first-token logits of every prompt (so that the max-abs bar is taken over all 128256
entries), and for the layers in LAYERS the K and V rows of the first, the last and one seeded inner position of every
prompt.  The GPU parity test of config 4 compares exactly these entries."""
import os
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
import synthetic_inputs as S                      # noqa: E402
from oracle import swiftkv_oracle as O            # noqa: E402

SEED, TOTAL, LEN_LO, LEN_HI, SWIFT_LAYER, GROUP, FACTOR = 3, 16384, 1024, 4096, 40, 1, 64
LAYERS = (0, 9, 19, 29, 39, 40, 49, 59, 69, 79)       # 0-based: first, every tenth, both sides of the SwiftKV boundary, last


def batch(full: bool):
    lens = S.lengths_to_total(SEED, TOTAL, LEN_LO, LEN_HI)
    return lens if full else [max(1, n // FACTOR) for n in lens]


def sample_positions(lens):
    """The seeded choice of cache rows; the GPU test imports this function to read the same ones."""
    rng = np.random.default_rng(20241003)
    return [sorted({0, n - 1, int(rng.integers(0, n))}) for n in lens]


def main():
    full = "--full" in sys.argv
    device = sys.argv[sys.argv.index("--device") + 1] if "--device" in sys.argv else "cpu"
    shape = S.LLAMA31_70B
    lens = batch(full)
    name = "config4_full_sample.npz" if full else "config4_truncated_sample.npz"
    tok = S.make_prompts(SEED, lens, shape.vocab).numpy()
    t0 = time.time()

    def f64(t):
        return t.cpu().double().numpy()

    def lm_head():
        return f64(S.matrix(SEED, 0xF002, shape.vocab, shape.hidden, torch.bfloat16, device))

    d, dq, dkv, f = shape.hidden, shape.d_q, shape.d_kv, shape.ffn
    dims = {"wq": (1, dq, d), "wk": (2, dkv, d), "wv": (3, dkv, d), "wo": (4, d, dq), "w_gate": (6, f, d), "w_up": (7, f, d),
            "w_down": (8, d, f)}            # tensor ids and shapes of synthetic_inputs.layer_weights
    gains = {"in_norm": 0, "post_norm": 5}

    class LazyLayer(dict):
        """A layer's tensors, each generated when first read: the SingleInputKV pass reads only a later layer's gain,
        W_K and W_V, the last token's pass everything else."""
        def __init__(self, j):
            super().__init__()
            self.j = j

        def __missing__(self, key):
            t = 16 * self.j
            if key in gains:
                v = f64(S.gain(SEED, t + gains[key], d, torch.bfloat16, device))
            else:
                tid, rows, cols = dims[key]
                v = f64(S.matrix(SEED, t + tid, rows, cols, torch.bfloat16, device))
            self[key] = v
            return v

    cache = {}

    def layer_cached(j):
        if j not in cache:
            cache.clear()
            cache[j] = LazyLayer(j)
            print(f"layer {j} at {time.time() - t0:.0f} s", flush=True)
        return cache[j]

    W = O.Weights(lambda ids: f64(S.matrix_rows(SEED, 0xF000, torch.as_tensor(np.asarray(ids)), shape.hidden, torch.bfloat16)),
                  f64(S.gain(SEED, 0xF001, shape.hidden, torch.bfloat16, device)), lm_head, layer_cached)
    cfg = O.Config(shape.vocab, shape.hidden, shape.n_layers, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                   shape.ffn, shape.rope_theta, shape.rms_eps)
    ref = O.swiftkv(cfg, W, tok, lens, SWIFT_LAYER, GROUP)
    print(f"oracle {time.time() - t0:.0f} s", flush=True)
    pos = sample_positions(lens)
    off = np.concatenate([[0], np.cumsum(lens)])
    rows = np.concatenate([off[b] + np.asarray(p) for b, p in enumerate(pos)])
    out = {"lens": np.asarray(lens, dtype=np.int32), "rows": rows.astype(np.int32), "logits": ref["logits"].astype(np.float32)}
    for j in LAYERS:
        out[f"K{j}"] = ref["K"][j][rows].astype(np.float32)
        out[f"V{j}"] = ref["V"][j][rows].astype(np.float32)
    np.savez_compressed(os.path.join(os.path.dirname(os.path.abspath(__file__)), name), **out)
    print(f"done {time.time() - t0:.0f} s", flush=True)


if __name__ == "__main__":
    main()
