"""Writes tests/golden/config2_full_sample.npz: sampled outputs of the CPU oracle on the FULL benchmark workload
(Llama-3.1-8B shape, bf16-valued weights, SwiftKV l = 16, g = 1, 8 prompts with lengths U[2048, 8192], seed 1).
With `--sweep N` it writes tests/golden/sweep_n<N>_full_sample.npz instead: one prompt of N tokens, seed 4, l = 16 (a
point of the prompt-length sweep; N = 4096 takes about a quarter of an hour after the weights, N = 16384 about four hours).

Calls only the oracle and the seeded input generators.  Takes about two hours on 8 cores and ~35 GB of host memory:
    python tests/golden/make_config2_full_sample.py
Stored (float32): for every prompt the first-token logits at 2048 seeded vocabulary indices plus the arg-max index
and value; for layers 1, 16, 17 and 32 the K and V rows of four positions per prompt (first, last and two seeded
ones).  The GPU parity test of the full-size run compares exactly these entries."""
import os
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
import synthetic_inputs as S                      # noqa: E402
from oracle import swiftkv_oracle as O            # noqa: E402

SEED, N_PROMPTS, LEN_LO, LEN_HI, SWIFT_LAYER, GROUP = 1, 8, 2048, 8192, 16, 1
LAYERS = (0, 15, 16, 31)
N_VOCAB_SAMPLES, N_POS = 2048, 4


def sample_plan(lens, vocab):
    """The seeded choice of entries; the GPU test imports this function to read the same ones."""
    rng = np.random.default_rng(20241003)
    vocab_idx = np.stack([np.sort(rng.choice(vocab, N_VOCAB_SAMPLES, replace=False)) for _ in lens])
    pos = np.stack([np.array([0, n - 1] + sorted(rng.choice(np.arange(1, n - 1), N_POS - 2, replace=False).tolist()))
                    for n in lens])
    return vocab_idx, pos


def main():
    shape = S.LLAMA31_8B
    seed, lens, name = SEED, S.uniform_lengths(SEED, N_PROMPTS, LEN_LO, LEN_HI), "config2_full_sample.npz"
    if len(sys.argv) > 2 and sys.argv[1] == "--sweep":
        seed, lens, name = 4, [int(sys.argv[2])], f"sweep_n{int(sys.argv[2])}_full_sample.npz"
    tok = S.make_prompts(seed, lens, shape.vocab).numpy()
    t0 = time.time()
    w = S.make_weights(shape, seed, torch.bfloat16, "cpu")
    print(f"weights {time.time() - t0:.0f} s", flush=True)

    def f64(t):
        return t.double().numpy()

    W = O.Weights(lambda ids: f64(w.embed[torch.as_tensor(np.asarray(ids), dtype=torch.long)]), f64(w.final_norm),
                  lambda: f64(w.lm_head), lambda j: {k: f64(v) for k, v in w.layers[j].items()})
    cfg = O.Config(shape.vocab, shape.hidden, shape.n_layers, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                   shape.ffn, shape.rope_theta, shape.rms_eps)
    ref = O.swiftkv(cfg, W, tok, lens, SWIFT_LAYER, GROUP)
    print(f"oracle {time.time() - t0:.0f} s", flush=True)
    vocab_idx, pos = sample_plan(lens, shape.vocab)
    off = np.concatenate([[0], np.cumsum(lens)])
    rows = (off[:-1, None] + pos).reshape(-1)
    out = {
        "lens": np.asarray(lens, dtype=np.int32), "vocab_idx": vocab_idx.astype(np.int32), "pos": pos.astype(np.int32),
        "logits": np.take_along_axis(ref["logits"], vocab_idx, axis=1).astype(np.float32),
        "argmax": ref["logits"].argmax(axis=1).astype(np.int32), "max": ref["logits"].max(axis=1).astype(np.float32),
        "logits_norm": np.linalg.norm(ref["logits"], axis=1).astype(np.float32),
    }
    for j in LAYERS:
        out[f"K{j}"] = ref["K"][j][rows].astype(np.float32)
        out[f"V{j}"] = ref["V"][j][rows].astype(np.float32)
    np.savez(os.path.join(os.path.dirname(os.path.abspath(__file__)), name), **out)
    print(f"done {time.time() - t0:.0f} s", flush=True)


if __name__ == "__main__":
    main()
