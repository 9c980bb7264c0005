"""A small, self-terminating case for profiler captures:
    python -m paper_2410_03960_b200.profile_case [tokens [steps [layers [swift_layer [n_prompts]]]]]

Runs a few SwiftKV prefills (default l = 1 of 2 layers) of a model with the Llama-3.1-8B widths, so that
every hot kernel (the QKV / O / SwiGLU / down / SingleInputKV GEMMs, the flash-attention kernel, the norms and
the last-token path) launches with its real shapes while the process holds only a few GB: the weights of one
layer (436 MB) plus activations exceed the 126 MB L2, so DRAM counters stay meaningful.
Environment: SWIFTKV_KERNEL_MASK, SWIFTKV_ACT_FORMAT (0 bf16, 1 half), SWIFTKV_KV_FORMAT=fp8 (per-token FP8 cache).
"""
from __future__ import annotations

import os
import sys

import torch

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import synthetic_inputs as S  # noqa: E402

import paper_2410_03960_b200 as P  # noqa: E402


def main() -> None:
    tokens = int(sys.argv[1]) if len(sys.argv) > 1 else 8192
    steps = int(sys.argv[2]) if len(sys.argv) > 2 else 3
    layers = int(sys.argv[3]) if len(sys.argv) > 3 else 2
    l = int(sys.argv[4]) if len(sys.argv) > 4 else 1
    n_prompts = int(sys.argv[5]) if len(sys.argv) > 5 else 1
    shape = S.ModelShape(128256, 4096, layers, 32, 8, 128, 14336, 500000.0, 1e-5, f"8b-width-{layers}-layers")
    w = S.make_weights(shape, 1, torch.bfloat16, "cuda:0")
    lens = [tokens // n_prompts] * n_prompts
    tokens = sum(lens)
    tok = S.make_prompts(1, lens, shape.vocab).cuda()
    kv_format = P.KV_FP8 if os.environ.get("SWIFTKV_KV_FORMAT") == "fp8" else P.KV_MODEL_DTYPE
    model = P.SwiftKVModel(shape, w, torch.bfloat16, tokens, n_prompts, l, 1, kv_format=kv_format)
    if os.environ.get("SWIFTKV_KERNEL_MASK"):
        model.set_kernel_mask(int(os.environ["SWIFTKV_KERNEL_MASK"]))
    if os.environ.get("SWIFTKV_ACT_FORMAT"):
        model.set_activation_format(int(os.environ["SWIFTKV_ACT_FORMAT"]))
    for _ in range(steps):
        model.prefill_device_tokens(tok, lens, l, 1)
    model.status()
    torch.cuda.synchronize()
    print("profile_case ok:", model.last_launch_count(), "launches per prefill,", tokens, "tokens")


if __name__ == "__main__":
    main()
