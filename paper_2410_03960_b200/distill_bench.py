"""Timing of the knowledge-recovery step (swiftkv_distill_grads; Sec. 3.4, Eq. 3) on a synthetic fp32 model.
Prints one JSON line (CUDA events, after a warm-up pass).

    python -m paper_2410_03960_b200.distill_bench [--layers 8] [--hidden 1024] [--prompts 4] [--length 512] [--precision 1]

Workload: a Llama-shaped fp32 model (hidden H, H/64 query heads of 64, a quarter as many KV heads, FFN 3.5 H, vocabulary
8192, random weights), `prompts` prompts of `length` tokens, l = layers / 2, g = 1, temperature 2.  The figure of merit is
executed FLOP/s: forward of the shared layers once, of the later layers twice (teacher and student), the two lm_head
products, and the backward pass of the student's later layers (data gradients of every GEMM, weight gradients of W_Q,
W_K, W_V only, attention backward as two recomputing passes)."""
import argparse
import json
import os
import sys

import torch

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import synthetic_inputs as S                      # noqa: E402
import paper_2410_03960_b200 as P                 # noqa: E402


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--layers", type=int, default=8)
    ap.add_argument("--hidden", type=int, default=1024)
    ap.add_argument("--prompts", type=int, default=4)
    ap.add_argument("--length", type=int, default=512)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--precision", type=int, default=1, help="0 fp32 CUDA cores, 1 tensor cores with split tf32 operands, 2 plain tf32")
    args = ap.parse_args()
    H, L = args.hidden, args.layers
    nq, hd = H // 64, 64
    nkv = max(1, nq // 4)
    F, V = int(3.5 * H), 8192
    shape = S.ModelShape(V, H, L, nq, nkv, hd, F, 500000.0, 1e-5, f"distill-{H}x{L}")
    w = S.make_weights(shape, 1, torch.float32, "cuda")
    lens = [args.length] * args.prompts
    T, l = sum(lens), L // 2
    tok = S.make_prompts(1, lens, V)
    model = P.SwiftKVModel(shape, w, torch.float32, T, len(lens), l, 1)
    st = {name: [None if j < l else w.layers[j][name].clone() for j in range(L)] for name in ("wq", "wk", "wv")}
    model.distill_grads(tok, lens, l, 1, 2.0, st, precision=args.precision)                      # warm-up
    a, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record()
    for _ in range(args.steps):
        loss, _ = model.distill_grads(tok, lens, l, 1, 2.0, st, precision=args.precision)
    e.record()
    torch.cuda.synchronize()
    model.status()
    ms = a.elapsed_time(e) / args.steps
    dq, dkv = nq * hd, nkv * hd
    proj = 2.0 * T * (2 * H * dq + 2 * H * dkv + 3 * H * F)           # one layer's GEMMs, forward
    attn = sum(4.0 * dq * n * (n + 1) / 2 for n in lens)               # one layer's attention, forward (causal half)
    fwd = (l + 2 * (L - l)) * (proj + attn) + 2 * 2.0 * T * H * V
    # backward of the L - l student layers: a data gradient per forward GEMM except W_K / W_V (x_{l+1} is frozen), weight
    # gradients of W_Q, W_K, W_V, attention backward = 2.5 x forward (five products of the same size) in two recomputing
    # passes (7 products executed); the lm_head's data gradient
    bwd = (L - l) * (2.0 * T * (2 * H * dq + 3 * H * F) + 2.0 * T * (H * dq + 2 * H * dkv) + 3.5 * attn) + 2.0 * T * H * V
    print(json.dumps({"what": "distill_step", "model": shape.name, "dtype": "f32", "tokens": T, "prompts": len(lens), "swift_layer": l,
                      "ms": round(ms, 2), "tokens_per_s": round(T / ms * 1e3, 1), "tflops_executed": round((fwd + bwd) / ms / 1e9, 2),
                      "loss": float(loss),
                      "gemms": ("fp32, CUDA cores", "tcgen05 kind::tf32, split operands (3 products)", "tcgen05 kind::tf32")[args.precision]}))
    model.close()


if __name__ == "__main__":
    main()
