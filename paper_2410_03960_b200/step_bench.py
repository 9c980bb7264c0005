"""Timing of the serving-style entry point (swiftkv_step) on the benchmark model: chunked prefill, decode steps,
paged cache rows and the FP8 cache.  Prints one JSON line per measurement (CUDA events, after a warm-up pass).

    python -m paper_2410_03960_b200.step_bench [--kv-format fp8] [--chunks 8192,2048,512] [--decode-steps 12] [--kernel-mask M]

Workload: the benchmark's batch (Llama-3.1-8B shape, random bf16 weights, 8 prompts with lengths U[2048, 8192],
seed 1, l = 16, g = 1).  A chunked prefill feeds every prompt `chunk` tokens per step (all prompts that still have
tokens left share a minibatch) until the caches of all prompts are complete; a decode step appends one token to each
of the 8 sequences.  Each sequence owns 65 pages of 128 cache rows, contiguous or (paged) interleaved."""
import argparse
import json
import os
import sys

import torch

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import synthetic_inputs as S                      # noqa: E402
import paper_2410_03960_b200 as P                 # noqa: E402

SEED, N_PROMPTS, LEN_LO, LEN_HI, SWIFT_LAYER, GROUP = 1, 8, 2048, 8192, 16, 1
PAGES_PER_SEQ = 65
DECODE_WARMUP = 8


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--kv-format", choices=("model", "fp8"), default="model")
    ap.add_argument("--chunks", default="8192,2048,512")
    ap.add_argument("--decode-steps", type=int, default=12)
    ap.add_argument("--profile", action="store_true", help="also print the kernel classes' CUDA-event times of each chunked run")
    ap.add_argument("--no-half-weight-cache", action="store_true",
                    help="copy the layers' matrices to half in every step instead of once (swiftkv_set_half_weight_cache)")
    ap.add_argument("--kernel-mask", type=int, default=None, help="swiftkv_set_kernel_mask value (default: the library's)")
    args = ap.parse_args()
    shape = S.LLAMA31_8B
    lens = S.uniform_lengths(SEED, N_PROMPTS, LEN_LO, LEN_HI)
    total, n_seq = sum(lens), len(lens)
    extra = args.decode_steps + DECODE_WARMUP
    toks = [S.token_ids(SEED, b, n + extra, shape.vocab) for b, n in enumerate(lens)]
    w = S.make_weights(shape, SEED, torch.bfloat16, "cuda")
    fmt = P.KV_FP8 if args.kv_format == "fp8" else P.KV_MODEL_DTYPE
    cap = PAGES_PER_SEQ * 128
    model = P.SwiftKVModel(shape, w, torch.bfloat16, cap * n_seq, n_seq, SWIFT_LAYER, GROUP, kv_format=fmt)
    if args.kernel_mask is not None:
        model.set_kernel_mask(args.kernel_mask)
    if not args.no_half_weight_cache:
        model.set_half_weight_cache(SWIFT_LAYER)
    # paged: sequence b owns pages b, b + 8, b + 16, ... (interleaved with the other sequences' pages)
    pages = [[b + n_seq * i for i in range(PAGES_PER_SEQ)] for b in range(n_seq)]

    def where(b, paged):
        return pages[b] if paged else b * cap

    def timed(fn):
        a, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        n = fn()
        e.record()
        torch.cuda.synchronize()
        model.status()
        return a.elapsed_time(e), n

    def chunked(chunk, paged):
        done, steps = [0] * n_seq, 0
        while any(d < n for d, n in zip(done, lens)):
            seqs, packed = [], []
            for b, n in enumerate(lens):
                if done[b] >= n:
                    continue
                k = min(chunk, n - done[b])
                seqs.append((k, done[b], where(b, paged), int(done[b] + k == n)))
                packed.append(toks[b][done[b]:done[b] + k])
                done[b] += k
            model.step(torch.cat(packed), seqs, SWIFT_LAYER, GROUP)
            steps += 1
        return steps

    base = {"model": "llama-3.1-8b shape bf16", "l": SWIFT_LAYER, "g": GROUP, "prompts": n_seq, "tokens": total,
            "kv_format": args.kv_format, "data": "synthetic",
            "half_weight_cache": not args.no_half_weight_cache}
    for chunk in [int(c) for c in args.chunks.split(",")]:
        for paged in (False, True):
            chunked(chunk, paged)
            ms, steps = timed(lambda: chunked(chunk, paged))
            print(json.dumps(dict(base, what="chunked_prefill", chunk=chunk, paged=paged, steps=steps, ms=round(ms, 2),
                                  tokens_per_s=round(total / ms * 1e3, 1))), flush=True)
            if args.profile:
                model.profile_enable(True)
                model.profile_read()
                chunked(chunk, paged)
                prof = model.profile_read()
                model.profile_enable(False)
                print(json.dumps(dict(what="kernel_classes_ms", chunk=chunk, paged=paged,
                                      **{k: [round(v[0], 2), v[1]] for k, v in prof.items()})), flush=True)
    for paged in (False, True):
        chunked(8192, paged)

        def decode(t0, t1):
            for t in range(t0, t1):
                model.step(torch.stack([toks[b][n + t] for b, n in enumerate(lens)]),
                           [(1, n + t, where(b, paged), 1) for b, n in enumerate(lens)], SWIFT_LAYER, GROUP)
            return t1 - t0

        decode(0, DECODE_WARMUP)       # (the first steps after a prefill run ~30 % slower: clocks and caches settle)
        ms, n = timed(lambda: decode(DECODE_WARMUP, DECODE_WARMUP + args.decode_steps))
        print(json.dumps(dict(base, what="decode_step", paged=paged, batch=n_seq, context=total // n_seq,
                              ms_per_step=round(ms / n, 3), tokens_per_s=round(n_seq * n / ms * 1e3, 1))), flush=True)


if __name__ == "__main__":
    main()
