"""FLOPs that a prefill actually executes (2 per multiply-add), used to turn times into TFLOP/s.

Counted: every GEMM as 2*M*N*K; causal attention as 4*d_q*n*(n+1)/2 per layer and prompt (QK^T and PV over the
unmasked half only); for layers > l only the fused K/V projection of all tokens plus the last token's own
work (Q/O/MLP and 4*d_q*n attention); the lm_head for the last tokens only; the embedding gather as 0.
"""
from __future__ import annotations

from typing import Dict, Sequence


def prefill_flops(hidden: int, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int, ffn: int, vocab: int,
                  seq_lens: Sequence[int], swift_layer: int, acrosskv_group: int = 1) -> Dict[str, float]:
    d, L, l, g = hidden, n_layers, swift_layer, acrosskv_group
    dq, dkv = n_q_heads * head_dim, n_kv_heads * head_dim
    T, B = sum(seq_lens), len(seq_lens)
    n_groups = -(-(L - l) // g)
    f_qo = 2 * d * dq + 2 * dq * d
    f_kv = 2 * d * 2 * dkv
    f_mlp = 6 * d * ffn
    gemm = T * l * (f_qo + f_kv + f_mlp) + T * n_groups * f_kv
    attn = sum(l * 4 * dq * n * (n + 1) / 2 for n in seq_lens)
    tail = B * (L - l) * (f_qo + f_mlp) + sum((L - l) * 4 * dq * n for n in seq_lens) + B * 2 * d * vocab
    return {"gemm": float(gemm), "attention": float(attn), "tail": float(tail), "total": float(gemm + attn + tail)}
