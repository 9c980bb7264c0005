"""Shared helpers of the test-suite: oracle adapters and error measures (no method arithmetic of their own)."""
from __future__ import annotations

from typing import Sequence

import numpy as np
import torch

import synthetic_inputs as S
from oracle import swiftkv_oracle as O


def oracle_config(shape: S.ModelShape) -> O.Config:
    return O.Config(shape.vocab, shape.hidden, shape.n_layers, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                    shape.ffn, shape.rope_theta, shape.rms_eps)


def oracle_weights(w: S.Weights) -> O.Weights:
    """The oracle sees exactly the bits the CUDA path gets (bf16 / fp32 values upcast to fp64), converted lazily
    one layer at a time so that large models never sit in host memory in fp64."""
    def f64(t: torch.Tensor) -> np.ndarray:
        return t.detach().to("cpu").double().numpy()

    def embed_rows(ids):
        idx = torch.as_tensor(np.asarray(ids), dtype=torch.long, device=w.embed.device)
        return f64(w.embed[idx])

    return O.Weights(embed_rows, f64(w.final_norm), lambda: f64(w.lm_head),
                     lambda j: {k: f64(v) for k, v in w.layers[j].items()})


def rel_l2(got, ref) -> float:
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    return float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300))


def to_np(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().double().numpy()


def check_prefill_against_oracle(model, ref, n_layers: int, kv_bar: float, logit_rel_bar: float, logit_abs_bar: float):
    """Element-by-element comparison of every layer's K / V cache and of the first-token logits."""
    worst_k = worst_v = 0.0
    for j in range(n_layers):
        K, V, _ = model.kv_cache_view(j)
        ek, ev = rel_l2(to_np(K), ref["K"][j]), rel_l2(to_np(V), ref["V"][j])
        assert np.isfinite(ek) and np.isfinite(ev), f"layer {j}: non-finite cache"
        assert ek <= kv_bar, f"layer {j}: K rel-L2 {ek:.3e} > {kv_bar}"
        assert ev <= kv_bar, f"layer {j}: V rel-L2 {ev:.3e} > {kv_bar}"
        worst_k, worst_v = max(worst_k, ek), max(worst_v, ev)
    lg = to_np(model.first_logits())
    worst_rel = max(rel_l2(lg[b], ref["logits"][b]) for b in range(lg.shape[0]))
    worst_abs = float(np.max(np.abs(lg - ref["logits"])))
    assert worst_rel <= logit_rel_bar, f"logits rel-L2 {worst_rel:.3e} > {logit_rel_bar}"
    assert worst_abs <= logit_abs_bar, f"logits max-abs {worst_abs:.3e} > {logit_abs_bar}"
    return {"k": worst_k, "v": worst_v, "logit_rel": worst_rel, "logit_abs": worst_abs}
