"""Seeded synthetic inputs (weights, norm gains, prompts) for tests and the benchmark.

This module holds NO arithmetic of the SwiftKV method: it only turns (seed, tensor id, flat index)
into numbers.  Everything is integer arithmetic on int64 tensors that never overflows, followed by a
single fp32 multiply (one IEEE rounding), so the same bits come out on the CPU and on a GPU.  Both the
CPU oracle's callers and the CUDA path's callers draw their inputs from here; neither implementation
imports it itself.

Recipe
  * matrices (projections, embedding, lm_head): approx. N(0, std) with std = 0.02 -- the centred sum of
    four 16-bit uniform lanes (Irwin-Hall, n = 4) times one fp32 constant, then rounded to the model dtype.
  * RMSNorm gains: 1 + 0.25 * u, u uniform in [-1, 1) on a 2^-15 grid (distinct per layer and channel so
    that folding a gain into a projection weight is a non-trivial test).
  * token ids: a function of (seed, prompt index, position) only, uniform in [0, vocab); a truncated
    prompt is therefore a prefix of the full prompt.
  * prompt lengths: uniform integers in [lo, hi] from the same mixer.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional

import torch

_M32 = 0xFFFFFFFF
# stddev of the centred sum of four independent uniform integers in [0, 65535]
_IRWIN_HALL4_STD = (4.0 * (65536.0 ** 2 - 1.0) / 12.0) ** 0.5


def _mul32(x: torch.Tensor, c: int) -> torch.Tensor:
    """(x * c) mod 2^32 for 0 <= x < 2^32, 0 <= c < 2^32, without leaving the positive int64 range."""
    lo = x & 0xFFFF
    hi = x >> 16
    return (lo * c + (((hi * c) & 0xFFFF) << 16)) & _M32


def _mix32(x: torch.Tensor) -> torch.Tensor:
    """A 32-bit avalanche mixer (xor-shift / multiply rounds) on int64 tensors holding 32-bit values."""
    x = x ^ (x >> 16)
    x = _mul32(x, 0x7FEB352D)
    x = x ^ (x >> 15)
    x = _mul32(x, 0x846CA68B)
    x = x ^ (x >> 16)
    return x


def _mix32_int(x: int) -> int:
    x &= _M32
    x ^= x >> 16
    x = (x * 0x7FEB352D) & _M32
    x ^= x >> 15
    x = (x * 0x846CA68B) & _M32
    x ^= x >> 16
    return x


def stream_key(seed: int, *ids: int) -> int:
    """Hash (seed, ids...) into a 32-bit stream key (host integers)."""
    k = _mix32_int(0x9E3779B9 ^ (seed & _M32))
    for i in ids:
        k = _mix32_int(k ^ _mix32_int((i + 0x632BE5AB) & _M32))
    return k


def raw_u32(key: int, n: int, device="cpu", start: int = 0, salt: int = 0) -> torch.Tensor:
    """n 32-bit hashes of the counters start..start+n-1 under `key` (int64 tensor with values < 2^32)."""
    idx = torch.arange(start, start + n, dtype=torch.int64, device=device)
    k2 = _mix32_int(key ^ (0x68E31DA4 * (salt + 1) & _M32))
    return _mix32(_mix32(idx ^ key) ^ k2)


def normal_like(key: int, n: int, std: float, device="cpu", start: int = 0) -> torch.Tensor:
    """n fp32 values, approximately N(0, std)."""
    a = raw_u32(key, n, device, start, salt=0)
    b = raw_u32(key, n, device, start, salt=1)
    s = (a & 0xFFFF) + (a >> 16) + (b & 0xFFFF) + (b >> 16) - 2 * 65535
    scale = torch.tensor(std / _IRWIN_HALL4_STD, dtype=torch.float32, device=device)
    return s.to(torch.float32) * scale


def matrix(seed: int, tensor_id: int, rows: int, cols: int, dtype: torch.dtype, device="cpu",
           std: float = 0.02, chunk_rows: Optional[int] = None) -> torch.Tensor:
    """[rows, cols] row-major matrix in `dtype`; element (r, c) depends only on (seed, tensor_id, r*cols+c)."""
    key = stream_key(seed, tensor_id)
    out = torch.empty((rows, cols), dtype=dtype, device=device)
    if chunk_rows is None:
        chunk_rows = max(1, (1 << 24) // cols)
    for r0 in range(0, rows, chunk_rows):
        r1 = min(rows, r0 + chunk_rows)
        v = normal_like(key, (r1 - r0) * cols, std, device, start=r0 * cols)
        out[r0:r1] = v.view(r1 - r0, cols).to(dtype)
    return out


def matrix_rows(seed: int, tensor_id: int, row_ids: torch.Tensor, cols: int, dtype: torch.dtype,
                std: float = 0.02) -> torch.Tensor:
    """Selected rows of matrix(seed, tensor_id, *, cols): avoids materialising a large embedding table."""
    key = stream_key(seed, tensor_id)
    rows = [normal_like(key, cols, std, row_ids.device, start=int(r) * cols).to(dtype) for r in row_ids.tolist()]
    return torch.stack(rows) if rows else torch.empty((0, cols), dtype=dtype)


def gain(seed: int, tensor_id: int, n: int, dtype: torch.dtype, device="cpu") -> torch.Tensor:
    """RMSNorm gain vector 1 + 0.25*u, u in [-1, 1)."""
    key = stream_key(seed, tensor_id)
    a = raw_u32(key, n, device) & 0xFFFF
    u = (a - 32768).to(torch.float32) * (1.0 / 32768.0)
    return (1.0 + 0.25 * u).to(dtype)


def token_ids(seed: int, prompt: int, length: int, vocab: int, device="cpu") -> torch.Tensor:
    """int32 ids of prompt `prompt`: id at position p depends only on (seed, prompt, p)."""
    key = stream_key(seed, 0x70C0, prompt)
    h = raw_u32(key, length, device)
    return ((h * vocab) >> 32).to(torch.int32)


def uniform_lengths(seed: int, n: int, lo: int, hi: int) -> List[int]:
    """n prompt lengths, uniform integers in [lo, hi] (both inclusive)."""
    key = stream_key(seed, 0x1E55)
    h = raw_u32(key, n)
    return [int(lo + (int(x) * (hi - lo + 1) >> 32)) for x in h.tolist()]


def lengths_to_total(seed: int, total: int, lo: int, hi: int) -> List[int]:
    """Draw lengths uniform in [lo, hi] until the running sum would pass `total`; the last prompt is the remainder."""
    out: List[int] = []
    left = total
    i = 0
    while left > 0:
        n = uniform_lengths(seed + 7919 * i, 1, lo, hi)[0]
        n = min(n, left)
        out.append(n)
        left -= n
        i += 1
    return out


# ---------------------------------------------------------------------------------------------------
# model description + weight set
# ---------------------------------------------------------------------------------------------------
@dataclass
class ModelShape:
    vocab: int
    hidden: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    rope_theta: float
    rms_eps: float = 1e-5
    name: str = ""

    @property
    def d_q(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def d_kv(self) -> int:
        return self.n_kv_heads * self.head_dim

    def n_params(self) -> int:
        per_layer = (2 * self.hidden * self.d_q + 2 * self.hidden * self.d_kv + 3 * self.hidden * self.ffn
                     + 2 * self.hidden)
        return self.n_layers * per_layer + 2 * self.vocab * self.hidden + self.hidden


TINY = ModelShape(512, 256, 4, 8, 2, 32, 688, 10000.0, 1e-5, "tiny")
LLAMA31_8B = ModelShape(128256, 4096, 32, 32, 8, 128, 14336, 500000.0, 1e-5, "llama-3.1-8b-shape")
LLAMA31_70B = ModelShape(128256, 8192, 80, 64, 8, 128, 28672, 500000.0, 1e-5, "llama-3.1-70b-shape")

# tensor ids: layer j (0-based) uses 16*j + k; globals use the 0xF000 range
_T_IN_NORM, _T_WQ, _T_WK, _T_WV, _T_WO, _T_POST_NORM, _T_WG, _T_WU, _T_WD = range(9)
_T_EMBED, _T_FINAL_NORM, _T_LM_HEAD = 0xF000, 0xF001, 0xF002

LAYER_TENSORS = ("in_norm", "wq", "wk", "wv", "wo", "post_norm", "w_gate", "w_up", "w_down")


def layer_weights(shape: ModelShape, seed: int, j: int, dtype: torch.dtype, device="cpu") -> Dict[str, torch.Tensor]:
    """Weights of layer j (0-based).  Matrices are [out_features, in_features] row-major."""
    d, dq, dkv, f = shape.hidden, shape.d_q, shape.d_kv, shape.ffn
    t = 16 * j
    return {
        "in_norm": gain(seed, t + _T_IN_NORM, d, dtype, device),
        "wq": matrix(seed, t + _T_WQ, dq, d, dtype, device),
        "wk": matrix(seed, t + _T_WK, dkv, d, dtype, device),
        "wv": matrix(seed, t + _T_WV, dkv, d, dtype, device),
        "wo": matrix(seed, t + _T_WO, d, dq, dtype, device),
        "post_norm": gain(seed, t + _T_POST_NORM, d, dtype, device),
        "w_gate": matrix(seed, t + _T_WG, f, d, dtype, device),
        "w_up": matrix(seed, t + _T_WU, f, d, dtype, device),
        "w_down": matrix(seed, t + _T_WD, d, f, dtype, device),
    }


def global_weights(shape: ModelShape, seed: int, dtype: torch.dtype, device="cpu") -> Dict[str, torch.Tensor]:
    return {
        "embed": matrix(seed, _T_EMBED, shape.vocab, shape.hidden, dtype, device),
        "final_norm": gain(seed, _T_FINAL_NORM, shape.hidden, dtype, device),
        "lm_head": matrix(seed, _T_LM_HEAD, shape.vocab, shape.hidden, dtype, device),
    }


@dataclass
class Weights:
    """A full weight set held on one device."""
    shape: ModelShape
    dtype: torch.dtype
    embed: torch.Tensor
    final_norm: torch.Tensor
    lm_head: torch.Tensor
    layers: List[Dict[str, torch.Tensor]] = field(default_factory=list)


def make_weights(shape: ModelShape, seed: int, dtype: torch.dtype, device="cpu") -> Weights:
    g = global_weights(shape, seed, dtype, device)
    layers = [layer_weights(shape, seed, j, dtype, device) for j in range(shape.n_layers)]
    return Weights(shape, dtype, g["embed"], g["final_norm"], g["lm_head"], layers)


def make_prompts(seed: int, lengths: List[int], vocab: int, device="cpu") -> torch.Tensor:
    """Packed int32 token ids of all prompts, prompt-major."""
    if not lengths:
        return torch.empty(0, dtype=torch.int32, device=device)
    return torch.cat([token_ids(seed, b, n, vocab, device) for b, n in enumerate(lengths)])
