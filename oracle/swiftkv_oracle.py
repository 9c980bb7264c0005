"""CPU oracle for SwiftKV prefill -- TEST INFRASTRUCTURE, not part of the product path.

A plain, slow, fp64 numpy restatement of (1) the unmodified Llama-style decoder prefill (Sec. 3.1) and
(2) the SwiftKV prefill (Sec. 3.2 Eq. 2, Sec. 3.3, Sec. 3.5), one step per line, no blocking, no fusion.
Only tests, the smoke check and the benchmark's CPU-baseline leg may import this module; it shares no code
with the CUDA library and never imports it.

Pins (see tests/test_oracle_pins.py): brute-force attention, RoPE/RMSNorm/softmax identities, the
identity-residual and constant-prompt special cases, l = L equals the baseline, g = 1 equals a separately
written per-layer Eq. 2 loop, the folded fused projection equals norm-then-project, Table 1's FLOP rows,
the KV-cache reduction percentages of Sec. 4, library routines (torch fp64) on the tiny configuration for both the
unmodified model and the re-wired one (every layer's cache and the logits), and, for `tail_layer`, the identity
"last row of a causal layer = tail_layer on that row's hidden state and the layer's cache".
The paper prints no worked numerical example of a forward pass, so K/V/logit VALUES are pinned by these
structural facts and library cross-checks only.

FP8 KV cache (appendix "KV quantization": per-token FP8 quantization of the cache, combined with AcrossKV):
`e4m3_decode` / `e4m3_encode` are the 8-bit format written out from its definition (1 sign, 4 exponent bits with
bias 7, 3 mantissa bits, no infinities, one NaN pattern, largest finite value 448), `quantize_per_token` gives
every token's K row and V row of a layer one fp32 scale (row maximum mapped to 448).  The code is an integer
decided by floating point, so that decision is taken in fp32 exactly as the kernel takes it: fp32 inputs,
correctly rounded fp32 divisions, round-to-nearest-even, saturation.  With `kv_fp8=True` the cache IS the
quantized representation: every attention read (prefill of layers <= l included) sees code * scale.
SimScore (Sec. 3.2, Eq. 1): `similarity`, `layer_inputs`, `simscore`; pins: hand values, torch's cosine_similarity,
the identity-residual model (every layer input equal, SimScore = 1), invariance to per-token rescaling.

Pins: the format's defining values and torch's float8_e4m3fn (decode table, encode of random values and of
every midpoint), a pure-Python nearest-value search, the half-step error bound, scale equivariance, and the
paper's combined cache reductions (62.5 % and 68.75 %).

Conventions.  Row vectors: a projection is  h @ W.T  with W stored [out_features, in_features] (the paper
writes W x, Eq. 2).  `l` (swift_layer) is a COUNT: layers 1..l (0-based 0..l-1) run on every prompt token;
s = output of layer l = the paper's x_{l+1}.  `g` = AcrossKV group size; groups are consecutive, aligned at
layer l+1, the first layer of a group projects K/V for the whole group; a short last group is allowed.
RoPE is the rotate-half form (pairs (i, i + hd/2)), positions restart at 0 for each prompt, K is cached
after RoPE, V as projected.  RMSNorm eps as configured; softmax scale 1/sqrt(head_dim); no biases; untied
embedding / lm_head.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Callable, Dict, List, Sequence

import numpy as np

F64 = np.float64


@dataclass
class Config:
    vocab: int
    hidden: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    rope_theta: float
    rms_eps: float = 1e-5

    @property
    def d_q(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def d_kv(self) -> int:
        return self.n_kv_heads * self.head_dim


class Weights:
    """Weight container.  `layer(j)` (0-based) returns a dict with in_norm, wq, wk, wv, wo, post_norm,
    w_gate, w_up, w_down as fp64 arrays; it may build them lazily so that very large models never have to
    be resident all at once.  `embed_rows(ids)` returns the embedding rows of the given token ids."""

    def __init__(self, embed_rows: Callable[[np.ndarray], np.ndarray], final_norm: np.ndarray,
                 lm_head: Callable[[], np.ndarray], layer: Callable[[int], Dict[str, np.ndarray]]):
        self.embed_rows = embed_rows
        self.final_norm = np.asarray(final_norm, dtype=F64)
        self._lm_head = lm_head
        self.layer = layer

    def lm_head(self) -> np.ndarray:
        return np.asarray(self._lm_head(), dtype=F64)

    @staticmethod
    def from_arrays(embed, final_norm, lm_head, layers: Sequence[Dict[str, np.ndarray]]) -> "Weights":
        embed = np.asarray(embed, dtype=F64)
        lm = np.asarray(lm_head, dtype=F64)
        layers = [{k: np.asarray(v, dtype=F64) for k, v in w.items()} for w in layers]
        return Weights(lambda ids: embed[np.asarray(ids, dtype=np.int64)], final_norm, lambda: lm,
                       lambda j: layers[j])


# ---------------------------------------------------------------------------------------------------
# operators (Sec. 3.1)
# ---------------------------------------------------------------------------------------------------
def rmsnorm(x: np.ndarray, gamma: np.ndarray, eps: float) -> np.ndarray:
    """y = x / sqrt(mean(x^2) + eps) * gamma, over the last axis."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * gamma


def unit_rms(x: np.ndarray, eps: float) -> np.ndarray:
    """x / sqrt(mean(x^2) + eps): the statistic shared by every later layer's input norm of s."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps)


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotary embedding, rotate-half pairing.  x: [n, heads, hd]; pos: [n] integer positions."""
    n, _, hd = x.shape
    half = hd // 2
    i = np.arange(half, dtype=F64)
    inv_freq = theta ** (-2.0 * i / hd)                       # [half]
    ang = np.asarray(pos, dtype=F64)[:, None] * inv_freq[None, :]   # [n, half]
    c = np.cos(ang)[:, None, :]
    s = np.sin(ang)[:, None, :]
    a = x[..., :half]
    b = x[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def softmax_rows(z: np.ndarray) -> np.ndarray:
    z = z - np.max(z, axis=-1, keepdims=True)
    e = np.exp(z)
    return e / np.sum(e, axis=-1, keepdims=True)


def silu(z: np.ndarray) -> np.ndarray:
    return z / (1.0 + np.exp(-z))


def causal_attention(q: np.ndarray, K: np.ndarray, V: np.ndarray) -> np.ndarray:
    """Causal grouped-query attention of one prompt against its own keys.
    q: [n, n_q, hd]; K, V: [n, n_kv, hd]; query head h reads KV head h // (n_q / n_kv).  Returns [n, n_q*hd]."""
    n, n_q, hd = q.shape
    n_kv = K.shape[1]
    rep = n_q // n_kv
    out = np.empty((n, n_q, hd), dtype=F64)
    allowed = np.tril(np.ones((n, n), dtype=bool))            # key t <= query p
    for h in range(n_q):
        kv = h // rep
        scores = q[:, h, :] @ K[:, kv, :].T / math.sqrt(hd)   # [n, n]
        scores = np.where(allowed, scores, -np.inf)
        out[:, h, :] = softmax_rows(scores) @ V[:, kv, :]
    return out.reshape(n, n_q * hd)


def single_query_attention(q: np.ndarray, K: np.ndarray, V: np.ndarray) -> np.ndarray:
    """One query token (the last of its prompt) against every cached key of that prompt, itself included.
    q: [n_q, hd]; K, V: [m, n_kv, hd].  Returns [n_q*hd]."""
    n_q, hd = q.shape
    rep = n_q // K.shape[1]
    out = np.empty((n_q, hd), dtype=F64)
    for h in range(n_q):
        kv = h // rep
        scores = K[:, kv, :] @ q[h] / math.sqrt(hd)           # [m]
        out[h] = softmax_rows(scores[None, :])[0] @ V[:, kv, :]
    return out.reshape(n_q * hd)


def mlp(m: np.ndarray, w: Dict[str, np.ndarray]) -> np.ndarray:
    return (silu(m @ w["w_gate"].T) * (m @ w["w_up"].T)) @ w["w_down"].T


# ---------------------------------------------------------------------------------------------------
# FP8 (e4m3, "fn" flavour: finite only) per-token quantization of cache rows (appendix, KV quantization)
# ---------------------------------------------------------------------------------------------------
E4M3_MAX = 448.0
AMAX_FLOOR = 2.0 ** -64          # rows that are all (nearly) zero: keeps the scale a normal fp32 number


def e4m3_decode(codes: np.ndarray) -> np.ndarray:
    """Value of each 8-bit code: sign s, exponent field e (4 bits, bias 7), mantissa field m (3 bits).
    e = 0: subnormal m/8 * 2^-6;  otherwise (1 + m/8) * 2^(e-7);  e = 15, m = 7 is NaN (there are no infinities)."""
    c = np.asarray(codes, dtype=np.uint8).astype(np.int64)
    s, e, m = c >> 7, (c >> 3) & 15, c & 7
    val = np.where(e == 0, (m / 8.0) * 2.0 ** -6, (1.0 + m / 8.0) * np.exp2((e - 7).astype(F64)))
    val = np.where((e == 15) & (m == 7), np.nan, val)
    return np.where(s == 1, -val, val)


def e4m3_encode(y: np.ndarray) -> np.ndarray:
    """Nearest e4m3 code of each fp32 value, ties to the even mantissa, magnitudes beyond 448 saturate to 448.
    Works on the exact value of the fp32 input (scaling by powers of two in fp64 is exact)."""
    y = np.asarray(y, dtype=np.float32).astype(F64)
    a = np.abs(y)
    sign = (np.signbit(y)).astype(np.int64) << 7
    # subnormal range [0, 2^-6): multiples of 2^-9; the count of steps IS the code (8 steps = first normal code)
    sub = np.rint(a * 2.0 ** 9).astype(np.int64)
    # normal range: a = (1 + f) * 2^e with f in [0, 1); mantissa steps of 1/8; a carry walks into the exponent field
    mant, ex = np.frexp(np.where(a > 0, a, 1.0))          # a = mant * 2^ex, mant in [0.5, 1)
    e = ex - 1
    q = np.rint((mant * 2.0 - 1.0) * 8.0).astype(np.int64)
    norm = ((e + 7) << 3) + q
    code = np.where(a < 2.0 ** -6, sub, norm)
    code = np.where(a > E4M3_MAX, 0x7E, np.minimum(code, 0x7E))
    code = np.where(np.isnan(y), 0x7F, code)
    return (code | sign).astype(np.uint8)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """fp32 values rounded to the nearest bfloat16 (8 significand bits; ties to even), returned as fp32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(np.shape(x))


def quantize_per_token(x: np.ndarray, row_dtype: str = "f32"):
    """x [n_rows, ...]: one scale per row (token).  scale = max(amax, 2^-64) / 448, code = e4m3(x / scale), every
    operation on fp32 values with one correctly rounded fp32 result (what `/` on numpy float32 arrays does).
    row_dtype: the type in which the rows exist before they are quantized -- "bf16" for a bf16 model (its K / V rows
    are bf16 values, so that is the precision the code decision is taken in), "f32" otherwise.
    Returns (codes uint8 like x, scale float32 [n_rows], dequantized float64 like x = value(code) * scale)."""
    x32 = np.asarray(x, dtype=np.float32)
    if row_dtype == "bf16":
        x32 = round_to_bf16(x32)
    else:
        assert row_dtype == "f32"
    flat = x32.reshape(x32.shape[0], -1)
    amax = np.maximum(np.max(np.abs(flat), axis=1), np.float32(AMAX_FLOOR)).astype(np.float32)
    scale = (amax / np.float32(E4M3_MAX)).astype(np.float32)
    y = (flat / scale[:, None]).astype(np.float32)
    codes = e4m3_encode(y)
    deq = e4m3_decode(codes) * scale.astype(F64)[:, None]
    return codes.reshape(x32.shape), scale, deq.reshape(x32.shape)


def decoder_layer(cfg: Config, w: Dict[str, np.ndarray], X: np.ndarray, pos: np.ndarray, kv_fp8: bool = False,
                  row_dtype: str = "f32"):
    """One unmodified decoder layer on all rows of one prompt.  Returns (X_out, K, V) with K after RoPE.
    kv_fp8: K (after RoPE) and V go through the cache's per-token FP8 representation before anyone attends to them."""
    n = X.shape[0]
    h = rmsnorm(X, w["in_norm"], cfg.rms_eps)
    q = (h @ w["wq"].T).reshape(n, cfg.n_q_heads, cfg.head_dim)
    k = (h @ w["wk"].T).reshape(n, cfg.n_kv_heads, cfg.head_dim)
    v = (h @ w["wv"].T).reshape(n, cfg.n_kv_heads, cfg.head_dim)
    q = rope(q, pos, cfg.rope_theta)
    k = rope(k, pos, cfg.rope_theta)
    if kv_fp8:
        k, v = quantize_per_token(k, row_dtype)[2], quantize_per_token(v, row_dtype)[2]
    a = causal_attention(q, k, v)
    X = X + a @ w["wo"].T
    m = rmsnorm(X, w["post_norm"], cfg.rms_eps)
    X = X + mlp(m, w)
    return X, k, v


def tail_layer(cfg: Config, w: Dict[str, np.ndarray], y: np.ndarray, p: int, K: np.ndarray, V: np.ndarray):
    """A later layer (> l) applied to the one continuing token of a prompt (position p).  No K/V projection
    happens here: the layer attends to the cache K, V[0..p] that the SwiftKV projection filled."""
    h = rmsnorm(y, w["in_norm"], cfg.rms_eps)
    q = (h @ w["wq"].T).reshape(1, cfg.n_q_heads, cfg.head_dim)
    q = rope(q, np.array([p]), cfg.rope_theta)[0]
    a = single_query_attention(q, K[: p + 1], V[: p + 1])
    y = y + a @ w["wo"].T
    m = rmsnorm(y, w["post_norm"], cfg.rms_eps)
    return y + mlp(m, w)


def _offsets(seq_lens: Sequence[int]) -> List[int]:
    off = [0]
    for n in seq_lens:
        off.append(off[-1] + int(n))
    return off


# ---------------------------------------------------------------------------------------------------
# the two models
# ---------------------------------------------------------------------------------------------------
def baseline(cfg: Config, W: Weights, tokens: np.ndarray, seq_lens: Sequence[int]):
    """Unmodified prefill (Sec. 3.1): every prompt token through all L layers.
    Returns {"K": [L] x [T, n_kv, hd], "V": same, "logits": [B, vocab]} in packed prompt-major token order."""
    return swiftkv(cfg, W, tokens, seq_lens, cfg.n_layers, 1)


def group_leader(l: int, g: int, j: int) -> int:
    """1-based layer j > l -> the 1-based layer whose K/V projection its AcrossKV group shares (Sec. 3.3)."""
    return l + 1 + g * ((j - l - 1) // g)


def swiftkv(cfg: Config, W: Weights, tokens: np.ndarray, seq_lens: Sequence[int], l: int, g: int = 1,
            kv_fp8: bool = False, row_dtype: str = "f32"):
    """SwiftKV prefill.  Layers 1..l as in the unmodified model; s = x_{l+1}; for every later layer j the
    cache is  K_j = rope(rmsnorm(s, gamma_in[r]) @ W_K[r].T),  V_j = rmsnorm(s, gamma_in[r]) @ W_V[r].T
    with r the leader of j's AcrossKV group (Eq. 2, Sec. 3.3); only the last token of each prompt runs
    layers l+1..L (footnote in Sec. 3.2; Sec. 3.5), attending to those caches.
    kv_fp8: every cache row is stored as per-token FP8 codes + scale; "K", "V" are then the dequantized values and
    "K_codes", "K_scale", "V_codes", "V_scale" the stored representation; row_dtype as in quantize_per_token."""
    L = cfg.n_layers
    assert 1 <= l <= L and g >= 1
    tokens = np.asarray(tokens, dtype=np.int64)
    off = _offsets(seq_lens)
    T, B = off[-1], len(seq_lens)
    assert tokens.shape[0] == T
    pos = np.concatenate([np.arange(n) for n in seq_lens]) if B else np.zeros(0, dtype=np.int64)

    X = np.asarray(W.embed_rows(tokens), dtype=F64)            # x_1
    K = [None] * L
    V = [None] * L
    for j in range(l):                                         # layers 1..l, all tokens
        w = W.layer(j)
        Kj = np.empty((T, cfg.n_kv_heads, cfg.head_dim), dtype=F64)
        Vj = np.empty_like(Kj)
        Xn = np.empty_like(X)
        for b in range(B):
            a, e = off[b], off[b + 1]
            Xn[a:e], Kj[a:e], Vj[a:e] = decoder_layer(cfg, w, X[a:e], pos[a:e], kv_fp8, row_dtype)
        X, K[j], V[j] = Xn, Kj, Vj
    s = X                                                      # x_{l+1}

    for j1 in range(l + 1, L + 1):                             # 1-based later layers
        r1 = group_leader(l, g, j1)
        if j1 == r1:
            w = W.layer(r1 - 1)
            h = rmsnorm(s, w["in_norm"], cfg.rms_eps)
            k = (h @ w["wk"].T).reshape(T, cfg.n_kv_heads, cfg.head_dim)
            K[j1 - 1] = rope(k, pos, cfg.rope_theta)
            V[j1 - 1] = (h @ w["wv"].T).reshape(T, cfg.n_kv_heads, cfg.head_dim)
            if kv_fp8:
                K[j1 - 1], V[j1 - 1] = quantize_per_token(K[j1 - 1], row_dtype)[2], quantize_per_token(V[j1 - 1], row_dtype)[2]
        else:
            K[j1 - 1] = K[r1 - 1]                              # alias: one cache per group
            V[j1 - 1] = V[r1 - 1]

    last = [off[b + 1] - 1 for b in range(B)]
    Y = s[last].copy()                                         # the continuing tokens
    for j in range(l, L):
        w = W.layer(j)
        for b in range(B):
            a, e = off[b], off[b + 1]
            Y[b] = tail_layer(cfg, w, Y[b], e - a - 1, K[j][a:e], V[j][a:e])
    logits = rmsnorm(Y, W.final_norm, cfg.rms_eps) @ W.lm_head().T
    out = {"K": K, "V": V, "logits": logits}
    if kv_fp8:
        # the stored representation: quantizing a dequantized row again returns its codes (every value is
        # code * scale with the row maximum at code 448, so the scale comes back up to one fp32 rounding)
        for name, planes in (("K", K), ("V", V)):
            qs = [quantize_per_token(pl) for pl in planes]
            out[name + "_codes"] = [q[0] for q in qs]
            out[name + "_scale"] = [q[1] for q in qs]
    return out


def swiftkv_eq2_ungrouped(cfg: Config, W: Weights, s: np.ndarray, pos: np.ndarray, l: int):
    """Eq. 2 written out with no grouping code at all: KV_j = W_KV^j applied to the normed s, for all j > l.
    Used to pin swiftkv(l, g=1).  Returns ({j: K_j}, {j: V_j}) with 0-based j."""
    Ks, Vs = {}, {}
    T = s.shape[0]
    for j in range(l, cfg.n_layers):
        w = W.layer(j)
        h = rmsnorm(s, w["in_norm"], cfg.rms_eps)
        Ks[j] = rope((h @ w["wk"].T).reshape(T, cfg.n_kv_heads, cfg.head_dim), pos, cfg.rope_theta)
        Vs[j] = (h @ w["wv"].T).reshape(T, cfg.n_kv_heads, cfg.head_dim)
    return Ks, Vs


def hidden_after(cfg: Config, W: Weights, tokens: np.ndarray, seq_lens: Sequence[int], n: int) -> np.ndarray:
    """Residual stream after n unmodified layers (x_{n+1}), all tokens."""
    tokens = np.asarray(tokens, dtype=np.int64)
    off = _offsets(seq_lens)
    pos = np.concatenate([np.arange(m) for m in seq_lens])
    X = np.asarray(W.embed_rows(tokens), dtype=F64)
    for j in range(n):
        w = W.layer(j)
        Xn = np.empty_like(X)
        for b in range(len(seq_lens)):
            a, e = off[b], off[b + 1]
            Xn[a:e], _, _ = decoder_layer(cfg, w, X[a:e], pos[a:e])
        X = Xn
    return X


# ---------------------------------------------------------------------------------------------------
# SimScore (Sec. 3.2, Eq. 1): how similar a layer's input is to the inputs of all later layers
# ---------------------------------------------------------------------------------------------------
def similarity(Xa: np.ndarray, Xb: np.ndarray) -> float:
    """Average over tokens i of the cosine similarity between Xa[i] and Xb[i]  (Xa, Xb: [n_tokens, hidden])."""
    dots = np.sum(Xa * Xb, axis=-1)
    return float(np.mean(dots / (np.linalg.norm(Xa, axis=-1) * np.linalg.norm(Xb, axis=-1))))


def layer_inputs(cfg: Config, W: Weights, tokens: np.ndarray, seq_lens: Sequence[int]) -> List[np.ndarray]:
    """x_1 .. x_L of the unmodified model: element l-1 is the input of (1-based) layer l, all tokens."""
    return [hidden_after(cfg, W, tokens, seq_lens, n) for n in range(cfg.n_layers)]


def simscore(xs: Sequence[np.ndarray]) -> np.ndarray:
    """Eq. 1 for every layer that has a later one.  xs[l-1] = x_l (input of layer l), l = 1..L.
    Returns s with s[l-1] = SimScore(x_l) = sum_{j=l+1..L} Similarity(x_l, x_j) / (L - l), l = 1..L-1."""
    L = len(xs)
    out = np.empty(L - 1, dtype=F64)
    for l in range(1, L):
        out[l - 1] = sum(similarity(xs[l - 1], xs[j - 1]) for j in range(l + 1, L + 1)) / (L - l)
    return out


# ---------------------------------------------------------------------------------------------------
# the fused, gain-folded SingleInputKV projection (Sec. 3.5; one GEMM for all later layers)
# ---------------------------------------------------------------------------------------------------
def folded_kv_weight(cfg: Config, W: Weights, l: int, g: int) -> np.ndarray:
    """Concatenate, over AcrossKV group leaders r, [diag(gamma_in[r]) folded into W_K[r] ; same for W_V[r]].
    Returns [n_groups * 2 * d_kv, hidden]; rows of leader number i occupy [i*2*d_kv, (i+1)*2*d_kv), K first."""
    blocks = []
    for r1 in range(l + 1, cfg.n_layers + 1, g):
        w = W.layer(r1 - 1)
        blocks.append(w["wk"] * w["in_norm"][None, :])
        blocks.append(w["wv"] * w["in_norm"][None, :])
    return np.concatenate(blocks, axis=0)


def fused_single_input_kv(cfg: Config, Wt: np.ndarray, s: np.ndarray, pos: np.ndarray):
    """One projection of the unit-rms s through the folded weight; K blocks get RoPE.
    Returns lists (K_i, V_i) per group leader i."""
    T = s.shape[0]
    out = unit_rms(s, cfg.rms_eps) @ Wt.T
    n_groups = Wt.shape[0] // (2 * cfg.d_kv)
    Ks, Vs = [], []
    for i in range(n_groups):
        blk = out[:, i * 2 * cfg.d_kv:(i + 1) * 2 * cfg.d_kv]
        Ks.append(rope(blk[:, :cfg.d_kv].reshape(T, cfg.n_kv_heads, cfg.head_dim), pos, cfg.rope_theta))
        Vs.append(blk[:, cfg.d_kv:].reshape(T, cfg.n_kv_heads, cfg.head_dim))
    return Ks, Vs


# ---------------------------------------------------------------------------------------------------
# closed forms the paper prints: Table 1 (GFLOPs per prefill token) and the KV-cache reduction of Sec. 4
# ---------------------------------------------------------------------------------------------------
def table1_gflops_per_token(cfg: Config, l: int, g: int, context: float) -> Dict[str, float]:
    """Per-prefill-token GFLOPs in the paper's Table 1 convention: 2 FLOPs per multiply-add; "Vocab" counts
    the embedding and the lm_head both as matmuls; K,V is projected for every layer <= l and once per
    AcrossKV group after it; Q,O / MLP / attention only for the l layers that prompt tokens run;
    attention = QK^T and PV against an average of context/2 keys (causal)."""
    L, d = cfg.n_layers, cfg.hidden
    n_groups = -(-(L - l) // g)
    vocab = 2 * (2 * d * cfg.vocab)
    kv = (l + n_groups) * 2 * d * (2 * cfg.d_kv)
    qo = l * (2 * d * cfg.d_q + 2 * cfg.d_q * d)
    mlp_f = l * 3 * 2 * d * cfg.ffn
    attn = l * 4 * cfg.d_q * (context / 2.0)
    tot = vocab + kv + qo + mlp_f + attn
    return {k: v / 1e9 for k, v in dict(vocab=vocab, kv=kv, qo=qo, mlp=mlp_f, attn=attn, total=tot).items()}


def kv_cache_reduction(n_layers: int, l: int, g: int, bytes_ratio: float = 1.0) -> float:
    """Fraction of KV-cache memory saved: layers > l keep one cache per AcrossKV group; bytes_ratio = bytes of a
    stored element over bytes of a 16-bit one (0.5 for the FP8 cache; the paper's figures ignore the scales)."""
    n_groups = -(-(n_layers - l) // g)
    return 1.0 - bytes_ratio * (l + n_groups) / n_layers
