"""CPU oracle for SwiftKV's knowledge-recovery step (Sec. 3.4, Eq. 3) -- TEST INFRASTRUCTURE, not part of the product path.

fp64 numpy, one step per line.  The teacher is the unmodified model (every token through every layer, Sec. 3.1); the
student is the same frozen model re-wired by SingleInputKV / AcrossKV (Sec. 3.2 Eq. 2, Sec. 3.3) with its OWN copies of
W_Q, W_K, W_V of the layers > l, which are the only trainable parameters ("Efficient Distillation": one frozen copy of
the model, an extra trainable copy of W_QKV of the later layers).  In training every prompt token runs every layer (each
position yields logits): layer j > l takes its queries from its own normalised input through the student's W_Q and
attends to K, V projected from x_{l+1} with the student's W_K, W_V of the group leader.  Eq. 3 names the two logit tensors;
the loss on them is the standard distillation loss at temperature tau (2.0 in the paper's training details):

    loss = tau^2 * mean over prompt tokens of KL( softmax(y_teacher / tau) || softmax(y_student / tau) ).

Readings where the paper is silent: the loss is the soft-target term alone (no hard-label term: the paper distils "using
the output logits of the original model"), with the usual tau^2 factor, averaged over all prompt tokens of the batch;
RMSNorm gains stay frozen (they are not part of W_QKV); with AcrossKV only a group leader's W_K, W_V are used, so the
other layers' W_K, W_V receive zero gradient.

The update rule: the paper's training details give a learning rate (3e-4), a weight decay (0.05) and a warm-up ratio but do
not name the optimiser; `adamw_update` is AdamW with decoupled weight decay (the usual choice for exactly that set of
hyper-parameters), pinned against torch.optim.AdamW.

`distill_grads` is the analytic backward pass written out operator by operator.  Pins (tests/test_distill_oracle_pins.py):
central finite differences of `distill_loss`, torch autograd (fp64) through a torch-assembled student, loss = 0 and zero
gradients when the student is not re-wired (l = L), KL >= 0, zero gradient for non-leader W_K / W_V.

Only tests and the smoke / benchmark CPU legs may import this module.  It imports the prefill oracle's operators
(`rmsnorm`, `rope`, `softmax_rows`, `silu`, `group_leader`) and nothing from the CUDA library.
"""
from __future__ import annotations

import math
from typing import Dict, List, Sequence

import numpy as np

from .swiftkv_oracle import F64, Config, Weights, _offsets, group_leader, rmsnorm, rope, silu, softmax_rows


def student_copies(cfg: Config, W: Weights, l: int) -> Dict[str, List[np.ndarray]]:
    """The trainable copies, initialised from the original model (Sec. 3.4): lists indexed by 0-based layer, None for layers <= l."""
    out = {"wq": [None] * cfg.n_layers, "wk": [None] * cfg.n_layers, "wv": [None] * cfg.n_layers}
    for j in range(l, cfg.n_layers):
        for name in out:
            out[name][j] = np.array(W.layer(j)[name], dtype=F64, copy=True)
    return out


def _attention_forward(q: np.ndarray, K: np.ndarray, V: np.ndarray):
    """Causal grouped-query attention of one prompt; returns the output [n, n_q, hd] and the probabilities [n_q, n, n]."""
    n, n_q, hd = q.shape
    rep = n_q // K.shape[1]
    allowed = np.tril(np.ones((n, n), dtype=bool))
    out = np.empty((n, n_q, hd), dtype=F64)
    P = np.empty((n_q, n, n), dtype=F64)
    for h in range(n_q):
        scores = q[:, h, :] @ K[:, h // rep, :].T / math.sqrt(hd)
        P[h] = softmax_rows(np.where(allowed, scores, -np.inf))
        out[:, h, :] = P[h] @ V[:, h // rep, :]
    return out, P


def _attention_backward(q, K, V, P, dO):
    """Gradients of `_attention_forward` with respect to q, K, V (dO: [n, n_q, hd])."""
    n, n_q, hd = q.shape
    rep = n_q // K.shape[1]
    dq = np.zeros_like(q)
    dK = np.zeros_like(K)
    dV = np.zeros_like(V)
    for h in range(n_q):
        kv = h // rep
        dV[:, kv, :] += P[h].T @ dO[:, h, :]
        dP = dO[:, h, :] @ V[:, kv, :].T
        dS = P[h] * (dP - np.sum(dP * P[h], axis=-1, keepdims=True))       # softmax backward, row by row
        dq[:, h, :] = dS @ K[:, kv, :] / math.sqrt(hd)
        dK[:, kv, :] += dS.T @ q[:, h, :] / math.sqrt(hd)
    return dq, dK, dV


def _rmsnorm_backward(x: np.ndarray, gamma: np.ndarray, eps: float, dy: np.ndarray) -> np.ndarray:
    """d/dx of  y = x * r * gamma,  r = (mean(x^2) + eps)^(-1/2)  (gamma frozen)."""
    r = 1.0 / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps)
    gdy = gamma * dy
    return r * gdy - x * (r ** 3) * np.mean(x * gdy, axis=-1, keepdims=True)


def _rope_backward(dx: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """The rotation is orthogonal: its transpose is the rotation by the negated angle."""
    return rope(dx, -np.asarray(pos), theta)


def teacher_logits(cfg: Config, W: Weights, tokens: np.ndarray, seq_lens: Sequence[int]) -> np.ndarray:
    """y_teacher of Eq. 3: the unmodified model's logits at EVERY prompt position, [T, vocab]."""
    S = student_copies(cfg, W, cfg.n_layers)
    return student_forward(cfg, W, S, tokens, seq_lens, cfg.n_layers, 1)["logits"]


def student_forward(cfg: Config, W: Weights, S: Dict[str, List[np.ndarray]], tokens: np.ndarray, seq_lens: Sequence[int],
                    l: int, g: int = 1) -> Dict[str, object]:
    """y_student of Eq. 3 at every prompt position, with what the backward pass needs."""
    L = cfg.n_layers
    tokens = np.asarray(tokens, dtype=np.int64)
    off = _offsets(seq_lens)
    T, B = off[-1], len(seq_lens)
    pos = np.concatenate([np.arange(n) for n in seq_lens])
    nq, nkv, hd = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim

    X = np.asarray(W.embed_rows(tokens), dtype=F64)
    saved = [None] * L
    s = None
    for j in range(L):
        w = W.layer(j)
        if j == l:
            s = X                                               # x_{l+1}
        rewired = j >= l
        h = rmsnorm(X, w["in_norm"], cfg.rms_eps)
        wq = S["wq"][j] if rewired else w["wq"]
        q = rope((h @ wq.T).reshape(T, nq, hd), pos, cfg.rope_theta)
        if rewired:
            r = group_leader(l, g, j + 1) - 1                   # 0-based leader of j's AcrossKV group
            hs = rmsnorm(s, W.layer(r)["in_norm"], cfg.rms_eps)
            k = rope((hs @ S["wk"][r].T).reshape(T, nkv, hd), pos, cfg.rope_theta)
            v = (hs @ S["wv"][r].T).reshape(T, nkv, hd)
        else:
            r, hs = j, h
            k = rope((h @ w["wk"].T).reshape(T, nkv, hd), pos, cfg.rope_theta)
            v = (h @ w["wv"].T).reshape(T, nkv, hd)
        a = np.empty((T, nq, hd), dtype=F64)
        P = [None] * B
        for b in range(B):
            lo, hi = off[b], off[b + 1]
            a[lo:hi], P[b] = _attention_forward(q[lo:hi], k[lo:hi], v[lo:hi])
        X1 = X + a.reshape(T, nq * hd) @ w["wo"].T
        m = rmsnorm(X1, w["post_norm"], cfg.rms_eps)
        gate, up = m @ w["w_gate"].T, m @ w["w_up"].T
        X2 = X1 + (silu(gate) * up) @ w["w_down"].T
        saved[j] = dict(X=X, h=h, q=q, k=k, v=v, P=P, X1=X1, m=m, gate=gate, up=up, leader=r, hs=hs)
        X = X2
    logits = rmsnorm(X, W.final_norm, cfg.rms_eps) @ W.lm_head().T
    return {"logits": logits, "X_last": X, "saved": saved, "pos": pos, "off": off}


def distill_loss_from_logits(y_teacher: np.ndarray, y_student: np.ndarray, tau: float) -> float:
    pt = softmax_rows(y_teacher / tau)
    log_ps = y_student / tau - np.max(y_student / tau, axis=-1, keepdims=True)
    log_ps = log_ps - np.log(np.sum(np.exp(log_ps), axis=-1, keepdims=True))
    log_pt = np.log(np.maximum(pt, 1e-300))
    return float(tau * tau * np.mean(np.sum(pt * (log_pt - log_ps), axis=-1)))


def distill_loss(cfg: Config, W: Weights, S, tokens, seq_lens, l: int, g: int = 1, tau: float = 2.0) -> float:
    yt = teacher_logits(cfg, W, tokens, seq_lens)
    ys = student_forward(cfg, W, S, tokens, seq_lens, l, g)["logits"]
    return distill_loss_from_logits(yt, ys, tau)


def distill_grads(cfg: Config, W: Weights, S, tokens, seq_lens, l: int, g: int = 1, tau: float = 2.0):
    """Loss of Eq. 3 and its gradients with respect to the student's W_Q, W_K, W_V of every layer > l.
    Returns (loss, {"wq": [...], "wk": [...], "wv": [...]}) -- lists indexed by 0-based layer, None for layers <= l."""
    L, nq, nkv, hd = cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    yt = teacher_logits(cfg, W, tokens, seq_lens)
    fw = student_forward(cfg, W, S, tokens, seq_lens, l, g)
    ys, pos, off = fw["logits"], fw["pos"], fw["off"]
    T, B = ys.shape[0], len(seq_lens)
    loss = distill_loss_from_logits(yt, ys, tau)

    dY = (tau / T) * (softmax_rows(ys / tau) - softmax_rows(yt / tau))          # d loss / d y_student
    dX = _rmsnorm_backward(fw["X_last"], W.final_norm, cfg.rms_eps, dY @ W.lm_head())
    grads = {"wq": [None] * L, "wk": [None] * L, "wv": [None] * L}
    dK_sum = {}
    dV_sum = {}
    for j in range(L - 1, l - 1, -1):
        w, sv = W.layer(j), fw["saved"][j]
        # MLP and its norm
        dact = dX @ w["w_down"]
        sig = 1.0 / (1.0 + np.exp(-sv["gate"]))
        dgate = dact * sv["up"] * sig * (1.0 + sv["gate"] * (1.0 - sig))
        dup = dact * silu(sv["gate"])
        dm = dgate @ w["w_gate"] + dup @ w["w_up"]
        dX1 = dX + _rmsnorm_backward(sv["X1"], w["post_norm"], cfg.rms_eps, dm)
        # attention
        da = (dX1 @ w["wo"]).reshape(T, nq, hd)
        dq = np.empty((T, nq, hd), dtype=F64)
        dk = np.empty((T, nkv, hd), dtype=F64)
        dv = np.empty((T, nkv, hd), dtype=F64)
        for b in range(B):
            lo, hi = off[b], off[b + 1]
            dq[lo:hi], dk[lo:hi], dv[lo:hi] = _attention_backward(sv["q"][lo:hi], sv["k"][lo:hi], sv["v"][lo:hi], sv["P"][b], da[lo:hi])
        # query path: W_Q of this layer, and on into the residual stream
        dq_pre = _rope_backward(dq, pos, cfg.rope_theta).reshape(T, nq * hd)
        grads["wq"][j] = dq_pre.T @ sv["h"]
        dX = dX1 + _rmsnorm_backward(sv["X"], w["in_norm"], cfg.rms_eps, dq_pre @ S["wq"][j])
        # key / value path: collected per AcrossKV group, applied at the leader (x_{l+1} itself is frozen below)
        r = sv["leader"]
        dK_sum[r] = dK_sum.get(r, 0.0) + dk
        dV_sum[r] = dV_sum.get(r, 0.0) + dv
        if j == r:
            dk_pre = _rope_backward(dK_sum[r], pos, cfg.rope_theta).reshape(T, nkv * hd)
            grads["wk"][j] = dk_pre.T @ sv["hs"]
            grads["wv"][j] = dV_sum[r].reshape(T, nkv * hd).T @ sv["hs"]
        else:
            grads["wk"][j] = np.zeros_like(S["wk"][j])
            grads["wv"][j] = np.zeros_like(S["wv"][j])
    return loss, grads


def adamw_update(param, grad, m, v, step: int, lr: float = 3e-4, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8,
                 weight_decay: float = 0.05):
    """One AdamW step (decoupled weight decay), `step` counted from 1.  Returns (param, m, v), all new arrays.
        p <- p (1 - lr wd);  m <- b1 m + (1 - b1) g;  v <- b2 v + (1 - b2) g^2;
        p <- p - lr (m / (1 - b1^t)) / (sqrt(v / (1 - b2^t)) + eps)."""
    param = np.asarray(param, dtype=F64) * (1.0 - lr * weight_decay)
    m = beta1 * np.asarray(m, dtype=F64) + (1.0 - beta1) * grad
    v = beta2 * np.asarray(v, dtype=F64) + (1.0 - beta2) * grad * grad
    m_hat = m / (1.0 - beta1 ** step)
    v_hat = v / (1.0 - beta2 ** step)
    return param - lr * m_hat / (np.sqrt(v_hat) + eps), m, v
