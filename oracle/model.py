"""Oracle: the transformer evaluated on a subset of rows against a full KV cache.  Test infrastructure.

The paper runs the dLLM on the rows of Eq. 5 only; those rows attend to *all* L
positions (the collected attention has shape H x |y*| x L, Section 4.2), using
freshly computed K/V for the selected rows and the cached K/V for every other
row.  The block itself is the pre-norm decoder block of the models the paper
names (LLaDA-8B, Dream-7B; Section 5.1): RMSNorm, rotary position embedding on
Q and K, bidirectional softmax attention (optionally grouped KV heads), output
projection with residual, RMSNorm, SwiGLU feed-forward with residual.

fp64 throughout; nothing is rounded between steps.  numpy's matmul is the only
library primitive.
"""
from __future__ import annotations

from typing import Dict, Tuple

import numpy as np


def rmsnorm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    """x / sqrt(mean(x^2) + eps) * gain, row-wise."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * gain


def rope(x: np.ndarray, pos: np.ndarray, base: float) -> np.ndarray:
    """Rotary embedding, half-split pairing: dims (t, t + Dh/2) rotate by pos * base^(-2t/Dh).

    x: [n][heads][Dh]; pos: [n] absolute positions.
    """
    n, H, Dh = x.shape
    half = Dh // 2
    t = np.arange(half, dtype=np.float64)
    inv_freq = np.power(float(base), -2.0 * t / Dh)
    ang = np.asarray(pos, dtype=np.float64)[:, None] * inv_freq[None, :]   # [n][half]
    cos, sin = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    lo, hi = x[..., :half], x[..., half:]
    return np.concatenate([lo * cos - hi * sin, hi * cos + lo * sin], axis=-1)


def softmax_rows(s: np.ndarray) -> np.ndarray:
    s = s - np.max(s, axis=-1, keepdims=True)
    e = np.exp(s)
    return e / np.sum(e, axis=-1, keepdims=True)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def layer_on_rows(x: np.ndarray, pos: np.ndarray, Kc: np.ndarray, Vc: np.ndarray,
                  w: Dict[str, np.ndarray], n_q_heads: int, n_kv_heads: int, head_dim: int,
                  rope_base: float, eps: float) -> Tuple[np.ndarray, np.ndarray]:
    """One decoder block on the selected rows of one sequence.

    x:   [n][d] residual stream of the selected rows, pos: [n] their positions.
    Kc, Vc: [L][Hkv][Dh] this layer's cache for this sequence; rows `pos` are
            overwritten with the new K/V *before* attention, all other rows are
            read as they are.
    Returns (new x [n][d], head-averaged attention probabilities [n][L]).
    """
    n, d = x.shape
    Hq, Hkv, Dh = n_q_heads, n_kv_heads, head_dim
    a = rmsnorm(x, w["g_attn"], eps)
    qkv = a @ w["wqkv"].T
    if w.get("bqkv") is not None:
        qkv = qkv + w["bqkv"]
    q = qkv[:, : Hq * Dh].reshape(n, Hq, Dh)
    k = qkv[:, Hq * Dh: (Hq + Hkv) * Dh].reshape(n, Hkv, Dh)
    v = qkv[:, (Hq + Hkv) * Dh:].reshape(n, Hkv, Dh)
    q = rope(q, pos, rope_base)
    k = rope(k, pos, rope_base)
    Kc[pos] = k
    Vc[pos] = v
    L = Kc.shape[0]
    group = Hq // Hkv
    abar = np.zeros((n, L), dtype=np.float64)
    o = np.zeros((n, Hq, Dh), dtype=np.float64)
    for h in range(Hq):
        g = h // group
        s = (q[:, h, :] @ Kc[:, g, :].T) / np.sqrt(float(Dh))      # [n][L], every key, no mask
        P = softmax_rows(s)
        o[:, h, :] = P @ Vc[:, g, :]
        abar += P
    abar /= Hq
    x = x + o.reshape(n, Hq * Dh) @ w["wo"].T
    m = rmsnorm(x, w["g_ffn"], eps)
    x = x + (silu(m @ w["w_gate"].T) * (m @ w["w_up"].T)) @ w["w_down"].T
    return x, abar


def lm_head_conf(x: np.ndarray, g_final: np.ndarray, w_lm: np.ndarray, eps: float
                 ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Eq. 1: distribution over the vocabulary for each given row, its argmax and that token's probability.

    Returns (conf [n] fp64, pred [n] int64 - lowest id among equal maxima, logits [n][V]).
    """
    logits = rmsnorm(x, g_final, eps) @ w_lm.T
    prob = softmax_rows(logits)
    pred = np.argmax(logits, axis=-1)
    conf = prob[np.arange(x.shape[0]), pred]
    return conf, pred.astype(np.int64), logits
