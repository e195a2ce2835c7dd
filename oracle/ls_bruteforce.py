"""Second, independent CPU routine -- TEST INFRASTRUCTURE.

Recomputes the decoder WITHOUT any cache, layer by layer on the whole sequence,
with explicit [T, T] causal attention matrices, in float64 numpy.  It exists to
pin the cached, token-by-token C oracle: a different program structure (matrix
form, library matmul), a different language, the same definition (Sec. 4.1 of
the paper for the residual decoder and the shared LM head g; standard Llama
definitions for RMSNorm, rotary embedding, grouped-query attention, SwiGLU).
Tiny models only: cost is O(T^2) per layer and greedy generation recomputes the
full sequence for every new token.
"""
from __future__ import annotations

import numpy as np


def _val(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def _rmsnorm(X, g, eps):
    return X / np.sqrt(np.mean(X * X, axis=-1, keepdims=True) + eps) * g


def _rope(X, positions, hd, theta):
    """X [T, H, hd]; pairs (j, j + hd/2) rotated by pos * theta^(-2j/hd)."""
    half = hd // 2
    inv = theta ** (-2.0 * np.arange(half) / hd)
    ang = positions[:, None, None] * inv[None, None, :]
    c, s = np.cos(ang), np.sin(ang)
    a, b = X[..., :half], X[..., half:]
    return np.concatenate([a * c - b * s, a * s + b * c], axis=-1)


def hidden_states(cfg, w, ids):
    """All hidden states x_0 .. x_L, each [T, D], for the sequence ``ids``."""
    T = len(ids)
    Hq, Hkv, hd = cfg.n_heads, cfg.n_kv_heads, cfg.head_dim
    pos = np.arange(T, dtype=np.float64)
    X = _val(w["tok_embed"])[np.asarray(ids)]
    states = [X.copy()]
    mask = np.triu(np.ones((T, T), dtype=bool), k=1)
    for l in range(cfg.n_layers):
        H = _rmsnorm(X, _val(w["attn_norm"][l]), cfg.rms_eps)
        Q = (H @ _val(w["wq"][l]).T).reshape(T, Hq, hd)
        K = (H @ _val(w["wk"][l]).T).reshape(T, Hkv, hd)
        V = (H @ _val(w["wv"][l]).T).reshape(T, Hkv, hd)
        Q, K = _rope(Q, pos, hd, cfg.rope_theta), _rope(K, pos, hd, cfg.rope_theta)
        rep = Hq // Hkv
        Kr, Vr = np.repeat(K, rep, axis=1), np.repeat(V, rep, axis=1)
        S = np.einsum("qhd,khd->hqk", Q, Kr) / np.sqrt(hd)
        S = np.where(mask[None], -np.inf, S)
        S = S - S.max(axis=-1, keepdims=True)
        A = np.exp(S)
        A = A / A.sum(axis=-1, keepdims=True)
        O = np.einsum("hqk,khd->qhd", A, Vr).reshape(T, Hq * hd)
        X = X + O @ _val(w["wo"][l]).T
        H = _rmsnorm(X, _val(w["ffn_norm"][l]), cfg.rms_eps)
        G = H @ _val(w["w_gate"][l]).T
        U = H @ _val(w["w_up"][l]).T
        X = X + ((G / (1.0 + np.exp(-G))) * U) @ _val(w["w_down"][l]).T
        states.append(X.copy())
    return states


def logits_at(cfg, w, ids, layer):
    """g(x_layer) for every position, [T, V]."""
    X = hidden_states(cfg, w, ids)[layer]
    return _rmsnorm(X, _val(w["final_norm"]), cfg.rms_eps) @ _val(w["lm_head"]).T


def greedy(cfg, w, prompt, max_new, layer=None):
    """Greedy continuation, recomputing the whole sequence for every token."""
    layer = cfg.n_layers if layer is None else layer
    ids = [int(t) for t in prompt]
    out = []
    for _ in range(max_new):
        z = logits_at(cfg, w, ids, layer)[-1]
        t = int(np.argmax(z))  # numpy returns the first maximum
        ids.append(t)
        out.append(t)
    return np.asarray(out, dtype=np.int32)
