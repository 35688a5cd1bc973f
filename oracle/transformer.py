"""CPU fp64 oracle, part 1: the decoder-only Transformer forward that verification runs.

TEST INFRASTRUCTURE ONLY.  Slow, plain numpy in float64, written to be checked by eye.  It shares
no code with the CUDA path and must never be imported by the product package.

The paper does not define the network (it runs Llama-family checkpoints through a stock
library, Section 4.1 "Hardware and Implementation"); the architecture below is the Llama
layer: pre-RMSNorm, rotary positions on half-split pairs, grouped-query attention, SwiGLU FFN,
no biases, untied LM head.  What the paper does define is *which keys each query row may see*
when several lengthened drafts are verified in one forward (Section 3.2, Eq. 7 and Eq. 8); that
enters here only as the boolean ``visible`` matrix, applied as a dense mask.

Pins (tests/test_oracle_transformer.py): logits equal an independent library implementation of
the Llama forward in float64; single-visible-key, uniform-score, RoPE and RMSNorm closed forms.
"""
from __future__ import annotations

import numpy as np


class Weights:
    """float64 copies of the model tensors (values are exactly the fp32 / bf16 inputs)."""

    def __init__(self, desc, w):
        f = lambda t: np.asarray(t.detach().to("cpu").double().numpy() if hasattr(t, "detach") else t, dtype=np.float64)
        self.desc = desc
        self.embed = f(w["embed"])
        self.final_norm = f(w["final_norm"])
        self.lm_head = f(w["lm_head"])
        self.layers = [{k: f(v) for k, v in lw.items()} for lw in w["layers"][: desc.n_layers]]


class KVCache:
    """K and V of every cached slot: arrays [n_layers, max_seq, n_kv_heads, head_dim]; ``length`` slots valid."""

    def __init__(self, desc, k=None, v=None, length=0):
        shp = (desc.n_layers, desc.max_seq, desc.n_kv_heads, desc.head_dim)
        self.k = np.zeros(shp) if k is None else np.array(k, dtype=np.float64)
        self.v = np.zeros(shp) if v is None else np.array(v, dtype=np.float64)
        self.length = length

    def clone(self):
        c = KVCache.__new__(KVCache)
        c.k, c.v, c.length = self.k.copy(), self.v.copy(), self.length
        return c


def rmsnorm(x, g, eps):
    """g * x / sqrt(mean(x^2) + eps), row-wise."""
    return g * x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps)


def rope(x, pos, theta):
    """Rotate pairs (x_i, x_{i+h/2}) of each head vector by the angle pos * theta^(-2i/h).
    x: [B, heads, h]; pos: [B] integer positions (0-based)."""
    h = x.shape[-1]
    half = h // 2
    inv = theta ** (-2.0 * np.arange(half, dtype=np.float64) / h)
    ang = np.asarray(pos, dtype=np.float64)[:, None] * inv[None, :]           # [B, half]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    a, b = x[..., :half], x[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def masked_attention(q, k, v, visible):
    """softmax(q k^T / sqrt(h)) v over visible keys only, written as the dense definition.
    q: [B, H, h]; k, v: [T, H_kv, h]; visible: bool [B, T]; query head a reads kv head a // (H / H_kv)."""
    B, H, h = q.shape
    Hkv = k.shape[1]
    out = np.zeros((B, H, h))
    for a in range(H):
        ka, va = k[:, a // (H // Hkv), :], v[:, a // (H // Hkv), :]
        s = q[:, a, :] @ ka.T / np.sqrt(float(h))
        s = np.where(visible, s, -np.inf)
        p = np.exp(s - s.max(axis=-1, keepdims=True))
        p /= p.sum(axis=-1, keepdims=True)
        out[:, a, :] = p @ va
    return out


def forward(W: Weights, cache: KVCache, tokens, pos, visible, n_layers=None):
    """One forward of a query block against the cache.

    The block's K/V are written to cache slots length .. length+B-1 (the caller advances or
    compacts ``cache.length`` afterwards).  ``visible[r, s]`` says whether block row r may attend
    cache slot s, for s in [0, length + B).  Returns the next-token logits [B, vocab]."""
    d = W.desc
    tokens = np.asarray(tokens)
    B, L = len(tokens), cache.length
    assert visible.shape == (B, L + B) and L + B <= d.max_seq
    x = W.embed[tokens]
    for l in range(d.n_layers if n_layers is None else n_layers):
        lw = W.layers[l]
        n1 = rmsnorm(x, lw["attn_norm"], d.rms_eps)
        q = rope((n1 @ lw["wq"].T).reshape(B, d.n_heads, d.head_dim), pos, d.rope_theta)
        k = rope((n1 @ lw["wk"].T).reshape(B, d.n_kv_heads, d.head_dim), pos, d.rope_theta)
        v = (n1 @ lw["wv"].T).reshape(B, d.n_kv_heads, d.head_dim)
        cache.k[l, L:L + B], cache.v[l, L:L + B] = k, v
        att = masked_attention(q, cache.k[l, :L + B], cache.v[l, :L + B], visible)
        x = x + att.reshape(B, -1) @ lw["wo"].T
        n2 = rmsnorm(x, lw["ffn_norm"], d.rms_eps)
        g, u = n2 @ lw["w_gate"].T, n2 @ lw["w_up"].T
        x = x + ((g / (1.0 + np.exp(-g))) * u) @ lw["w_down"].T
    return rmsnorm(x, W.final_norm, d.rms_eps) @ W.lm_head.T


def argmax_rows(logits):
    """Greedy choice per row; ties go to the smallest token id (np.argmax returns the first maximum)."""
    return np.argmax(logits, axis=-1).astype(np.int64)


def causal_visible(L, B):
    """Plain autoregressive visibility: row r sees slots 0 .. L + r."""
    return np.arange(L + B)[None, :] <= (L + np.arange(B))[:, None]
