"""Dense, contiguous, full-matrix restatement of a decoder forward in numpy (fp64).

Used only to pin the oracle: the whole sequence (context + chunk) is laid out contiguously,
attention is one [S x S] causally masked softmax per head computed with library matmuls,
there is no cache, no paging and no chunking.  Written independently of the C oracle.
"""
from __future__ import annotations

import numpy as np


def f64(t) -> np.ndarray:
    import torch
    return t.to(torch.float64).numpy() if isinstance(t, torch.Tensor) else np.asarray(t, dtype=np.float64)


def rms(x, g, eps):
    return x / np.sqrt((x * x).mean(axis=-1, keepdims=True) + eps) * g


def rope_all(v, base):
    """v: [S, H, hd]; position of row s is s."""
    S, H, hd = v.shape
    half = hd // 2
    theta = base ** (-2.0 * np.arange(half) / hd)
    ang = np.arange(S)[:, None] * theta[None, :]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    a, b = v[..., :half], v[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def _bf16(a):
    """Round a float64 array to bf16 (nearest even) with torch's conversion, back to float64."""
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()


def dense_forward(shape, glob, layers, tokens, bf16_operands=False):
    """Returns logits [S, V] and the per-layer post-RoPE K and V ([S, Hkv, hd]).
    bf16_operands: round every activation that enters a matrix product (or would be cached) to bf16."""
    rnd = _bf16 if bf16_operands else (lambda a: a)
    S = len(tokens)
    Hq, Hkv, hd = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    x = f64(glob["embed"])[np.asarray(tokens)]
    mask = np.tril(np.ones((S, S), dtype=bool))
    kvs = []
    for w in layers:
        h = rnd(rms(x, f64(w["norm1"]), shape.rms_eps))
        q = rnd(rope_all((h @ f64(w["wq"]).T).reshape(S, Hq, hd), shape.rope_base))
        k = rnd(rope_all((h @ f64(w["wk"]).T).reshape(S, Hkv, hd), shape.rope_base))
        v = rnd((h @ f64(w["wv"]).T).reshape(S, Hkv, hd))
        kvs.append((k, v))
        kr, vr = np.repeat(k, Hq // Hkv, axis=1), np.repeat(v, Hq // Hkv, axis=1)
        sc = np.einsum("shd,thd->hst", q, kr) / np.sqrt(hd)
        sc = np.where(mask[None], sc, -np.inf)
        sc = np.exp(sc - sc.max(axis=-1, keepdims=True))
        pr = sc / sc.sum(axis=-1, keepdims=True)
        att = rnd(np.einsum("hst,thd->shd", pr, vr).reshape(S, Hq * hd))
        x = x + att @ f64(w["wo"]).T
        h2 = rnd(rms(x, f64(w["norm2"]), shape.rms_eps))
        g, u = h2 @ f64(w["wg"]).T, h2 @ f64(w["wu"]).T
        x = x + rnd(g / (1.0 + np.exp(-g)) * u) @ f64(w["wd"]).T
    logits = rnd(rms(x, f64(glob["final_norm"]), shape.rms_eps)) @ f64(glob["lm_head"]).T
    return logits, kvs
