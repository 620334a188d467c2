"""Rotary position embedding of query and key heads, fp64 (TEST INFRASTRUCTURE ONLY).

The paper does not define the position encoding: its models (Experimental Setup: Qwen2.5-1.5B-Instruct,
Phi-4-mini-instruct) are standard decoder-only Transformers with rotary embeddings, and Section 2 says
that attention itself is unchanged.  This is the textbook definition (RoFormer): a head vector x of
even length D is seen as D/2 coordinate pairs, pair j is rotated by the angle pos * theta^(-2j/D).
The pairing is the "half split" one of those models' public implementations: pair j = (x[j], x[j + D/2]).

    y[j]       = x[j] * cos(a_j) - x[j + D/2] * sin(a_j)
    y[j + D/2] = x[j + D/2] * cos(a_j) + x[j] * sin(a_j),      a_j = pos * theta ** (-2 j / D)

Pinned by tests/test_rope_oracle_pins.py: position 0 is the identity; the norm of every pair is kept;
a worked 4-dimensional example; rotations add up (R_a R_b = R_{a+b}); and the defining property of the
method, <R_m q, R_n k> depends on m - n only.
"""
import numpy as np


def rope(x, pos, theta=10000.0):
    """x: [..., D] (D even); pos: scalar or array broadcastable to x.shape[:-1].  Returns fp64 [..., D]."""
    x = np.asarray(x, dtype=np.float64)
    D = x.shape[-1]
    half = D // 2
    j = np.arange(half, dtype=np.float64)
    inv_freq = theta ** (-2.0 * j / D)
    ang = np.asarray(pos, dtype=np.float64)[..., None] * inv_freq
    c, s = np.cos(ang), np.sin(ang)
    lo, hi = x[..., :half], x[..., half:]
    return np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)


def split_and_rope(qkv, pos, q_heads, kv_heads, head_dim, theta=10000.0):
    """qkv: [n, (q_heads + 2 kv_heads) * head_dim], the packed output of a QKV projection; pos: [n].
    Returns (q [n, q_heads, D] rotated, k [n, kv_heads, D] rotated, v [n, kv_heads, D] untouched)."""
    qkv = np.asarray(qkv, dtype=np.float64)
    n = qkv.shape[0]
    a, b = q_heads * head_dim, (q_heads + kv_heads) * head_dim
    q = qkv[:, :a].reshape(n, q_heads, head_dim)
    k = qkv[:, a:b].reshape(n, kv_heads, head_dim)
    v = qkv[:, b:].reshape(n, kv_heads, head_dim)
    p = np.asarray(pos, dtype=np.float64)[:, None]
    return rope(q, p, theta), rope(k, p, theta), v
