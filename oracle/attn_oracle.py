"""ORACLE -- test infrastructure only (tests/, __graft_entry__.smoke() and bench.py's cpu_baseline may use it; the
product never does).  Plain float64 NumPy, slow and obvious.

What sits between the attention projections of a decoder block when one new token is decoded against a cache of
keys and values.  The paper's Section 2 (Preliminaries, "Vision-Language-Action models") names the projections
W_Q, W_K, W_V, W_O of every transformer block and its deployment appendix names the backbone (a LLaMA-2 stack); the
operation between W_Q/W_K/W_V and W_O is not restated there: it is the textbook scaled-dot-product attention with
rotary position embedding, written out here from its definition.

    rope(x, pos)           rotary embedding of one token's heads, "rotate-half" pairing (i, i + D/2)
    attn_decode(q, K, V)   softmax(q K^T * scale) V per head, grouped-query sharing of K/V heads
    attn_bound(q, K, V)    sum_p softmax_p |V_p|: the magnitude the kernel's rounding errors scale with

No blocking, no running maximum, no reordering: the softmax is exp(s - max s) / sum, the output a plain weighted sum.
"""
from __future__ import annotations

import numpy as np


def rope(x: np.ndarray, pos: int, theta: float = 10000.0) -> np.ndarray:
    """x [H][D] (any float type) -> float64 [H][D].  Pair (i, i + D/2) of every head is rotated by the angle
    pos * theta^(-2 i / D):  (a, b) -> (a cos - b sin, b cos + a sin)."""
    x = np.asarray(x, dtype=np.float64)
    H, D = x.shape
    assert D % 2 == 0
    i = np.arange(D // 2, dtype=np.float64)
    ang = float(pos) * theta ** (-2.0 * i / D)
    c, s = np.cos(ang), np.sin(ang)
    a, b = x[:, : D // 2], x[:, D // 2:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=1)


def _scores(q, K, L, scale, G):
    """Softmax weights [H][L] of the query heads against positions 0..L-1 of their key heads."""
    q = np.asarray(q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    H = q.shape[0]
    P = np.empty((H, L), dtype=np.float64)
    for h in range(H):
        s = (K[h // G, :L, :] @ q[h]) * scale
        e = np.exp(s - s.max())
        P[h] = e / e.sum()
    return P


def attn_decode(q: np.ndarray, K: np.ndarray, V: np.ndarray, L: int, scale: float | None = None) -> np.ndarray:
    """q [H][D]; K, V [Hkv][Lmax][D] (head-major caches), positions 0..L-1 valid; H a multiple of Hkv: query head h
    reads key/value head h // (H / Hkv).  Returns float64 [H][D]."""
    H, D = np.asarray(q).shape
    Hkv = np.asarray(K).shape[0]
    assert H % Hkv == 0 and 1 <= L <= np.asarray(K).shape[1]
    G = H // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    P = _scores(q, K, L, scale, G)
    V = np.asarray(V, dtype=np.float64)
    out = np.empty((H, D), dtype=np.float64)
    for h in range(H):
        out[h] = P[h] @ V[h // G, :L, :]
    return out


def attn_bound(q: np.ndarray, K: np.ndarray, V: np.ndarray, L: int, scale: float | None = None) -> np.ndarray:
    """T[h][d] = sum_p softmax_p(h) |V[p][d]|: what an error of relative size eps in the weights or in V turns into."""
    H, D = np.asarray(q).shape
    Hkv = np.asarray(K).shape[0]
    G = H // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    P = _scores(q, K, L, scale, G)
    V = np.abs(np.asarray(V, dtype=np.float64))
    return np.stack([P[h] @ V[h // G, :L, :] for h in range(H)])


def attn_decode_tokens(q: np.ndarray, K: np.ndarray, V: np.ndarray, L: int, scale: float | None = None) -> np.ndarray:
    """Several new tokens at once (the last M of the L cached positions are theirs): q [M][H][D]; token m sees positions
    0 .. L - M + m (itself and everything before it: causal attention).  Returns float64 [M][H][D]."""
    q = np.asarray(q)
    M = q.shape[0]
    assert 1 <= M <= L
    return np.stack([attn_decode(q[m], K, V, L - (M - 1 - m), scale) for m in range(M)])


def attn_bound_tokens(q: np.ndarray, K: np.ndarray, V: np.ndarray, L: int, scale: float | None = None) -> np.ndarray:
    q = np.asarray(q)
    M = q.shape[0]
    return np.stack([attn_bound(q[m], K, V, L - (M - 1 - m), scale) for m in range(M)])
