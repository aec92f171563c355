"""Seeded synthetic inputs shaped like the quantised VLA backbones' linears.

This module only draws numbers and lists shapes.  It holds none of the
quantisation or matmul arithmetic and is the one module that tests may hand to
both the CUDA path and the CPU oracle.

Shapes follow the transformer-block matrix set J = {Q, K, V, O, up, down,
gate} of Section 3; a shape is written (N, K) = (out features, in features).
"""
from __future__ import annotations

import numpy as np

MATS = ("q", "k", "v", "o", "gate", "up", "down")


def llama7b_layer():
    """LLaMA-2-7B-shaped block: hidden 4096, MLP 11008."""
    return [("q", 4096, 4096), ("k", 4096, 4096), ("v", 4096, 4096), ("o", 4096, 4096),
            ("gate", 11008, 4096), ("up", 11008, 4096), ("down", 4096, 11008)]


def gemma2b_layer():
    """Gemma-2B-shaped block: hidden 2048, one 256-wide KV head, MLP 16384."""
    return [("q", 2048, 2048), ("k", 256, 2048), ("v", 256, 2048), ("o", 2048, 2048),
            ("gate", 16384, 2048), ("up", 16384, 2048), ("down", 2048, 16384)]


def expert_layer():
    """Action-expert block: hidden 1024, shared head geometry (q width 2048,
    KV width 256), MLP 4096."""
    return [("q", 2048, 1024), ("k", 256, 1024), ("v", 256, 1024), ("o", 1024, 2048),
            ("gate", 4096, 1024), ("up", 4096, 1024), ("down", 1024, 4096)]


def tiny_layer(hidden=256, mlp=384):
    """Small block with the same structure, for tests that the oracle finishes
    in seconds; sizes span several tiles and a ragged tail."""
    return [("q", hidden, hidden), ("k", hidden, hidden), ("v", hidden, hidden), ("o", hidden, hidden),
            ("gate", mlp, hidden), ("up", mlp, hidden), ("down", hidden, mlp)]


def _rng(*key) -> np.random.Generator:
    return np.random.default_rng(np.random.SeedSequence([int(k) & 0xFFFFFFFF for k in key]))


def weights(N: int, K: int, *key, outliers: bool = False) -> np.ndarray:
    """fp32 [N][K], iid N(0, 0.02); with `outliers`, an independent
    Bernoulli(0.001) subset is multiplied by 20."""
    g = _rng(0x57, *key)
    W = (g.standard_normal((N, K), dtype=np.float32) * np.float32(0.02)).astype(np.float32)
    if outliers:
        mask = g.random((N, K), dtype=np.float32) < np.float32(0.001)
        W = np.where(mask, W * np.float32(20.0), W).astype(np.float32)
    return W


def activations(M: int, K: int, *key, kind: str = "normal") -> np.ndarray:
    """fp32 [M][K].  'normal': iid N(0,1).  'vision_text': the first half of
    the rows N(0,1) times a per-row scale U(0.5, 2) (vision patches), the rest
    N(0,1) (text)."""
    g = _rng(0xA7, *key)
    x = g.standard_normal((M, K), dtype=np.float32)
    if kind == "vision_text":
        nv = M // 2
        s = g.uniform(0.5, 2.0, size=(nv, 1)).astype(np.float32)
        x[:nv] *= s
    elif kind != "normal":
        raise ValueError(kind)
    return x


def draw_bits(sizes, mean_bits: float, seed: int):
    """Per-matrix bit-widths from {2,3,4} whose parameter-weighted mean is
    `mean_bits` (to within 0.005).

    Draw iid with p = (0.6, 0.3, 0.1) for a 2.5 target, uniform otherwise;
    then walk a seeded permutation, moving one matrix at a time one bit toward
    the target while that brings the mean closer.
    """
    sizes = np.asarray(sizes, dtype=np.float64)
    g = _rng(0xB1, seed)
    p = (0.6, 0.3, 0.1) if mean_bits <= 2.75 else (1 / 3, 1 / 3, 1 / 3)
    bits = g.choice([2, 3, 4], size=len(sizes), p=p).astype(np.int64)
    total = sizes.sum()

    def mean():
        return float((bits * sizes).sum() / total)

    for _ in range(64):
        if abs(mean() - mean_bits) <= 0.005:
            break
        moved = False
        for i in g.permutation(len(sizes)):
            err = mean() - mean_bits
            if abs(err) <= 0.005:
                break
            step = -1 if err > 0 else 1
            nb = bits[i] + step
            if nb < 2 or nb > 4:
                continue
            new_err = err + step * sizes[i] / total
            if abs(new_err) < abs(err):
                bits[i] = nb
                moved = True
        if not moved:
            break
    return [int(b) for b in bits]


def stack_shapes(layer, n_layers: int):
    """[(layer index, name, N, K)] for n_layers copies of a block."""
    return [(l, name, N, K) for l in range(n_layers) for (name, N, K) in layer]


# ---- device-side generation for full-size stacks (the host generator would
# ---- take minutes for 6.5e9 weights); the oracle sees sampled rows copied back
def weights_device(N: int, K: int, seed: int, outliers: bool = False, device="cuda"):
    """fp32 [N][K] on the GPU, N(0,0.02) (+ optional 0.1 % x20 outliers), from
    a seeded torch generator."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) & 0x7FFFFFFF)
    W = torch.empty((N, K), dtype=torch.float32, device=device)
    W.normal_(0.0, 0.02, generator=g)
    if outliers:
        mask = torch.empty((N, K), dtype=torch.float32, device=device).uniform_(0.0, 1.0, generator=g) < 0.001
        W = torch.where(mask, W * 20.0, W)
    return W


def calibration(K: int, d_in: int, d_out: int, d_act: int, *key, relevance: float = 0.5, redundancy: float = 0.5):
    """Calibration samples for the inter-tensor stage (Section 4.1): backbone inputs X [K][d_in], the outputs
    Z [K][d_out] of one weight matrix and action labels Y [K][d_act], float32, roughly unit variance per feature.
    Z mixes a random projection of X (weight `redundancy`), a latent that also drives Y (weight `relevance`) and
    independent noise, so that HSIC(X, Z) and HSIC(Z, Y) move with the two knobs."""
    g = _rng(0xCA, *key)
    X = g.standard_normal((K, d_in), dtype=np.float32)
    latent = g.standard_normal((K, d_act), dtype=np.float32)
    P = g.standard_normal((d_in, d_out), dtype=np.float32) / np.float32(np.sqrt(d_in))
    R = g.standard_normal((d_act, d_out), dtype=np.float32) / np.float32(np.sqrt(d_act))
    noise = g.standard_normal((K, d_out), dtype=np.float32)
    rest = max(0.0, 1.0 - redundancy**2 - relevance**2) ** 0.5
    Z = (np.float32(redundancy) * np.tanh(X @ P) * np.float32(1.6) + np.float32(relevance) * (latent @ R) + np.float32(rest) * noise)
    Y = np.tanh(latent) + np.float32(0.1) * g.standard_normal((K, d_act), dtype=np.float32)
    return X, Z.astype(np.float32), Y.astype(np.float32)


def sensitivities(n_layers: int, per_layer: int, *key) -> np.ndarray:
    """Seeded stand-in for the Eq. 5 scores of a stack: positive, log-normally spread, a fifth of them negative."""
    g = _rng(0x5E, *key)
    S = np.exp(g.standard_normal(n_layers * per_layer)) * 1e-3
    S[g.random(n_layers * per_layer) < 0.2] *= -0.3
    return S
