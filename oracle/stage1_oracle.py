"""Plain NumPy oracle for the inter-tensor stage: HSIC sensitivities and the
layer-balanced bit allocation.

TEST INFRASTRUCTURE ONLY: imported by tests, the smoke check and the
benchmark's CPU baseline.  It shares no code with the CUDA path and is never
tuned for speed.  Everything is float64.

What it states (paper passages in brackets):

* RBF kernel matrix [Section 3, HSIC paragraph: the Gaussian (RBF) kernel is the one used]:
  k(a, a') = exp(-|a - a'|^2 / (2 sigma^2)).  The paper does not print the
  bandwidth; here sigma is an argument.
* empirical HSIC [Eq. 2]: (K-1)^-2 tr(K_A C K_B C), C = I - 11^T / K.
* sensitivity of a matrix [Eq. 5]: -alpha HSIC(X, Z) + beta HSIC(Z, Y).
* predicted error and objective [Eq. 6]: eta(t) = 2^(-2 b(t)),
  E_l = sum_j S_j eta(t_j) over the matrices of layer l, objective sum_l E_l^2,
  subject to the parameter-weighted mean bit-width <= b_bar.
* solver ["Solver" paragraph of Section 4.1]: every matrix starts at the
  cheapest type; each step applies the single-type upgrade with the largest
  (E_l^2 - E~_l^2) / extra bits.  Readings taken where the text is open: an
  upgrade moves a matrix to the next type of the ascending list; extra bits =
  (b_new - b_old) * number of weights; only upgrades that keep the budget are
  candidates; the loop ends when no candidate is left or the best candidate
  does not lower the objective; ties go to the lowest matrix index.

Pins: tests/test_oracle_stage1.py (closed forms for K = 2, the V-statistic
form of the appendix, invariances, pure-Python brute force, exhaustive search
on small allocation problems).  No function here is "parity unpinned".
"""
from __future__ import annotations

import numpy as np


# --------------------------------------------------------------------------
# HSIC [Eq. 2]
# --------------------------------------------------------------------------
def sq_dists(A: np.ndarray) -> np.ndarray:
    """D[i][j] = |a_i - a_j|^2 from the differences themselves (no Gram-matrix shortcut)."""
    A = np.asarray(A, dtype=np.float64)
    K = A.shape[0]
    D = np.empty((K, K), dtype=np.float64)
    for i in range(K):
        diff = A - A[i]
        D[i] = np.einsum("kd,kd->k", diff, diff)
    return D


def rbf_gram(A: np.ndarray, sigma: float) -> np.ndarray:
    """[K_A]_ij = exp(-|a_i - a_j|^2 / (2 sigma^2))  [Section 3, HSIC paragraph]."""
    if not sigma > 0:
        raise ValueError("sigma must be positive")
    return np.exp(-sq_dists(A) / (2.0 * float(sigma) ** 2))


def centering(K: int) -> np.ndarray:
    """C = I - (1/K) 1 1^T  [below Eq. 2]."""
    return np.eye(K, dtype=np.float64) - np.full((K, K), 1.0 / K, dtype=np.float64)


def hsic(KA: np.ndarray, KB: np.ndarray) -> float:
    """(K-1)^-2 tr(K_A C K_B C)  [Eq. 2], the four-factor product written out."""
    KA = np.asarray(KA, dtype=np.float64)
    KB = np.asarray(KB, dtype=np.float64)
    K = KA.shape[0]
    if KA.shape != (K, K) or KB.shape != (K, K) or K < 2:
        raise ValueError("two K x K kernel matrices with K >= 2 are needed")
    C = centering(K)
    return float(np.trace(KA @ C @ KB @ C) / float(K - 1) ** 2)


def hsic_large(KA: np.ndarray, KB: np.ndarray) -> float:
    """Eq. 2 for sample counts where the four-factor product of `hsic` is out of reach: C K_A C is formed by removing
    row means, column means and adding back the grand mean (what multiplying by C on both sides does), then
    tr(K_A C K_B C) = sum_ij (C K_A C)_ij [K_B]_ji.  Pinned against `hsic` on small sizes."""
    KA = np.asarray(KA, dtype=np.float64)
    KB = np.asarray(KB, dtype=np.float64)
    K = KA.shape[0]
    centred = KA - KA.mean(axis=1, keepdims=True) - KA.mean(axis=0, keepdims=True) + KA.mean()
    return float(np.sum(centred * KB.T) / float(K - 1) ** 2)


def sensitivity(hsic_xz: float, hsic_zy: float, alpha: float, beta: float) -> float:
    """S(W) = -alpha HSIC(X, Z) + beta HSIC(Z, Y)  [Eq. 5]."""
    return -float(alpha) * float(hsic_xz) + float(beta) * float(hsic_zy)


def sensitivity_from_samples(X, Z, Y, sigma_x, sigma_z, sigma_y, alpha, beta):
    """Eq. 5 from the calibration samples: X [K][d_in], Z [K][d_j], Y [K][d_a].
    Returns (S, HSIC(X, Z), HSIC(Z, Y))."""
    KX, KZ, KY = rbf_gram(X, sigma_x), rbf_gram(Z, sigma_z), rbf_gram(Y, sigma_y)
    hxz, hzy = hsic(KX, KZ), hsic(KZ, KY)
    return sensitivity(hxz, hzy, alpha, beta), hxz, hzy


# --------------------------------------------------------------------------
# Bit allocation [Eq. 6 and the solver paragraph]
# --------------------------------------------------------------------------
def eta(bits: int) -> float:
    """Per-element squared-error scale of an n-bit type: 2^(-2 n)  [above Eq. 6]."""
    return 2.0 ** (-2 * int(bits))


def layer_errors(S, bits, layer_of, n_layers=None) -> np.ndarray:
    """E_l = sum over the matrices j of layer l of S_j eta(t_j)  [Eq. 6]."""
    S = np.asarray(S, dtype=np.float64)
    layer_of = np.asarray(layer_of, dtype=np.int64)
    L = int(layer_of.max()) + 1 if n_layers is None else int(n_layers)
    E = np.zeros(L, dtype=np.float64)
    for j in range(S.shape[0]):
        E[layer_of[j]] += S[j] * eta(bits[j])
    return E


def objective(S, bits, layer_of) -> float:
    """sum_l E_l^2  [Eq. 6]."""
    E = layer_errors(S, bits, layer_of)
    return float(np.sum(E * E))


def mean_bits(bits, numel) -> float:
    """Parameter-weighted mean bit-width, the left side of the constraint of Eq. 6."""
    bits = np.asarray(bits, dtype=np.float64)
    numel = np.asarray(numel, dtype=np.float64)
    return float(np.sum(bits * numel) / np.sum(numel))


def allocate_bits(S, numel, layer_of, types, budget):
    """Greedy solver of Eq. 6.  `types`: ascending list of bit-widths; `budget`: b_bar.
    Returns (bits per matrix, list of applied steps (matrix, from, to, ratio))."""
    S = np.asarray(S, dtype=np.float64)
    numel = [int(v) for v in numel]
    layer_of = [int(v) for v in layer_of]
    types = [int(t) for t in types]
    n = S.shape[0]
    if sorted(set(types)) != types or not types:
        raise ValueError("types must be a strictly ascending list")
    total = sum(numel)
    level = [0] * n                              # index into types
    used = types[0] * total                      # sum of b(t_j) |W_j|
    if used > budget * total:
        raise ValueError("the budget is below the cheapest type")
    L = max(layer_of) + 1
    E = [0.0] * L
    for j in range(n):
        E[layer_of[j]] += S[j] * eta(types[0])
    steps = []
    while True:
        best, best_ratio, best_E = -1, 0.0, 0.0
        for j in range(n):
            if level[j] + 1 >= len(types):
                continue
            b0, b1 = types[level[j]], types[level[j] + 1]
            extra = (b1 - b0) * numel[j]
            if used + extra > budget * total:
                continue
            l = layer_of[j]
            E_new = E[l] + S[j] * (eta(b1) - eta(b0))
            ratio = (E[l] * E[l] - E_new * E_new) / extra
            if best < 0 or ratio > best_ratio:
                best, best_ratio, best_E = j, ratio, E_new
        if best < 0 or not best_ratio > 0.0:
            break
        b0, b1 = types[level[best]], types[level[best] + 1]
        steps.append((best, b0, b1, best_ratio))
        used += (b1 - b0) * numel[best]
        E[layer_of[best]] = best_E
        level[best] += 1
    return np.array([types[v] for v in level], dtype=np.int64), steps
