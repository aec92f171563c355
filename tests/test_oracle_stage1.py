"""Pins for the inter-tensor oracle (HSIC of Eq. 2, sensitivity of Eq. 5, allocation of Eq. 6).

None of these re-types the oracle's own formula: they are closed forms, the
appendix's V-statistic form, invariances of the estimator, pure-Python brute
force, and exhaustive search over small allocation problems.
"""
import itertools
import math

import numpy as np
import pytest

from oracle import stage1_oracle as S1


def _samples(K, d, seed, scale=1.0):
    return np.random.default_rng(seed).standard_normal((K, d)) * scale


# ---------------------------------------------------------------- kernel matrix
def test_rbf_gram_brute_force_python_loops():
    A = _samples(7, 5, 1)
    sigma = 1.7
    G = S1.rbf_gram(A, sigma)
    for i in range(7):
        for j in range(7):
            d2 = 0.0
            for k in range(5):
                d2 += (float(A[i, k]) - float(A[j, k])) ** 2
            assert G[i, j] == pytest.approx(math.exp(-d2 / (2 * sigma * sigma)), rel=1e-14)


def test_rbf_gram_structure():
    A = _samples(20, 9, 2)
    G = S1.rbf_gram(A, 3.0)
    assert np.array_equal(np.diag(G), np.ones(20))          # k(a, a) = 1
    assert np.array_equal(G, G.T)
    assert np.all((G > 0) & (G <= 1))
    assert np.linalg.eigvalsh(G).min() > -1e-12               # a Gaussian kernel matrix is positive semi-definite


def test_rbf_gram_two_points_on_a_line():
    # |a - a'| = 3, sigma = 1.5: exp(-9 / 4.5) = exp(-2)
    G = S1.rbf_gram(np.array([[0.0], [3.0]]), 1.5)
    assert G[0, 1] == pytest.approx(math.exp(-2.0), rel=1e-15)


def test_rbf_gram_invariant_under_shift_and_rotation():
    A = _samples(12, 6, 3)
    Q, _ = np.linalg.qr(_samples(6, 6, 4))
    G0 = S1.rbf_gram(A, 2.0)
    assert np.allclose(S1.rbf_gram(A @ Q + 5.0, 2.0), G0, rtol=1e-12, atol=0)
    # scaling the data and the bandwidth together changes nothing
    assert np.allclose(S1.rbf_gram(3.0 * A, 6.0), G0, rtol=1e-12, atol=0)


# ---------------------------------------------------------------- Eq. 2
def test_hsic_two_samples_closed_form():
    """K = 2: C K C = ((1 - a)/2) [[1,-1],[-1,1]], so tr(K_A C K_B C) = (1 - a)(1 - b) and (K-1)^2 = 1."""
    for a, b in ((0.3, 0.8), (0.0, 0.5), (1.0, 0.2)):
        KA = np.array([[1.0, a], [a, 1.0]])
        KB = np.array([[1.0, b], [b, 1.0]])
        assert S1.hsic(KA, KB) == pytest.approx((1 - a) * (1 - b), abs=1e-15)


def test_hsic_equals_v_statistic_form_of_the_appendix():
    """The population form (three expectations, Appendix A) with sample means in place of the
    expectations equals tr(K_A C K_B C) / K^2, i.e. Eq. 2 times ((K-1)/K)^2."""
    K = 9
    KA = S1.rbf_gram(_samples(K, 4, 5), 1.5)
    KB = S1.rbf_gram(_samples(K, 3, 6), 1.2)
    t1 = sum(KA[i, j] * KB[i, j] for i in range(K) for j in range(K)) / K**2
    t2 = (sum(KA[i, j] for i in range(K) for j in range(K)) / K**2) * (sum(KB[i, j] for i in range(K) for j in range(K)) / K**2)
    t3 = sum((sum(KA[i, j] for j in range(K)) / K) * (sum(KB[i, j] for j in range(K)) / K) for i in range(K)) / K
    v_stat = t1 + t2 - 2 * t3
    assert S1.hsic(KA, KB) == pytest.approx(v_stat * K**2 / (K - 1) ** 2, rel=1e-12)


def test_hsic_brute_force_python_loops():
    K = 6
    KA = S1.rbf_gram(_samples(K, 3, 7), 1.0)
    KB = S1.rbf_gram(_samples(K, 2, 8), 1.0)
    C = [[(1.0 if i == j else 0.0) - 1.0 / K for j in range(K)] for i in range(K)]

    def mm(P, Q):
        return [[sum(P[i][k] * Q[k][j] for k in range(K)) for j in range(K)] for i in range(K)]

    M = mm(mm(mm(KA.tolist(), C), KB.tolist()), C)
    assert S1.hsic(KA, KB) == pytest.approx(sum(M[i][i] for i in range(K)) / (K - 1) ** 2, rel=1e-12)


def test_hsic_symmetry_permutation_and_constant_variable():
    K = 15
    A, B = _samples(K, 5, 9), _samples(K, 4, 10)
    KA, KB = S1.rbf_gram(A, 2.0), S1.rbf_gram(B, 2.0)
    h = S1.hsic(KA, KB)
    assert S1.hsic(KB, KA) == pytest.approx(h, rel=1e-12)
    p = np.random.default_rng(11).permutation(K)
    assert S1.hsic(KA[np.ix_(p, p)], KB[np.ix_(p, p)]) == pytest.approx(h, rel=1e-12)
    # a variable that takes one value only: K_B = 1 1^T, C 1 = 0, HSIC = 0
    assert abs(S1.hsic(KA, np.ones((K, K)))) < 1e-15
    # adding a constant matrix to either kernel matrix changes nothing (C removes it)
    assert S1.hsic(KA + 0.37, KB) == pytest.approx(h, rel=1e-11)
    assert h >= -1e-15      # trace of a product of two centred positive semi-definite matrices


def test_hsic_self_is_centred_frobenius_norm():
    K = 11
    KA = S1.rbf_gram(_samples(K, 3, 12), 1.3)
    row = KA.mean(axis=1, keepdims=True)
    centred = KA - row - row.T + KA.mean()
    assert S1.hsic(KA, KA) == pytest.approx(np.sum(centred**2) / (K - 1) ** 2, rel=1e-12)


def test_hsic_large_equals_the_literal_trace():
    for K, seed in ((2, 20), (7, 21), (40, 22)):
        g = np.random.default_rng(seed)
        KA = S1.rbf_gram(g.standard_normal((K, 3)), 1.1)
        KB = S1.rbf_gram(g.standard_normal((K, 2)), 0.9)
        assert S1.hsic_large(KA, KB) == pytest.approx(S1.hsic(KA, KB), rel=1e-11, abs=1e-16)
        # also for matrices that are not symmetric (the transpose in the trace matters)
        A, B = g.random((K, K)), g.random((K, K))
        assert S1.hsic_large(A, B) == pytest.approx(S1.hsic(A, B), rel=1e-10, abs=1e-14)


def test_hsic_tells_dependence_from_independence():
    K = 200
    g = np.random.default_rng(13)
    A = g.standard_normal((K, 3))
    dep = np.tanh(A @ g.standard_normal((3, 2))) + 0.05 * g.standard_normal((K, 2))
    ind = g.standard_normal((K, 2))
    KA = S1.rbf_gram(A, math.sqrt(3.0))
    h_dep = S1.hsic(KA, S1.rbf_gram(dep, 1.0))
    h_ind = S1.hsic(KA, S1.rbf_gram(ind, math.sqrt(2.0)))
    assert h_dep > 10 * h_ind > 0


# ---------------------------------------------------------------- Eq. 5
def test_sensitivity_signs_and_weights():
    assert S1.sensitivity(0.2, 0.5, 1.0, 1.0) == pytest.approx(0.3)
    assert S1.sensitivity(0.2, 0.5, 0.0, 2.0) == pytest.approx(1.0)       # task relevance only
    assert S1.sensitivity(0.2, 0.5, 3.0, 0.0) == pytest.approx(-0.6)      # input redundancy only, subtracted
    X, Z, Y = _samples(10, 4, 14), _samples(10, 3, 15), _samples(10, 2, 16)
    s, hxz, hzy = S1.sensitivity_from_samples(X, Z, Y, 2.0, 1.7, 1.4, 0.5, 4.0)
    assert hxz == pytest.approx(S1.hsic(S1.rbf_gram(X, 2.0), S1.rbf_gram(Z, 1.7)), rel=1e-13)
    assert hzy == pytest.approx(S1.hsic(S1.rbf_gram(Z, 1.7), S1.rbf_gram(Y, 1.4)), rel=1e-13)
    assert s == pytest.approx(-0.5 * hxz + 4.0 * hzy, rel=1e-13)


# ---------------------------------------------------------------- Eq. 6
def test_eta_and_layer_errors_by_hand():
    assert [S1.eta(b) for b in (2, 3, 4)] == [1 / 16, 1 / 64, 1 / 256]
    S = [1.0, 2.0, 4.0]
    # layer 0 holds matrices 0 and 2, layer 1 holds matrix 1
    E = S1.layer_errors(S, [2, 3, 4], [0, 1, 0])
    assert E.tolist() == [1 / 16 + 4 / 256, 2 / 64]
    assert S1.objective(S, [2, 3, 4], [0, 1, 0]) == (1 / 16 + 4 / 256) ** 2 + (2 / 64) ** 2
    assert S1.mean_bits([2, 3, 4], [10, 10, 20]) == (20 + 30 + 80) / 40


def _problem(n, L, seed, signed=False):
    g = np.random.default_rng(seed)
    S = g.uniform(0.1, 2.0, n)
    if signed:
        S[g.random(n) < 0.25] *= -1.0
    numel = g.choice([16, 43, 4, 64], n)
    layer_of = np.arange(n) % L
    return S, numel, layer_of


def _exhaustive(S, numel, layer_of, types, budget):
    best, arg = None, None
    for combo in itertools.product(types, repeat=len(S)):
        if S1.mean_bits(combo, numel) <= budget + 1e-15:
            v = S1.objective(S, combo, layer_of)
            if best is None or v < best:
                best, arg = v, combo
    return best, arg


@pytest.mark.parametrize("seed", range(6))
def test_allocation_feasible_and_each_step_is_the_best_ratio(seed):
    S, numel, layer_of = _problem(9, 3, seed, signed=(seed % 2 == 1))
    types, budget = [2, 3, 4], 2.8
    bits, steps = S1.allocate_bits(S, numel, layer_of, types, budget)
    assert S1.mean_bits(bits, numel) <= budget
    assert set(bits.tolist()) <= set(types)
    # replay: before every applied step no other feasible single upgrade has a larger gain per bit
    cur = [2] * len(S)
    total = int(np.sum(numel))
    for (j, b0, b1, ratio) in steps:
        assert cur[j] == b0 and b1 == b0 + 1
        obj0 = S1.objective(S, cur, layer_of)
        for c in range(len(S)):
            if cur[c] == 4:
                continue
            trial = list(cur)
            trial[c] += 1
            if np.dot(trial, numel) > budget * total:
                continue
            r = (obj0 - S1.objective(S, trial, layer_of)) / numel[c]
            assert r <= ratio * (1 + 1e-9) + 1e-18
        cur[j] = b1
        assert ratio > 0
    assert cur == bits.tolist()
    # the objective never goes up along the path and ends no better than the exhaustive optimum
    opt, _ = _exhaustive(S, numel, layer_of, types, budget)
    assert S1.objective(S, bits, layer_of) >= opt - 1e-18
    assert S1.objective(S, bits, layer_of) <= S1.objective(S, [2] * len(S), layer_of)


def test_allocation_reaches_the_optimum_on_separable_problems():
    """One matrix per layer and equal sizes: the objective is a sum of independent convex terms and every
    upgrade costs the same, so the greedy path is optimal whenever the budget is used up exactly."""
    S = np.array([3.0, 1.0, 0.2, 2.0])
    numel = [10, 10, 10, 10]
    layer_of = [0, 1, 2, 3]
    for budget in (2.25, 2.5, 2.75, 3.0, 3.5):
        bits, _ = S1.allocate_bits(S, numel, layer_of, [2, 3, 4], budget)
        opt, arg = _exhaustive(S, numel, layer_of, [2, 3, 4], budget)
        assert S1.objective(S, bits, layer_of) == pytest.approx(opt, rel=1e-12)
    # the most sensitive matrix gets the first upgrade
    bits, steps = S1.allocate_bits(S, numel, layer_of, [2, 3, 4], 2.25)
    assert bits.tolist() == [3, 2, 2, 2] and steps[0][0] == 0


def test_allocation_limits_and_invariances():
    S, numel, layer_of = _problem(12, 4, 20)
    types = [2, 3, 4]
    # budget at the cheapest type: nothing moves; generous budget: everything at the top type
    assert S1.allocate_bits(S, numel, layer_of, types, 2.0)[0].tolist() == [2] * 12
    assert S1.allocate_bits(S, numel, layer_of, types, 4.0)[0].tolist() == [4] * 12
    with pytest.raises(ValueError):
        S1.allocate_bits(S, numel, layer_of, types, 1.9)
    base, _ = S1.allocate_bits(S, numel, layer_of, types, 2.9)
    # a common positive factor on the sensitivities changes every ratio by its square: same choice
    assert S1.allocate_bits(4.0 * S, numel, layer_of, types, 2.9)[0].tolist() == base.tolist()
    # relabelling the layers changes nothing
    assert S1.allocate_bits(S, numel, (layer_of + 1) % 4, types, 2.9)[0].tolist() == base.tolist()
    # a matrix with zero sensitivity is never upgraded while others can be
    S0 = S.copy()
    S0[5] = 0.0
    assert S1.allocate_bits(S0, numel, layer_of, types, 2.5)[0][5] == 2


def test_allocation_balances_layers_unlike_a_linear_sum():
    """Two layers, one of them ten times as sensitive: with the squared per-layer objective the budget goes to
    the sensitive layer first (the squared error of a layer falls fastest where the layer error is largest)."""
    S = np.array([10.0, 10.0, 1.0, 1.0])
    bits, steps = S1.allocate_bits(S, [8, 8, 8, 8], [0, 0, 1, 1], [2, 3, 4], 2.5)
    assert bits.tolist() == [3, 3, 2, 2]
    assert [s[0] for s in steps] == [0, 1]


def test_negative_sensitivity():
    """S < 0 (input redundancy outweighs task relevance, Eq. 5) in a layer of its own: more bits shrink
    |S| eta and so lower E^2 all the same - the rule is about E^2, not about the sign.  By hand: gains per
    upgrade are 1/256 - 1/4096 for the first matrix, 1/1024 - 1/16384 for the second, then 1/4096 - 1/65536
    for the first again: the order is matrix 0, matrix 1, and the budget of 3.0 is then used up."""
    bits, steps = S1.allocate_bits(np.array([-1.0, 0.5]), [4, 4], [0, 1], [2, 3, 4], 3.0)
    assert bits.tolist() == [3, 3] and [s[0] for s in steps] == [0, 1]
    assert steps[0][3] == pytest.approx((1 / 256 - 1 / 4096) / 4, rel=1e-15)
    # inside one layer a negative term offsets a positive one: E = (-1 + 1.5)/16 = 1/32; upgrading either
    # matrix alone moves E further from zero (-1/16 + 1.5/64 or -1/64 + 1.5/16), so no step lowers E^2
    bits, steps = S1.allocate_bits(np.array([-1.0, 1.5]), [4, 4], [0, 0], [2, 3, 4], 3.0)
    assert bits.tolist() == [2, 2] and steps == []
