"""Pins of the attention oracle (oracle/attn_oracle.py) against what the mathematics fixes: closed forms, invariants,
special cases and a pure-Python brute force.  Chosen so that a plausible mistake (a transposed operand, a wrong pairing
or sign in the rotation, a missing scale, a wrong key/value head for a query head, positions past L leaking in) fails
at least one of them."""
import math

import numpy as np

from oracle import attn_oracle as A


def _rng(seed):
    return np.random.default_rng(seed)


# ---- rotary embedding -------------------------------------------------------------------------------------------
def test_rope_closed_forms():
    # D = 2: one pair, angle = pos * theta^0 = pos
    x = np.array([[1.0, 0.0], [0.0, 2.0]])
    y = A.rope(x, 3)
    assert np.allclose(y[0], [math.cos(3), math.sin(3)], atol=1e-15)
    assert np.allclose(y[1], [-2 * math.sin(3), 2 * math.cos(3)], atol=1e-15)
    # D = 4, theta = 10000: pairs (0, 2) and (1, 3) with angles pos and pos / 100
    x = np.array([[1.0, 1.0, 0.0, 0.0]])
    y = A.rope(x, 7, 10000.0)
    assert np.allclose(y[0], [math.cos(7), math.cos(0.07), math.sin(7), math.sin(0.07)], atol=1e-15)
    # another base: second pair's angle is pos * theta^(-1/2)
    y = A.rope(x, 5, 4.0)
    assert np.allclose(y[0], [math.cos(5), math.cos(2.5), math.sin(5), math.sin(2.5)], atol=1e-15)


def test_rope_identity_norm_and_composition():
    g = _rng(1)
    x = g.standard_normal((3, 16))
    assert np.array_equal(A.rope(x, 0), x)
    for pos in (1, 17, 4095):
        y = A.rope(x, pos)
        # every pair keeps its length
        assert np.allclose(y[:, :8] ** 2 + y[:, 8:] ** 2, x[:, :8] ** 2 + x[:, 8:] ** 2, rtol=1e-12)
    assert np.allclose(A.rope(A.rope(x, 5), 11), A.rope(x, 16), atol=1e-12)


def test_rope_scores_depend_on_relative_position_only():
    g = _rng(2)
    q, k = g.standard_normal((1, 32)), g.standard_normal((1, 32))
    ref = float((A.rope(q, 9) @ A.rope(k, 0).T)[0, 0])
    for shift in (1, 100, 3000):
        assert abs(float((A.rope(q, 9 + shift) @ A.rope(k, shift).T)[0, 0]) - ref) < 1e-9
    # and it is not position-free: another distance gives another score
    assert abs(float((A.rope(q, 10) @ A.rope(k, 0).T)[0, 0]) - ref) > 1e-6


# ---- attention ---------------------------------------------------------------------------------------------------
def _brute(q, K, V, L, scale):
    H, D = len(q), len(q[0])
    G = H // len(K)
    out = []
    for h in range(H):
        kv = h // G
        s = [scale * sum(q[h][d] * K[kv][p][d] for d in range(D)) for p in range(L)]
        m = max(s)
        e = [math.exp(v - m) for v in s]
        z = sum(e)
        out.append([sum(e[p] * V[kv][p][d] for p in range(L)) / z for d in range(D)])
    return out


def test_attention_brute_force_tiny():
    g = _rng(3)
    for H, Hkv, D, Lmax, L in ((2, 2, 4, 5, 5), (4, 2, 6, 7, 3), (6, 1, 2, 9, 9), (1, 1, 8, 1, 1)):
        q = g.standard_normal((H, D))
        K = g.standard_normal((Hkv, Lmax, D))
        V = g.standard_normal((Hkv, Lmax, D))
        for scale in (None, 0.3):
            got = A.attn_decode(q, K, V, L, scale)
            ref = _brute(q.tolist(), K.tolist(), V.tolist(), L, 1.0 / math.sqrt(D) if scale is None else scale)
            assert np.allclose(got, np.array(ref), atol=1e-13)


def test_attention_special_cases():
    g = _rng(4)
    H, Hkv, D, Lmax = 4, 2, 8, 12
    q = g.standard_normal((H, D))
    K = g.standard_normal((Hkv, Lmax, D))
    V = g.standard_normal((Hkv, Lmax, D))
    # one position: the output is that position's value row, for the head's own key/value head
    o = A.attn_decode(q, K, V, 1)
    assert np.allclose(o[0], V[0, 0]) and np.allclose(o[1], V[0, 0]) and np.allclose(o[2], V[1, 0]) and np.allclose(o[3], V[1, 0])
    # zero query: uniform weights, the mean of the valid rows
    o = A.attn_decode(np.zeros((H, D)), K, V, 7)
    assert np.allclose(o[0], V[0, :7].mean(axis=0)) and np.allclose(o[3], V[1, :7].mean(axis=0))
    # a key that dominates: its value row comes out
    K2 = K.copy()
    K2[0, 4] = 50.0 * q[0] / np.linalg.norm(q[0])
    o = A.attn_decode(q, K2, V, 9, scale=1.0)
    assert np.allclose(o[0], V[0, 4], atol=1e-8)
    # the output is a convex combination of the value rows
    o = A.attn_decode(q, K, V, 10)
    for h in range(H):
        rows = V[h // 2, :10]
        assert np.all(o[h] <= rows.max(axis=0) + 1e-12) and np.all(o[h] >= rows.min(axis=0) - 1e-12)


def test_attention_invariances():
    g = _rng(5)
    H, Hkv, D, Lmax, L = 3, 3, 6, 10, 8
    q = g.standard_normal((H, D))
    K = g.standard_normal((Hkv, Lmax, D))
    V = g.standard_normal((Hkv, Lmax, D))
    ref = A.attn_decode(q, K, V, L)
    # positions past L never matter, whatever they hold
    K2, V2 = K.copy(), V.copy()
    K2[:, L:] = 1e30
    V2[:, L:] = np.nan
    assert np.array_equal(A.attn_decode(q, K2, V2, L), ref)
    # the order of the positions does not matter (keys and values permuted together)
    perm = g.permutation(L)
    K3, V3 = K.copy(), V.copy()
    K3[:, :L] = K[:, perm]
    V3[:, :L] = V[:, perm]
    assert np.allclose(A.attn_decode(q, K3, V3, L), ref, atol=1e-13)
    # adding to every key of a head a vector orthogonal to nothing in particular shifts all its scores by the same
    # amount (u . q): the weights do not change
    u = g.standard_normal(D)
    K4 = K.copy()
    K4[0, :L] += u
    assert np.allclose(A.attn_decode(q, K4, V, L)[0], ref[0], atol=1e-12)
    # scale is applied to the scores: doubling q with half the scale is the same thing
    assert np.allclose(A.attn_decode(2 * q, K, V, L, scale=0.5 / math.sqrt(D)), ref, atol=1e-13)
    # linear in V
    assert np.allclose(A.attn_decode(q, K, 3 * V, L), 3 * ref, atol=1e-13)


def test_attention_bound():
    g = _rng(6)
    q = g.standard_normal((4, 8))
    K = g.standard_normal((2, 6, 8))
    V = g.standard_normal((2, 6, 8))
    T = A.attn_bound(q, K, V, 6)
    assert np.all(T >= np.abs(A.attn_decode(q, K, V, 6)) - 1e-15)
    assert np.allclose(A.attn_bound(q, K, np.abs(V), 6), A.attn_decode(q, K, np.abs(V), 6))


def test_attention_of_several_new_tokens_is_causal():
    g = _rng(7)
    M, H, Hkv, D, Lmax, L = 3, 4, 2, 6, 12, 9
    q = g.standard_normal((M, H, D))
    K = g.standard_normal((Hkv, Lmax, D))
    V = g.standard_normal((Hkv, Lmax, D))
    out = A.attn_decode_tokens(q, K, V, L)
    assert out.shape == (M, H, D)
    # brute force: token m sees positions 0 .. L - M + m
    for m in range(M):
        ref = _brute(q[m].tolist(), K.tolist(), V.tolist(), L - (M - 1 - m), 1.0 / math.sqrt(D))
        assert np.allclose(out[m], np.array(ref), atol=1e-13)
    # the last token is the single-token case; the first one sees M - 1 positions fewer
    assert np.array_equal(out[M - 1], A.attn_decode(q[M - 1], K, V, L))
    assert np.array_equal(out[0], A.attn_decode(q[0], K, V, L - M + 1))
    # what comes after a token does not reach it: changing the last position changes the last token only
    K2, V2 = K.copy(), V.copy()
    K2[:, L - 1] += 1.0
    V2[:, L - 1] -= 2.0
    out2 = A.attn_decode_tokens(q, K2, V2, L)
    assert np.array_equal(out2[: M - 1], out[: M - 1]) and not np.allclose(out2[M - 1], out[M - 1])
    # one token: the plain function
    assert np.array_equal(A.attn_decode_tokens(q[:1], K, V, L)[0], A.attn_decode(q[0], K, V, L))
    T = A.attn_bound_tokens(q, K, V, L)
    assert T.shape == out.shape and np.all(T >= np.abs(out) - 1e-15)
