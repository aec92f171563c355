"""Pins for the oracle's intra-tensor scale optimisation (Section 3.3, Eq. 10 and Eq. 11)."""
import struct

import numpy as np
import pytest

from oracle import aq_oracle as O
from paper_2605_24011_b200 import synth


def _f32(x):
    return struct.unpack("<f", struct.pack("<f", x))[0]


@pytest.mark.parametrize("bits", (2, 3, 4))
def test_alternation_never_raises_phi(bits):
    """Eq. 11: each half step (nearest codes; closed-form parameters) minimises Phi_b over its own variable."""
    W = synth.weights(32, 256, 70, bits, outliers=True)
    F = np.abs(synth.weights(32, 256, 71, bits)).astype(np.float32) + 1e-3
    for Fm in (None, F):
        s, m, q, trace = O.scale_opt_ideal(W, bits, Fm, rounds=5)
        for a, b in zip(trace, trace[1:]):
            assert np.all(b <= a * (1 + 1e-12) + 1e-300)
        assert np.all(trace[-1] <= trace[0])


def test_least_squares_step_is_the_weighted_regression():
    """For fixed codes the parameter step is weighted least squares of w on (q, 1): numpy's solver agrees."""
    rng = np.random.default_rng(3)
    w = rng.normal(0, 0.02, 32)
    q = rng.integers(0, 8, 32).astype(np.float64)
    om = rng.uniform(0.1, 2.0, 32)
    S0, S1, S2, Sw, Swq = om.sum(), (om * q).sum(), (om * q * q).sum(), (om * w).sum(), (om * w * q).sum()
    det = S0 * S2 - S1 * S1
    s = (S0 * Swq - S1 * Sw) / det
    m = (Sw - s * S1) / S0
    A = np.stack([q, np.ones(32)], axis=1) * np.sqrt(om)[:, None]
    sol, *_ = np.linalg.lstsq(A, w * np.sqrt(om), rcond=None)
    assert np.allclose([s, m], sol, rtol=1e-10, atol=1e-14)


@pytest.mark.parametrize("bits", (2, 3, 4))
def test_code_step_is_the_per_element_argmin(bits):
    """For fixed (scale, min) the code of each element is the codebook entry nearest to it, whatever its weight."""
    W = synth.weights(4, 64, 72, bits)
    s, m, q, _ = O.scale_opt_ideal(W, bits, None, rounds=1)          # q was chosen for the RTN parameters
    Wb = W.astype(np.float64).reshape(4, 2, 32)
    mn, mx = Wb.min(axis=2), Wb.max(axis=2)
    s0 = (mx - mn) / O.code_max(bits)
    codes = np.arange(O.code_max(bits) + 1)
    err = np.abs(Wb[..., None] - (s0[:, :, None, None] * codes + mn[:, :, None, None]))
    assert np.array_equal(err.argmin(axis=3).reshape(4, 64), q)


@pytest.mark.parametrize("bits", (2, 3, 4))
def test_optimised_blocks_are_never_worse_than_round_to_nearest(bits):
    W = synth.weights(64, 512, 73, bits, outliers=True)
    F = (np.abs(synth.weights(64, 512, 74, bits)) * 50 + 0.01).astype(np.float32)
    for Fm in (None, F):
        d0, m0, q0 = O.quantize(W, bits)
        d1, m1, q1 = O.quantize_opt(W, bits, Fm)
        assert q1.max() <= O.code_max(bits)
        p0 = O.block_phi(W, d0, m0, q0, Fm)
        p1 = O.block_phi(W, d1, m1, q1, Fm)
        assert np.all(p1 <= p0 * (1 + 1e-4) + 1e-30)          # (the choice is made on binary32 sums)
        assert p1.sum() < 0.9 * p0.sum()                       # and it does help on such data


def test_blocks_on_the_grid_and_constant_blocks_keep_their_round_to_nearest_form():
    rng = np.random.default_rng(5)
    q = rng.integers(0, 16, (8, 64)).astype(np.float32)
    q[:, 0], q[:, 1], q[:, 32], q[:, 33] = 0, 15, 0, 15
    W = (np.float32(-0.375) + np.float32(0.03125) * q).astype(np.float32)
    W[3, :32] = np.float32(0.125)                              # a constant block
    a, b = O.quantize(W, 4), O.quantize_opt(W, 4)
    assert all(np.array_equal(x, y) for x, y in zip(a, b))
    assert np.all(b[0][3, 0] == 0) and np.all(b[2][3, :32] == 0)


def test_fisher_scores_enter_as_weights_only():
    W = synth.weights(16, 128, 75, 3, outliers=True)
    ones = np.ones_like(W)
    a = O.quantize_opt(W, 3, None)
    assert all(np.array_equal(x, y) for x, y in zip(a, O.quantize_opt(W, 3, ones)))
    assert all(np.array_equal(x, y) for x, y in zip(a, O.quantize_opt(W, 3, ones * np.float32(8))))   # exact rescaling
    F = ones.copy(); F[:, ::2] = 100.0                        # make the even elements matter: their error must shrink
    d0, m0, q0 = a
    d1, m1, q1 = O.quantize_opt(W, 3, F)
    def err_even(d, m, q):
        what = d.astype(np.float64).repeat(32, axis=1) * q + m.astype(np.float64).repeat(32, axis=1)
        return ((W - what)[:, ::2] ** 2).sum()
    assert err_even(d1, m1, q1) < err_even(d0, m0, q0)


def test_sum32_order():
    """The stated summation order, replayed with explicit binary32 rounding in pure Python."""
    rng = np.random.default_rng(9)
    x = (rng.normal(0, 1, 32) * 10.0 ** rng.integers(-6, 6, 32)).astype(np.float32)
    g = []
    for k in range(4):
        a = float(x[8 * k])
        for i in range(1, 8):
            a = _f32(a + float(x[8 * k + i]))
        g.append(a)
    want = _f32(_f32(g[0] + g[1]) + _f32(g[2] + g[3]))
    assert float(O._sum32(x[None, :])[0]) == want


def _opt_vs_plain(bits, Fm, seed):
    """quantize_opt (binary32, fixed summation order) beside the plain float64 statement of Eq. 10-11."""
    W = synth.weights(64, 512, seed, bits, outliers=True)
    d, m, q = O.quantize_opt(W, bits, Fm, rounds=4)
    d0, m0, q0 = O.quantize(W, bits)
    s, mi, _, _ = O.scale_opt_ideal(W, bits, Fm, rounds=4)
    dI, mI = s.astype(np.float16), mi.astype(np.float16)             # the plain result in the container's precision
    qI, _ = O.quantize_ideal(W, dI, mI, bits)                        # ... and its nearest codes, in float64
    return W, (d, m, q), (d0, m0, q0), (dI, mI, qI)


@pytest.mark.parametrize("bits", (2, 3, 4))
@pytest.mark.parametrize("fisher", (False, True))
def test_quantize_opt_lands_on_the_plain_alternation(bits, fisher):
    """Wherever quantize_opt leaves the round-to-nearest form, its (scale, min) are the float64 alternation's
    (Eq. 11, `scale_opt_ideal`) rounded to binary16 -- except in the few blocks where a binary32 quotient and its
    float64 twin fall on different sides of a rounding boundary in some round and the two runs part."""
    Fm = (np.abs(synth.weights(64, 512, 174, bits)) * 50 + 0.01).astype(np.float32) if fisher else None
    W, (d, m, q), (d0, m0, q0), (dI, mI, qI) = _opt_vs_plain(bits, Fm, 173)
    switched = (d != d0) | (m != m0)
    assert switched.mean() > 0.9                                     # on such data nearly every block gains
    same = (d == dI) & (m == mI)
    assert same[switched].mean() >= 0.99
    # blocks that took the plain parameters also took the plain codes, except at exact near-ties of the quotient
    blk = np.repeat(switched & same, 32, axis=1)
    assert (q[blk] != qI[blk]).mean() < 1e-3


@pytest.mark.parametrize("bits", (2, 3, 4))
@pytest.mark.parametrize("fisher", (False, True))
def test_quantize_opt_is_as_good_as_the_better_plain_candidate(bits, fisher):
    """Per block, Phi_b (Eq. 10, float64) of quantize_opt's output is no worse than the better of round-to-nearest
    and the float64 alternation rounded to binary16 (which is what its final selection claims to pick)."""
    Fm = (np.abs(synth.weights(64, 512, 176, bits)) * 50 + 0.01).astype(np.float32) if fisher else None
    W, (d, m, q), (d0, m0, q0), (dI, mI, qI) = _opt_vs_plain(bits, Fm, 175)
    phi = O.block_phi(W, d, m, q, Fm)
    best = np.minimum(O.block_phi(W, d0, m0, q0, Fm), O.block_phi(W, dI, mI, qI, Fm))
    assert np.all(phi <= best * (1 + 1e-3) + 1e-30)
    assert abs(phi.sum() / best.sum() - 1) < 1e-4
