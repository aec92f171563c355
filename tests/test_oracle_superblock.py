"""Pins for the oracle's super-block format (Section 3, "Weight quantization": S blocks share a scale and a zero point
that compress the per-block parameters).  Closed forms, invariants, a hand-derived record, a pure-Python brute force
and the cases in which the two-level format must coincide with the plain one.  No GPU."""
import struct

import numpy as np
import pytest

from oracle import aq_oracle as O
from paper_2605_24011_b200 import synth

BITS = (2, 3, 4)


def _f16(x):
    return float(np.float16(np.float32(x)))


@pytest.mark.parametrize("bits", BITS)
def test_sizes_and_ranges(bits):
    N, K = 12, 768
    W = synth.weights(N, K, 201, bits, outliers=True)
    D, Dm, Mn, u, v, q = O.quantize_sb(W, bits)
    assert D.shape == Dm.shape == Mn.shape == (N, K // 256) and u.shape == v.shape == (N, K // 32) and q.shape == (N, K)
    assert u.max() <= 63 and v.max() <= 63 and q.max() <= O.code_max(bits)
    buf = O.pack_sb(D, Dm, Mn, u, v, q, bits)
    assert buf.size == O.packed_nbytes_sb(N, K, bits) == N * K * (bits * 16 + 9) // 128
    assert buf.size * 8 / (N * K) == bits + 0.5625
    # the largest scale of a super-block takes (nearly) the largest code, the smallest minimum takes code 0
    uS, vS = u.reshape(N, -1, 8), v.reshape(N, -1, 8)
    assert np.all(uS.max(axis=2) >= 62) and np.all(vS.min(axis=2) == 0)


@pytest.mark.parametrize("bits", BITS)
def test_pack_unpack_roundtrip(bits):
    rng = np.random.default_rng(7 + bits)
    N, K = 5, 512
    q = rng.integers(0, O.code_max(bits) + 1, (N, K)).astype(np.uint8)
    u = rng.integers(0, 64, (N, K // 32)).astype(np.uint8)
    v = rng.integers(0, 64, (N, K // 32)).astype(np.uint8)
    D, Dm, Mn = (rng.normal(0, 1, (N, K // 256)).astype(np.float16) for _ in range(3))
    buf = O.pack_sb(D, Dm, Mn, u, v, q, bits)
    back = O.unpack_sb(buf, bits, N, K)
    for a, b in zip((D, Dm, Mn, u, v, q), back):
        assert np.array_equal(a.view(np.uint16) if a.dtype == np.float16 else a, b.view(np.uint16) if b.dtype == np.float16 else b)
    # every bit of the record is accounted for: flipping any bit changes the unpacked tuple
    for pos in rng.integers(0, buf.size * 8, 40):
        c = buf.copy(); c[pos // 8] ^= 1 << (pos % 8)
        other = O.unpack_sb(c, bits, N, K)
        assert any(not np.array_equal(np.asarray(a).view(np.uint8), np.asarray(b).view(np.uint8)) for a, b in zip(back, other))


def test_hand_derived_record():
    """One super-block, 2-bit, built so that everything is exact: block b holds the values {0, 1, 2, 3} * (b + 1) / 64
    + b / 8 (each 8 times).  Block scale s_b = (b + 1) / 64, block minimum b / 8.  D = f16(8/64 / 63) is not a power of two,
    so take the rule at its word: u_b = rint(s_b / D), decoded scale f16(D u_b)."""
    bits = 2
    W = np.zeros((1, 256), dtype=np.float32)
    for b in range(8):
        W[0, 32 * b:32 * b + 32] = np.tile(np.arange(4, dtype=np.float32), 8) * np.float32((b + 1) / 64) + np.float32(b / 8)
    D, Dm, Mn, u, v, q = O.quantize_sb(W, bits)
    Dv = np.float32(np.float16(np.float32(np.float32(0.125) / np.float32(63))))
    assert float(D[0, 0]) == float(Dv)
    assert u[0].tolist() == [int(np.rint(np.float32(np.float32((b + 1) / 64) / Dv))) for b in range(8)] == [8, 16, 24, 32, 39, 47, 55, 63]
    assert float(Mn[0, 0]) == 0.0 and float(Dm[0, 0]) == _f16(np.float32(0.875) / np.float32(63))
    assert v[0].tolist() == [0, 9, 18, 27, 36, 45, 54, 63]
    # bytes: three binary16 little-endian, then the 12-bit (u | v << 6) stream, then the codes
    buf = O.pack_sb(D, Dm, Mn, u, v, q, bits)
    assert bytes(buf[0:6]) == struct.pack("<eee", float(D[0, 0]), float(Dm[0, 0]), 0.0)
    stream = 0
    for b in range(8):
        stream |= (int(u[0, b]) | (int(v[0, b]) << 6)) << (12 * b)
    assert bytes(buf[6:18]) == stream.to_bytes(12, "little")
    code_stream = 0
    for i in range(32):
        code_stream |= int(q[0, i]) << (2 * i)
    assert bytes(buf[18:26]) == code_stream.to_bytes(8, "little")
    assert buf.size == 18 + 64


@pytest.mark.parametrize("bits", BITS)
def test_brute_force_small(bits):
    """quantize_sb against a per-element pure-Python loop with explicit binary32 / binary16 roundings."""
    f32, f16 = np.float32, np.float16
    W = synth.weights(3, 256, 203, bits, outliers=True)
    D, Dm, Mn, u, v, q = O.quantize_sb(W, bits)
    L = f32(O.code_max(bits))
    for r in range(3):
        s, mn = [], []
        for b in range(8):
            blk = W[r, 32 * b:32 * b + 32]
            lo, hi = f32(min(blk)), f32(max(blk))
            s.append(f32(f32(hi - lo) / L)); mn.append(lo)
        Dr = f16(f32(max(s) / f32(63)))
        Mnr = f16(min(mn))
        Dmr = f16(f32(max(f32(max(mn) - f32(Mnr)), f32(0)) / f32(63)))
        assert Dr == D[r, 0] and Mnr == Mn[r, 0] and Dmr == Dm[r, 0]
        for b in range(8):
            ub = 0 if f32(Dr) == 0 else int(min(63, max(0, np.rint(f32(s[b] / f32(Dr))))))
            vb = 0 if f32(Dmr) == 0 else int(min(63, max(0, np.rint(f32(f32(mn[b] - f32(Mnr)) / f32(Dmr))))))
            assert ub == u[r, b] and vb == v[r, b]
            sc = f16(f32(f32(Dr) * f32(ub)))
            mi = f16(f32(np.float64(f32(Dmr)) * vb + np.float64(f32(Mnr))))
            for i in range(32):
                w = W[r, 32 * b + i]
                code = 0 if f32(sc) == 0 else int(min(L, max(0, np.rint(f32(f32(w - f32(mi)) / f32(sc))))))
                assert code == q[r, 32 * b + i]


@pytest.mark.parametrize("bits", BITS)
def test_error_within_the_two_level_bound(bits):
    """|w - w_hat| <= scale/2 + |min - block min| + L |scale - exact block scale|: half a step of the decoded grid, plus
    what coding the block's minimum and scale moved the grid's ends."""
    W = synth.weights(48, 1024, 205, bits, outliers=True)
    D, Dm, Mn, u, v, q = O.quantize_sb(W, bits)
    d, m = O.sb_block_params(D, Dm, Mn, u, v)
    L = O.code_max(bits)
    Wb = W.astype(np.float64).reshape(48, -1, 32)
    what = O.dequant_f64(d, m, q).reshape(48, -1, 32)
    mn, mx = Wb.min(axis=2), Wb.max(axis=2)
    d64, m64 = d.astype(np.float64), m.astype(np.float64)
    bound = d64 / 2 + np.abs(mn - m64) + L * np.abs((mx - mn) / L - d64)
    assert np.all(np.abs(Wb - what) <= bound[..., None] * (1 + 1e-6) + 1e-12)
    # and the extra error over the plain format is small on such data: the coded parameters are close to the plain ones
    d0, m0, q0 = O.quantize(W, bits)
    e_sb, e_plain = np.abs(Wb - what).mean(), np.abs(W.astype(np.float64) - O.dequant_f64(d0, m0, q0)).mean()
    assert e_sb <= 1.25 * e_plain


@pytest.mark.parametrize("bits", BITS)
def test_coincides_with_the_plain_format_when_the_parameters_are_on_the_grid(bits):
    """Blocks whose scales are D * integer and whose minima are Mn + Dm * integer exactly (binary16-exact values): the
    codes u, v reproduce them, so codes and decoded weights equal the plain quantiser's."""
    rng = np.random.default_rng(11)
    L = O.code_max(bits)
    W = np.zeros((4, 512), dtype=np.float32)
    for r in range(4):
        for S in range(2):
            ub = rng.permutation(np.arange(1, 64))[:8]; ub[0] = 63
            vb = rng.permutation(np.arange(0, 64))[:8]; vb[1] = 0; vb[2] = 63
            for b in range(8):
                sc, mi = 2.0 ** -10 * ub[b], -0.25 + 2.0 ** -9 * vb[b]
                codes = rng.integers(0, L + 1, 32); codes[0], codes[1] = 0, L
                W[r, 256 * S + 32 * b:256 * S + 32 * b + 32] = (sc * codes + mi).astype(np.float32)
    D, Dm, Mn, u, v, q = O.quantize_sb(W, bits)
    d, m = O.sb_block_params(D, Dm, Mn, u, v)
    d0, m0, q0 = O.quantize(W, bits)
    assert np.array_equal(d, d0) and np.array_equal(m, m0) and np.array_equal(q, q0)
    assert np.array_equal(O.dequant_f32(d, m, q), W)


def test_degenerate_super_blocks():
    W = np.zeros((2, 256), dtype=np.float32)
    W[1, :] = 0.37                                           # constant: every scale 0, one minimum
    D, Dm, Mn, u, v, q = O.quantize_sb(W, 3)
    assert np.all(u == 0) and np.all(v == 0) and np.all(q == 0) and np.all(D == 0) and np.all(Dm == 0)
    d, m = O.sb_block_params(D, Dm, Mn, u, v)
    assert np.all(O.dequant_f32(d, m, q)[0] == 0) and np.all(O.dequant_f32(d, m, q)[1] == np.float32(np.float16(0.37)))
