"""Pins for the CPU oracle: closed forms, invariants, hand-derived bytes and a
pure-Python brute force.  Each check is chosen so that a plausible slip in the
oracle (dropped term, wrong sign or index, transposed operand, wrong bit
order) fails at least one of them.  No GPU."""
import math
import os
import struct

import numpy as np
import pytest

import brute
from oracle import aq_oracle as O
from paper_2605_24011_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "block_records.txt")
BITS = (2, 3, 4)


def _golden_cases():
    cases = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, bits, wrule, hexrec, crule = [s.strip() for s in line.split(";")]
            w = [float(eval(wrule, {"i": i})) for i in range(32)]
            codes = [int(eval(crule, {"i": i})) for i in range(32)]
            cases.append((name, int(bits), w, bytes.fromhex(hexrec), codes))
    return cases


@pytest.mark.parametrize("case", _golden_cases(), ids=lambda c: c[0])
def test_golden_block_records(case):
    """Hand-derived records: quantise + pack reproduce the bytes; unpack +
    dequant give back codes and values."""
    name, bits, w, rec, codes = case
    W = np.array([w], dtype=np.float32)
    d, m, q = O.quantize(W, bits)
    assert q[0].tolist() == codes
    buf = O.pack(d, m, q, bits)
    assert bytes(buf) == rec
    d2, m2, q2 = O.unpack(np.frombuffer(rec, dtype=np.uint8), bits, 1, 32)
    assert q2[0].tolist() == codes
    w32 = O.dequant_f32(d2, m2, q2)[0]
    if name == "E":
        assert np.all(w32 == np.float32(np.float16(np.float32(0.3))))
    elif name != "D":
        assert w32.tolist() == [float(np.float32(v)) for v in w]   # grid-exact


@pytest.mark.parametrize("bits", BITS)
def test_closed_forms_sizes(bits):
    N, K = 24, 160
    W = synth.weights(N, K, 1, bits)
    d, m, q = O.quantize(W, bits)
    buf = O.pack(d, m, q, bits)
    assert buf.size == N * K * (bits + 1) // 8 == O.packed_nbytes(N, K, bits)
    assert buf.size * 8 / (N * K) == bits + 1          # bits per weight
    assert {2: 12, 3: 16, 4: 20}[bits] == 4 + 4 * bits  # bytes per block


def test_7b_stack_bytes_closed_form():
    """2.5-bit mean code width over the 7B-shaped stack stores 3.5 bits per
    weight: 6,476,005,376 weights -> 2,833,252,352 bytes."""
    layer = synth.llama7b_layer()
    w = 32 * sum(N * K for _, N, K in layer)
    assert w == 6_476_005_376
    assert w * 3.5 / 8 == 2_833_252_352
    assert O.packed_nbytes(4096, 4096, 4) == 10_485_760
    # loose sanity against the paper's memory table: fp16 14.3 GB at 3.0/16
    assert abs(14.3 * 3.0 / 16 - 2.7) < 0.05


@pytest.mark.parametrize("bits", BITS)
@pytest.mark.parametrize("outliers", (False, True))
def test_codes_in_range_and_roundtrip_bound(bits, outliers):
    """codes in [0, 2^b-1]; |w - w_hat| <= d/2 + |mn - m| + L |(mx-mn)/L - d|
    (the last two terms are the fp16 rounding of min and scale)."""
    W = synth.weights(64, 512, 2, bits, outliers=outliers)
    d, m, q = O.quantize(W, bits)
    L = O.code_max(bits)
    assert q.min() >= 0 and q.max() <= L
    What = O.dequant_f64(d, m, q).reshape(64, -1, 32)
    Wb = W.astype(np.float64).reshape(64, -1, 32)
    mn, mx = Wb.min(2), Wb.max(2)
    d64, m64 = d.astype(np.float64), m.astype(np.float64)
    # t is evaluated in binary32: allow its rounding (<= 2^-23 relative on (w-m))
    slack = np.abs(mn - m64) + L * np.abs((mx - mn) / L - d64) + 2.0 ** -22 * (np.abs(Wb).max(2) + np.abs(m64))
    bound = d64 / 2 + slack
    assert np.all(np.abs(Wb - What) <= bound[:, :, None])
    # each block with d > 0 uses both ends of the code range
    nz = d64 > 0
    qb = q.reshape(64, -1, 32)
    assert np.all(qb.min(2)[nz] == 0) and np.all(qb.max(2)[nz] == L)


@pytest.mark.parametrize("bits", BITS)
def test_brute_force_8x64(bits):
    """Per-element pure-Python loop on an 8x64 matrix: codes, scales, bytes,
    dequantised values and the linear all agree with the oracle."""
    N, K = 8, 64
    W = synth.weights(N, K, 3, bits, outliers=True)
    x = synth.activations(3, K, 3, bits).astype(np.float16)
    d, m, q = O.quantize(W, bits)
    buf = O.pack(d, m, q, bits)
    blocks, raw = brute.matrix([[float(v) for v in row] for row in W], bits)
    assert bytes(buf) == raw
    w32 = O.dequant_f32(d, m, q)
    w16 = O.dequant(d, m, q, "f16")
    wbf = O.dequant(d, m, q, "bf16")
    for n in range(N):
        for j, (bd, bm, codes) in enumerate(blocks[n]):
            assert float(d[n, j]) == bd and float(m[n, j]) == bm
            for i, c in enumerate(codes):
                k = 32 * j + i
                assert int(q[n, k]) == c
                v = brute.dequant_elem_f32(bd, bm, c)
                assert float(w32[n, k]) == v
                assert int(w16[n, k]) == struct.unpack("<H", struct.pack("<e", v))[0]
                # bf16 by hand: round the binary32 pattern to 16 bits, ties to even
                u = struct.unpack("<I", struct.pack("<f", v))[0]
                lower = u & 0xFFFF
                hi = u >> 16
                if lower > 0x8000 or (lower == 0x8000 and (hi & 1)):
                    hi += 1
                assert int(wbf[n, k]) == hi
    y, T = O.linear(d, m, q, x.astype(np.float64))
    for t in range(x.shape[0]):
        xs = [float(v) for v in x[t]]
        for n in range(N):
            yy, tt = brute.linear_row(blocks[n], xs)
            assert abs(y[t, n] - yy) <= 1e-12 * max(1.0, tt)
            assert abs(T[t, n] - tt) <= 1e-12 * max(1.0, tt)


@pytest.mark.parametrize("bits", BITS)
def test_grid_exact_blocks_roundtrip(bits):
    """Blocks built on an exactly representable grid m + d*q (d a power of
    two, codes touching 0 and L) come back with the same codes and values."""
    rng = np.random.default_rng(5)
    L = O.code_max(bits)
    N, nb = 16, 6
    q0 = rng.integers(0, L + 1, size=(N, nb, 32))
    q0[:, :, 0] = 0
    q0[:, :, 1] = L
    dd = 2.0 ** rng.integers(-8, -2, size=(N, nb, 1))
    mm = -dd * rng.integers(0, L + 1, size=(N, nb, 1))
    W = (mm + dd * q0).astype(np.float32).reshape(N, nb * 32)
    d, m, q = O.quantize(W, bits)
    assert np.array_equal(q.reshape(N, nb, 32), q0)
    assert np.array_equal(d.astype(np.float64), dd[:, :, 0])
    assert np.array_equal(O.dequant_f32(d, m, q), W)
    assert np.array_equal(O.dequant_f64(d, m, q), W.astype(np.float64))


@pytest.mark.parametrize("bits", BITS)
def test_ideal_quantiser_differs_only_at_near_ties(bits):
    W = synth.weights(128, 1024, 6, bits)
    d, m, q = O.quantize(W, bits)
    qs, frac = O.quantize_ideal(W, d, m, bits)
    diff = q != qs
    assert np.all(np.abs(frac[diff] - 0.5) < 1e-5)
    assert diff.mean() < 1e-4


@pytest.mark.parametrize("bits", BITS)
def test_pack_unpack_identity_and_bit_order(bits):
    rng = np.random.default_rng(7)
    N, K = 5, 96
    L = O.code_max(bits)
    q = rng.integers(0, L + 1, size=(N, K)).astype(np.uint8)
    d = rng.standard_normal((N, K // 32)).astype(np.float16)
    m = rng.standard_normal((N, K // 32)).astype(np.float16)
    buf = O.pack(d, m, q, bits)
    d2, m2, q2 = O.unpack(buf, bits, N, K)
    assert np.array_equal(q, q2)
    assert np.array_equal(d.view(np.uint16), d2.view(np.uint16))
    assert np.array_equal(m.view(np.uint16), m2.view(np.uint16))
    rec = buf.reshape(N, K // 32, 4 + 4 * bits)
    # scale/min little-endian fp16 at bytes 0..3
    assert struct.unpack("<e", bytes(rec[2, 1, 0:2]))[0] == float(d[2, 1])
    assert struct.unpack("<e", bytes(rec[2, 1, 2:4]))[0] == float(m[2, 1])
    codes = q.reshape(N, K // 32, 32)[2, 1]
    body = rec[2, 1, 4:]
    if bits == 4:
        assert all(int(body[p]) == int(codes[2 * p]) | int(codes[2 * p + 1]) << 4 for p in range(16))
    if bits == 2:
        assert all(int(body[p]) == sum(int(codes[4 * p + s]) << (2 * s) for s in range(4)) for p in range(8))
    big = sum(int(c) << (bits * i) for i, c in enumerate(codes))
    assert bytes(body) == big.to_bytes(4 * bits, "little")


@pytest.mark.parametrize("bits", BITS)
def test_dequant_matches_exact_value_rounded_once(bits):
    """f32(d)*f32(q) is exact, so the fp32 result equals the exact value
    rounded once to binary32; fp16 output is that value rounded once more."""
    W = synth.weights(32, 256, 8, bits, outliers=True)
    d, m, q = O.quantize(W, bits)
    exact = O.dequant_f64(d, m, q)
    w32 = O.dequant_f32(d, m, q)
    assert np.array_equal(w32, exact.astype(np.float32))
    assert np.array_equal(O.dequant(d, m, q, "f16"), exact.astype(np.float32).astype(np.float16).view(np.uint16))
    # bf16 bits decode to a neighbour of the fp32 value within half a bf16 ulp
    bf = O.bf16_bits_to_f64(O.dequant(d, m, q, "bf16"))
    assert np.all(np.abs(bf - w32) <= 2.0 ** -8 * np.abs(w32) + 1e-40)
    # constant block -> value f16(min) everywhere
    Wc = np.full((1, 32), 0.3, dtype=np.float32)
    dc, mc, qc = O.quantize(Wc, bits)
    assert float(dc[0, 0]) == 0.0 and not qc.any()
    assert np.all(O.dequant_f32(dc, mc, qc) == np.float32(np.float16(np.float32(0.3))))


def test_bf16_rounding_special_values():
    x = np.array([1.0, 1.00390625, 1.01171875, -1.00390625, 3.3895314e38, 0.0], dtype=np.float32)
    # 1 + 2^-8 is a tie -> even (1.0); 1 + 3*2^-8 is a tie -> 1 + 2^-6 (even mantissa)
    b = O.f32_to_bf16_bits(x)
    assert b.tolist()[:4] == [0x3F80, 0x3F80, 0x3F82, 0xBF80]
    assert b[5] == 0
    assert O.bf16_bits_to_f64(np.array([0x3F80, 0xC000], dtype=np.uint16)).tolist() == [1.0, -2.0]


@pytest.mark.parametrize("bits", BITS)
def test_linear_structure(bits):
    """unit vector -> a column of w_hat; ones -> row sums; 2x -> 2y exactly;
    a row permutation of W permutes y; row t of a batch equals the single-row
    call; T dominates |y|."""
    N, K = 48, 320
    W = synth.weights(N, K, 9, bits)
    d, m, q = O.quantize(W, bits)
    What = O.dequant_f64(d, m, q)
    for k in (0, 31, 32, 319):
        e = np.zeros((1, K)); e[0, k] = 1.0
        y, T = O.linear(d, m, q, e)
        assert np.array_equal(y[0], What[:, k]) and np.array_equal(T[0], np.abs(What[:, k]))
    y1, _ = O.linear(d, m, q, np.ones((1, K)))
    assert np.allclose(y1[0], [math.fsum(r) for r in What], rtol=0, atol=1e-12)
    x = synth.activations(8, K, 9, bits).astype(np.float16).astype(np.float64)
    y, T = O.linear(d, m, q, x)
    y2, _ = O.linear(d, m, q, 2 * x)
    assert np.array_equal(y2, 2 * y)
    assert y.shape == (8, N) and np.all(T >= np.abs(y) - 1e-12)
    perm = np.random.default_rng(1).permutation(N)
    dp, mp, qp = O.quantize(W[perm], bits)
    yp, _ = O.linear(dp, mp, qp, x)
    assert np.allclose(yp, y[:, perm], rtol=0, atol=1e-12)
    for t in (0, 7):
        yt, _ = O.linear(d, m, q, x[t:t + 1])
        assert np.allclose(yt[0], y[t], rtol=0, atol=1e-12)
    # not transposed: y[t][n] pairs x row t with W row n
    assert abs(y[3, 5] - math.fsum(x[3] * What[5])) < 1e-12
    assert np.all(O.linear_excess(y, y, T) == 0)


def test_silu_and_rms():
    g = np.linspace(-20, 20, 4001)
    eg = np.exp(-np.abs(g))                              # x * logistic(x), overflow-free form
    ref = g * np.where(g >= 0, 1.0 / (1.0 + eg), eg / (1.0 + eg))
    assert np.allclose(O.silu(g), ref, rtol=1e-13, atol=1e-15)
    assert O.silu(np.array([0.0]))[0] == 0.0
    assert abs(O.silu(np.array([1.0]))[0] - 1.0 / (1.0 + math.exp(-1.0))) < 1e-15
    assert np.allclose(O.silu_mul(g, 3.0), 3.0 * ref, rtol=1e-13, atol=1e-15)
    h = np.array([[3.0, 4.0, 0.0, 0.0]])
    assert abs(O.rms_scale(h, eps=0.0)[0, 0] - 1.0 / 2.5) < 1e-15


def test_draw_bits_hits_mean():
    sizes = [N * K for (_, _, N, K) in synth.stack_shapes(synth.llama7b_layer(), 32)]
    bits = synth.draw_bits(sizes, 2.5, 0)
    mean = sum(b * s for b, s in zip(bits, sizes)) / sum(sizes)
    assert abs(mean - 2.5) <= 0.005 and set(bits) <= {2, 3, 4}
    sizes = [N * K for (_, _, N, K) in synth.stack_shapes(synth.gemma2b_layer(), 18)]
    bits = synth.draw_bits(sizes, 3.0, 1)
    mean = sum(b * s for b, s in zip(bits, sizes)) / sum(sizes)
    assert abs(mean - 3.0) <= 0.005
    assert sum(sizes) == 1_981_808_640
    assert 18 * sum(N * K for _, N, K in synth.expert_layer()) == 311_427_072
