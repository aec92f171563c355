"""Property-based pins of the oracle (hypothesis): statements that hold for every input, checked on drawn inputs
that include the awkward ones (constant blocks, huge and tiny magnitudes, mixed signs).  Independent of the
example-based pins in test_oracle_pins.py; nothing here calls the CUDA path."""
import numpy as np
import pytest

hypothesis = pytest.importorskip("hypothesis")
from hypothesis import given, settings, strategies as st   # noqa: E402
from hypothesis.extra import numpy as hnp                   # noqa: E402

from oracle import aq_oracle as O        # noqa: E402
from oracle import stage1_oracle as S1   # noqa: E402

BITS = st.sampled_from((2, 3, 4))
finite32 = st.floats(min_value=-6.0e4, max_value=6.0e4, allow_nan=False, allow_infinity=False, width=32)


def weights(rows=st.integers(1, 5), blocks=st.integers(1, 3)):
    return st.tuples(rows, blocks).flatmap(lambda rb: hnp.arrays(np.float32, (rb[0], 32 * rb[1]), elements=finite32))


@settings(max_examples=60, deadline=None)
@given(W=weights(), bits=BITS)
def test_quantiser_invariants(W, bits):
    d, m, q = O.quantize(W, bits)
    L = O.code_max(bits)
    N, K = W.shape
    assert q.shape == (N, K) and q.min() >= 0 and q.max() <= L
    Wb = W.reshape(N, K // 32, 32).astype(np.float64)
    d64, m64 = d.astype(np.float64), m.astype(np.float64)
    mn, mx = Wb.min(axis=2), Wb.max(axis=2)
    # the stored minimum is the block minimum rounded to binary16; the scale is the rounded (max - min) / L
    assert np.array_equal(m, mn.astype(np.float32).astype(np.float16))
    finite = np.isfinite(d64) & np.isfinite(m64)
    what = O.dequant_f64(d, m, q).reshape(N, K // 32, 32)
    # reconstruction error: half a step plus what the rounding of min and scale to binary16 moved the grid
    slack = np.abs(mn - m64) + L * np.abs((mx.astype(np.float32) - mn.astype(np.float32)).astype(np.float64) / L - d64)
    bound = (d64 / 2 + slack)[..., None] * (1 + 1e-6) + 1e-30
    ok = finite[..., None] & np.isfinite(what)
    assert np.all(np.abs(Wb - what)[ok] <= np.broadcast_to(bound, what.shape)[ok])
    # scale zero <=> every code of the block is zero is implied one way: scale 0 gives codes 0
    zero = (d64 == 0)
    assert np.all(q.reshape(N, K // 32, 32)[zero] == 0)
    # the extreme elements of a block with a usable scale take the extreme codes (up to one step of rounding), as long
    # as rounding min and scale to binary16 moved the grid by less than half a step (a block like 59985 .. 59986, whose
    # minimum rounds to a multiple of 32, lands wholly on one end of the grid: covered by the error bound above)
    usable = finite & (d64 > 0) & (slack <= d64 / 2)
    qb = q.reshape(N, K // 32, 32)
    assert np.all(qb.min(axis=2)[usable] <= 1)
    assert np.all(qb.max(axis=2)[usable] >= L - 1)


@settings(max_examples=60, deadline=None)
@given(bits=BITS, data=st.data())
def test_container_roundtrip_and_size(bits, data):
    N = data.draw(st.integers(1, 6))
    nb = data.draw(st.integers(1, 4))
    K = 32 * nb
    q = data.draw(hnp.arrays(np.uint8, (N, K), elements=st.integers(0, O.code_max(bits))))
    d = data.draw(hnp.arrays(np.float16, (N, nb), elements=st.floats(-100, 100, width=16)))
    m = data.draw(hnp.arrays(np.float16, (N, nb), elements=st.floats(-100, 100, width=16)))
    buf = O.pack(d, m, q, bits)
    assert buf.dtype == np.uint8 and buf.size == O.packed_nbytes(N, K, bits) == N * K * (bits + 1) // 8
    d2, m2, q2 = O.unpack(buf, bits, N, K)
    assert np.array_equal(d2.view(np.uint16), d.view(np.uint16)) and np.array_equal(m2.view(np.uint16), m.view(np.uint16))
    assert np.array_equal(q2, q)
    # changing one code changes only the bytes of its own block record
    i, k = data.draw(st.integers(0, N - 1)), data.draw(st.integers(0, K - 1))
    q3 = q.copy()
    q3[i, k] = (int(q3[i, k]) + 1) % (O.code_max(bits) + 1)
    diff = np.nonzero(O.pack(d, m, q3, bits) != buf)[0]
    rec = 4 + 4 * bits
    blk = i * nb + k // 32
    assert diff.size >= 1 and np.all((diff >= blk * rec + 4) & (diff < (blk + 1) * rec))


@settings(max_examples=40, deadline=None)
@given(W=weights(rows=st.integers(1, 4), blocks=st.integers(1, 2)), bits=BITS, data=st.data())
def test_linear_is_linear_and_bounded(W, bits, data):
    d, m, q = O.quantize(np.clip(W, -100, 100), bits)
    K = W.shape[1]
    x = data.draw(hnp.arrays(np.float64, (2, K), elements=st.floats(-8, 8, width=16)))
    y, T = O.linear(d, m, q, x)
    what = O.dequant_f64(d, m, q)
    assert np.all(np.abs(y) <= T * (1 + 1e-12) + 1e-300)
    assert np.allclose(T, np.abs(x) @ np.abs(what).T, rtol=1e-12, atol=0)
    y2, _ = O.linear(d, m, q, 2.0 * x)
    assert np.array_equal(y2, 2.0 * y)
    ys, _ = O.linear(d, m, q, x[:1] + x[1:])
    assert np.allclose(ys, y[:1] + y[1:], rtol=1e-9, atol=1e-9 * (T.sum() + 1))


@settings(max_examples=40, deadline=None)
@given(data=st.data())
def test_hsic_properties(data):
    K = data.draw(st.integers(2, 12))
    A = data.draw(hnp.arrays(np.float64, (K, 3), elements=st.floats(-3, 3)))
    B = data.draw(hnp.arrays(np.float64, (K, 2), elements=st.floats(-3, 3)))
    KA, KB = S1.rbf_gram(A, 1.5), S1.rbf_gram(B, 0.8)
    h = S1.hsic(KA, KB)
    assert h >= -1e-12
    assert S1.hsic(KB, KA) == pytest.approx(h, rel=1e-9, abs=1e-14)
    assert S1.hsic_large(KA, KB) == pytest.approx(h, rel=1e-9, abs=1e-14)
    # Cauchy-Schwarz for the centred kernel matrices: HSIC(A,B)^2 <= HSIC(A,A) HSIC(B,B)
    assert h * h <= S1.hsic(KA, KA) * S1.hsic(KB, KB) * (1 + 1e-9) + 1e-24


@settings(max_examples=40, deadline=None)
@given(data=st.data())
def test_allocation_properties(data):
    n = data.draw(st.integers(1, 10))
    S = np.array(data.draw(st.lists(st.floats(-2, 2), min_size=n, max_size=n)))
    numel = data.draw(st.lists(st.sampled_from((32, 64, 96, 4096)), min_size=n, max_size=n))
    layer_of = data.draw(st.lists(st.integers(0, 3), min_size=n, max_size=n))
    budget = data.draw(st.floats(2.0, 4.0))
    bits, steps = S1.allocate_bits(S, numel, layer_of, [2, 3, 4], budget)
    assert S1.mean_bits(bits, numel) <= budget + 1e-12
    # the objective never rises along the greedy path, and every step has a positive gain per bit
    cur = [2] * n
    obj = S1.objective(S, cur, layer_of)
    for (j, b0, b1, ratio) in steps:
        assert cur[j] == b0 and ratio > 0
        cur[j] = b1
        nxt = S1.objective(S, cur, layer_of)
        assert nxt < obj + 1e-18
        obj = nxt
    assert cur == bits.tolist()
