"""Edge cases of the CUDA path against the oracle: the smallest and the most lopsided shapes, degenerate blocks
(constant, one outlier, scales that round to zero or sit in the binary16 subnormals), activations at the ends of the
binary16 / bfloat16 range, and zeros of both signs.

Tolerance: |y - y_oracle| <= 2e-3 T + 1e-5 with T = sum_k |x_k w_hat_k| on every path and for both activation
types (the tensor-core path rounds a dequantised weight to binary16, 2^-11, and widens bfloat16 activations to
binary16 exactly; a bfloat16 row outside binary16's range travels scaled by a power of two)."""
import numpy as np
import pytest

from oracle import aq_oracle as O

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

BITS = (2, 3, 4)


@pytest.fixture(scope="module")
def aq():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2605_24011_b200 import aq as mod
    return mod


def _check_all(aq, W, bits, xs, allow_range=False):
    """pack -> export bytes, dequant bits, and linear for every (x, dtype) in xs."""
    N, K = W.shape
    h = aq.aq_pack(bits, 32, torch.from_numpy(W).cuda())
    d, m, q = O.quantize(W, bits)
    assert np.array_equal(aq.aq_export(h, allow_range_error=allow_range), O.pack(d, m, q, bits))
    for name, tdt in (("f16", torch.float16), ("bf16", torch.bfloat16)):
        out = torch.empty((N, K), dtype=tdt, device="cuda")
        aq.aq_dequant(h, out)
        assert np.array_equal(out.view(torch.int16).cpu().numpy().view(np.uint16), O.dequant(d, m, q, name))
    for x32, tdt in xs:
        xt = torch.from_numpy(x32).to(tdt)
        M = xt.shape[0]
        y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        aq.aq_linear(h, xt.cuda(), y)
        aq.aq_check()
        yo, T = O.linear(d, m, q, xt.to(torch.float64).numpy())
        got = y.double().cpu().numpy()
        assert np.all(np.isfinite(got))
        ex = O.linear_excess(got, yo, T)
        assert ex.max() <= 1.0, f"M={M} {tdt}: normalised error {ex.max():.3f}"
    h.free()


@pytest.mark.parametrize("bits", BITS)
@pytest.mark.parametrize("shape", ((1, 32), (1, 4096), (17, 32), (3, 288), (70000, 32), (16, 65536)))
def test_extreme_shapes(aq, bits, shape):
    N, K = shape
    g = np.random.default_rng(N * 7 + K)
    W = (g.standard_normal((N, K)) * 0.02).astype(np.float32)
    xs = [(g.standard_normal((M, K)).astype(np.float32), dt) for M, dt in ((1, torch.float16), (5, torch.float16), (8, torch.bfloat16), (33, torch.bfloat16), (200, torch.float16))]
    if N * K > 2_000_000:
        xs = xs[:3] + [(g.standard_normal((130, K)).astype(np.float32), torch.bfloat16)]
    _check_all(aq, W, bits, xs)


@pytest.mark.parametrize("bits", BITS)
def test_degenerate_blocks(aq, bits):
    g = np.random.default_rng(70 + bits)
    N, K = 48, 256
    W = (g.standard_normal((N, K)) * 0.02).astype(np.float32)
    W[0, :32] = 0.0                       # all-zero block
    W[1, :32] = 0.37                      # constant block: scale 0, every code 0
    W[2, 32:64] = -1e-3                   # constant negative
    W[3, :32] = 0.0; W[3, 5] = 3.0        # one outlier in a zero block
    W[4, :32] = np.linspace(-1.0, 1.0, 32)                 # exactly spans the grid
    W[5, :32] = 1e-7 * g.standard_normal(32)               # scale in the binary16 subnormals
    W[6, :32] = 1e-9 * g.standard_normal(32)               # scale rounds to zero in binary16
    W[7, :32] = 1000.0 + g.standard_normal(32)             # large minimum, small spread
    W[8, :32] = np.where(np.arange(32) % 2 == 0, 60000.0, -60000.0)   # scale near the top of the codebook range
    W[9, :32] = -np.abs(W[9, :32])        # one sign only
    W[10] = 0.0                           # a whole zero row
    xs = [(g.standard_normal((M, K)).astype(np.float32), dt) for M, dt in ((1, torch.float16), (8, torch.float16), (4, torch.bfloat16), (64, torch.bfloat16))]
    _check_all(aq, W, bits, xs)


@pytest.mark.parametrize("bits", BITS)
def test_activation_extremes(aq, bits):
    """Huge, tiny (subnormal) and zero activations: the one-token path multiplies codes held as binary16 subnormals, so
    products as small as 2^-24 * 2^-24 must survive in the float32 accumulators."""
    g = np.random.default_rng(80 + bits)
    N, K = 64, 512
    W = (g.standard_normal((N, K)) * 0.02).astype(np.float32)
    base = g.standard_normal((8, K)).astype(np.float32)
    big16 = base * 20000.0                                  # |x| up to the top of binary16
    tiny16 = base * 2.0**-20                                # binary16 subnormals
    mixed = base.copy(); mixed[:, ::3] = 0.0; mixed[:, 1::7] = -0.0; mixed[:, 5::11] *= 3.0e4; mixed[:, 2::13] *= 1e-6
    onehot = np.zeros((8, K), dtype=np.float32); onehot[np.arange(8), [0, 31, 32, 255, 256, 300, 510, 511]] = [1, -1, 65504, 6e-8, -2.0, 0.5, 1e-3, 7]
    big_bf = base * 1e30                                    # bfloat16 has the float32 exponent range
    tiny_bf = base * 1e-30
    xs = []
    for x in (big16, tiny16, mixed, onehot):
        xs += [(np.clip(x, -65504, 65504)[:1], torch.float16), (np.clip(x, -65504, 65504), torch.float16), (np.clip(x, -65504, 65504)[:3], torch.float16)]
    for x in (big_bf, tiny_bf, mixed, onehot):
        xs += [(x[:1], torch.bfloat16), (x, torch.bfloat16)]
    xs += [(np.repeat(mixed, 10, axis=0), torch.bfloat16), (np.repeat(np.clip(big16, -65504, 65504), 5, axis=0), torch.float16)]   # tensor-core path
    # ... with bfloat16 rows far outside binary16's range (scaled by a power of two on the way in), far below it,
    # and rows where a few elements are
    xs += [(np.repeat(big_bf, 10, axis=0), torch.bfloat16), (np.repeat(tiny_bf, 10, axis=0), torch.bfloat16),
           (np.repeat(onehot, 10, axis=0), torch.bfloat16), (np.concatenate([big_bf, base, tiny_bf, mixed] * 3), torch.bfloat16)]
    _check_all(aq, W, bits, xs)
