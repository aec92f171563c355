"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle
on the same seeded inputs.  Integer/byte work must be bit-exact; linear
outputs must satisfy |y - y_oracle| <= 2e-3 * sum_k |x_k w_k| + 1e-5."""
import numpy as np
import pytest

from oracle import aq_oracle as O
from paper_2605_24011_b200 import synth

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

BITS = (2, 3, 4)


@pytest.fixture(scope="module")
def aq():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2605_24011_b200 import aq as mod
    return mod


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _x_host(M, K, dtype, *key, kind="normal"):
    """Activations rounded to the storage dtype; returns (torch tensor on GPU, float64 numpy)."""
    x32 = synth.activations(M, K, *key, kind=kind)
    xt = torch.from_numpy(x32).to(dtype)
    return xt.cuda(), xt.to(torch.float64).numpy()


# shapes: several tiles + ragged tails (N not a multiple of 16, K not of 128/256)
SHAPES = [(100, 96), (272, 1280), (512, 1024), (48, 4096 + 32)]


@pytest.mark.parametrize("bits", BITS)
@pytest.mark.parametrize("shape", SHAPES)
def test_pack_export_bytes_equal_oracle(aq, bits, shape):
    N, K = shape
    W = synth.weights(N, K, 11, bits, N, outliers=True)
    h = aq.aq_pack(bits, 32, _dev(W))
    got = aq.aq_export(h)
    d, m, q = O.quantize(W, bits)
    want = O.pack(d, m, q, bits)
    info = aq.aq_info(h)
    assert info["status"] == 0 and info["packed_bytes"] == want.size == O.packed_nbytes(N, K, bits)
    assert info["device_bytes"] >= want.size
    assert got.size == want.size
    assert np.array_equal(got, want)
    # import of those bytes exports the same bytes
    h2 = aq.aq_import(bits, 32, N, K, want)
    assert np.array_equal(aq.aq_export(h2), want)
    h.free(); h2.free()


@pytest.mark.parametrize("bits", BITS)
def test_import_arbitrary_codes(aq, bits):
    """Bytes that no quantiser produced (random codes, random fp16 params)."""
    rng = np.random.default_rng(bits)
    N, K = 40, 320
    q = rng.integers(0, (1 << bits), size=(N, K)).astype(np.uint8)
    d = (rng.standard_normal((N, K // 32)) * 0.01).astype(np.float16)
    m = (rng.standard_normal((N, K // 32)) * 0.05).astype(np.float16)
    canon = O.pack(d, m, q, bits)
    h = aq.aq_import(bits, 32, N, K, canon)
    assert np.array_equal(aq.aq_export(h), canon)
    out = torch.empty((N, K), dtype=torch.float32, device="cuda")
    aq.aq_dequant(h, out)
    assert np.array_equal(out.cpu().numpy().view(np.uint32), O.dequant(d, m, q, "f32"))
    h.free()


@pytest.mark.parametrize("bits", BITS)
@pytest.mark.parametrize("shape", SHAPES)
def test_dequant_bit_exact(aq, bits, shape):
    N, K = shape
    W = synth.weights(N, K, 12, bits, N, outliers=True)
    h = aq.aq_pack(bits, 32, _dev(W))
    d, m, q = O.quantize(W, bits)
    for name, dt, view in (("f16", torch.float16, np.uint16), ("bf16", torch.bfloat16, np.uint16), ("f32", torch.float32, np.uint32)):
        out = torch.full((N, K), float("nan"), dtype=dt, device="cuda")
        aq.aq_dequant(h, out)
        got = out.view(torch.int16 if view is np.uint16 else torch.int32).cpu().numpy().view(view)
        assert np.array_equal(got, O.dequant(d, m, q, name)), name
    h.free()


def _check_linear(aq, h, d, m, q, x_dev, x64, out_dtype):
    M = x64.shape[0]
    N = d.shape[0]
    y = torch.full((M, N), float("nan"), dtype=out_dtype, device="cuda")
    aq.aq_linear(h, x_dev, y)
    yo, T = O.linear(d, m, q, x64)
    got = y.to(torch.float64).cpu().numpy()
    assert np.all(np.isfinite(got))
    ex = O.linear_excess(got, yo, T)
    assert ex.max() <= 1.0, f"worst normalised error {ex.max():.3f}"
    return got, ex.max()


@pytest.mark.parametrize("bits", BITS)
@pytest.mark.parametrize("M", (1, 2, 3, 4, 7, 8))
@pytest.mark.parametrize("dtype", ("f16", "bf16"))
def test_linear_decode_within_bound(aq, bits, M, dtype):
    tdt = torch.float16 if dtype == "f16" else torch.bfloat16
    for (N, K) in ((272, 1280), (100, 96), (512, 4096)):
        W = synth.weights(N, K, 13, bits, N, outliers=True)
        h = aq.aq_pack(bits, 32, _dev(W))
        d, m, q = O.quantize(W, bits)
        x_dev, x64 = _x_host(M, K, tdt, 13, bits, M)
        _check_linear(aq, h, d, m, q, x_dev, x64, tdt)
        _check_linear(aq, h, d, m, q, x_dev, x64, torch.float32)     # unrounded accumulators
        # a second call on the same handle sees clean scratch
        _check_linear(aq, h, d, m, q, x_dev, x64, tdt)
        h.free()


@pytest.mark.parametrize("bits", BITS)
def test_linear_structured_inputs(aq, bits):
    """unit vector -> a column of w_hat; ones -> row sums; 2x -> exactly 2y (fp32 out);
    row t of an M=8 call against the M=1 call."""
    N, K = 256, 512
    W = synth.weights(N, K, 14, bits)
    h = aq.aq_pack(bits, 32, _dev(W))
    d, m, q = O.quantize(W, bits)
    What = O.dequant_f64(d, m, q)
    for k in (0, 7, 8, 31, 32, 255, 256, 511):
        e = torch.zeros((1, K), dtype=torch.float16, device="cuda"); e[0, k] = 1.0
        y = torch.empty((1, N), dtype=torch.float32, device="cuda")
        aq.aq_linear(h, e, y)
        got = y.double().cpu().numpy()[0]
        assert np.all(np.abs(got - What[:, k]) <= 2e-3 * np.abs(What[:, k]) + 1e-5), k
    ones = torch.ones((1, K), dtype=torch.float16, device="cuda")
    y = torch.empty((1, N), dtype=torch.float32, device="cuda")
    aq.aq_linear(h, ones, y)
    assert np.all(np.abs(y.double().cpu().numpy()[0] - What.sum(1)) <= 2e-3 * np.abs(What).sum(1) + 1e-5)
    x_dev, x64 = _x_host(8, K, torch.float16, 14, bits)
    y8 = torch.empty((8, N), dtype=torch.float32, device="cuda")
    aq.aq_linear(h, x_dev, y8)
    yo, T = O.linear(d, m, q, x64)
    for t in (0, 5, 7):
        y1 = torch.empty((1, N), dtype=torch.float32, device="cuda")
        aq.aq_linear(h, x_dev[t:t + 1].contiguous(), y1)
        assert np.all(np.abs((y1[0] - y8[t]).double().cpu().numpy()) <= 2 * (2e-3 * T[t] + 1e-5))
    h.free()


def test_range_error_is_reported(aq):
    W = synth.weights(32, 64, 15)
    W[3, 40] = np.inf
    h = aq.aq_pack(4, 32, _dev(W))
    assert aq.aq_info(h)["status"] == aq.AQ_ERR_RANGE
    h.free()
    W = synth.weights(32, 64, 15) * np.float32(1e7)     # min/scale overflow binary16
    h = aq.aq_pack(4, 32, _dev(W))
    assert aq.aq_info(h)["status"] == aq.AQ_ERR_RANGE
    h.free()
    W = synth.weights(32, 64, 15)
    h = aq.aq_pack(4, 32, _dev(W))
    assert aq.aq_info(h)["status"] == aq.AQ_OK
    h.free()


def test_bad_arguments_launch_nothing(aq):
    W = _dev(synth.weights(32, 64, 16))
    h = aq.aq_pack(4, 32, W)
    x = torch.zeros((1, 64), dtype=torch.float16, device="cuda")
    y = torch.zeros((1, 32), dtype=torch.float16, device="cuda")
    lib = aq.raw_lib()
    assert lib.aq_linear(h.raw, x.data_ptr(), y.data_ptr(), 0, 0, None) == aq.AQ_ERR_INVALID_ARG
    assert lib.aq_linear(h.raw, x.data_ptr(), y.data_ptr(), aq.AQ_MAX_M + 1, 0, None) == aq.AQ_ERR_INVALID_ARG
    assert lib.aq_linear(h.raw, x.data_ptr() + 2, y.data_ptr(), 1, 0, None) == aq.AQ_ERR_INVALID_ARG
    assert lib.aq_linear(h.raw, x.data_ptr(), y.data_ptr(), 1, aq.AQ_F32, None) == aq.AQ_ERR_UNSUPPORTED
    assert lib.aq_linear(h.raw, 0, y.data_ptr(), 1, 0, None) == aq.AQ_ERR_INVALID_ARG
    assert lib.aq_dequant(h.raw, y.data_ptr(), 7, None) == aq.AQ_ERR_INVALID_ARG
    with pytest.raises(aq.AqError):
        aq.aq_pack(5, 32, W)
    torch.cuda.synchronize()
    h.free()


def test_config1_single_linear_4bit(aq):
    """K = N = 4096, 4-bit, seed 0: export bytes, dequant and M=1 linear."""
    N = K = 4096
    W = synth.weights(N, K, 0)
    h = aq.aq_pack(4, 32, _dev(W))
    d, m, q = O.quantize(W, 4)
    canon = O.pack(d, m, q, 4)
    assert canon.size == 10_485_760
    assert np.array_equal(aq.aq_export(h), canon)
    out = torch.empty((N, K), dtype=torch.float16, device="cuda")
    aq.aq_dequant(h, out)
    assert np.array_equal(out.view(torch.int16).cpu().numpy().view(np.uint16), O.dequant(d, m, q, "f16"))
    x_dev, x64 = _x_host(1, K, torch.float16, 0)
    _check_linear(aq, h, d, m, q, x_dev, x64, torch.float16)
    h.free()
