"""GPU parity of the prefill (tensor-core) path of aq_linear against the oracle."""
import numpy as np
import pytest

from oracle import aq_oracle as O
from paper_2605_24011_b200 import synth

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def aq():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2605_24011_b200 import aq as mod
    return mod


def _run(aq, bits, N, K, M, dtype, kind="normal", out_f32=True, seed=21):
    tdt = torch.float16 if dtype == "f16" else torch.bfloat16
    W = synth.weights(N, K, seed, bits, N, outliers=True)
    h = aq.aq_pack(bits, 32, torch.from_numpy(W).cuda())
    d, m, q = O.quantize(W, bits)
    x32 = synth.activations(M, K, seed, bits, M, kind=kind)
    xt = torch.from_numpy(x32).to(tdt)
    x64 = xt.to(torch.float64).numpy()
    y = torch.full((M, N), float("nan"), dtype=torch.float32 if out_f32 else tdt, device="cuda")
    aq.aq_linear(h, xt.cuda(), y)
    aq.aq_check()
    got = y.to(torch.float64).cpu().numpy()
    yo, T = O.linear(d, m, q, x64)
    assert np.all(np.isfinite(got))
    ex = O.linear_excess(got, yo, T)
    assert ex.max() <= 1.0, f"worst normalised error {ex.max():.3f} at {np.unravel_index(ex.argmax(), ex.shape)}"
    h.free()
    return ex.max()


@pytest.mark.parametrize("bits", (4, 2, 3))
def test_gemm_smallest(aq, bits):
    """One CTA tile, one k-slab pair: the first thing to pass."""
    _run(aq, bits, 128, 256, 16, "bf16")


@pytest.mark.parametrize("bits", (2, 3, 4))
@pytest.mark.parametrize("M", (9, 16, 31, 50, 64, 100, 256, 300))
def test_gemm_token_counts(aq, bits, M):
    _run(aq, bits, 384, 1024, M, "bf16")


@pytest.mark.parametrize("bits", (2, 3, 4))
@pytest.mark.parametrize("shape", ((256, 11008), (100, 96), (272, 1280), (2048, 2048), (1024, 16384)))
def test_gemm_shapes(aq, bits, shape):
    N, K = shape
    _run(aq, bits, N, K, 50, "bf16")
    _run(aq, bits, N, K, 64, "f16", out_f32=False)


@pytest.mark.parametrize("bits", (2, 3, 4))
@pytest.mark.parametrize("M", (512, 768))
def test_gemm_prefill_rows(aq, bits, M):
    _run(aq, bits, 512, 4096, M, "bf16", kind="vision_text", out_f32=False)


@pytest.mark.parametrize("bits", (2, 3, 4))
def test_gemm_row_count_not_a_multiple_of_four(aq, bits):
    """The output row pitch is then not 16-byte aligned: the epilogue falls back from TMA to plain stores / atomics."""
    _run(aq, bits, 250, 512, 40, "bf16")
    _run(aq, bits, 1030, 1024, 300, "f16")


@pytest.mark.parametrize("M", (1024, 1300, 4096))
def test_gemm_many_tokens(aq, M):
    """Several token super-tiles, the last one ragged; M = 4096 is the largest call the library takes."""
    _run(aq, 3, 160, 512, M, "bf16")


def test_gemm_m_consistency_with_decode(aq):
    """Rows of an M=64 tensor-core call agree with the M=1 streaming call on the same handle."""
    bits, N, K = 3, 256, 1024
    W = synth.weights(N, K, 22, bits)
    h = aq.aq_pack(bits, 32, torch.from_numpy(W).cuda())
    d, m, q = O.quantize(W, bits)
    xt = torch.from_numpy(synth.activations(64, K, 22)).to(torch.float16)
    _, T = O.linear(d, m, q, xt.to(torch.float64).numpy())
    y = torch.empty((64, N), dtype=torch.float32, device="cuda")
    aq.aq_linear(h, xt.cuda(), y)
    for t in (0, 17, 63):
        y1 = torch.empty((1, N), dtype=torch.float32, device="cuda")
        aq.aq_linear(h, xt[t:t + 1].cuda(), y1)
        assert np.all(np.abs((y1[0] - y[t]).double().cpu().numpy()) <= 2 * (2e-3 * T[t] + 1e-5))
    aq.aq_check()
    h.free()
