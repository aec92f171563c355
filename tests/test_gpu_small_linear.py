"""aq_linear with M <= 8 on matrices small enough for the one-launch row-tile kernel (one CTA per 16-row tile, sums along
k in registers and shared memory, outputs written by the CTA itself), on both sides of every limit that selects it
(row tiles against four per SM, 256-k slabs between 2 and 64, outputs small enough for the fused write), against
the oracle at the stated tolerance.  N values that are not multiples of 16 check that padded rows stay out of y."""
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


def _check(aq, N, K, bits, Ms, dtypes, seed):
    W = synth.weights(N, K, seed, bits, outliers=True)
    h = aq.aq_pack(bits, 32, torch.from_numpy(W).cuda())
    d, m, q = O.quantize(W, bits)
    for M in Ms:
        for name in dtypes:
            tdt = torch.float16 if name == "f16" else torch.bfloat16
            xt = torch.from_numpy(synth.activations(M, K, seed, bits, M)).to(tdt)
            yo, T = O.linear(d, m, q, xt.to(torch.float64).numpy())
            # output in the activation type (the kernel casts) and in float32
            y = torch.full((M, N), float("nan"), dtype=tdt, device="cuda")
            guard = torch.full((64,), 7.0, dtype=tdt, device="cuda")      # allocated right behind y in most cases
            aq.aq_linear(h, xt.cuda(), y)
            y32 = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
            aq.aq_linear(h, xt.cuda(), y32)
            aq.aq_check()
            got32 = y32.double().cpu().numpy()
            assert np.all(np.isfinite(got32))
            assert O.linear_excess(got32, yo, T).max() <= 1.0, f"N={N} K={K} bits={bits} M={M} {name} f32 output"
            got = y.double().cpu().numpy()
            assert np.all(np.isfinite(got))
            # the cast adds half an ulp of the output type
            ulp = 2.0 ** (-11 if name == "f16" else -8)
            assert np.all(np.abs(got - yo) <= 2e-3 * T + 1e-5 + ulp * np.abs(yo)), f"N={N} K={K} bits={bits} M={M} {name}"
            assert torch.all(guard == 7.0)
    h.free()


@pytest.mark.parametrize("bits", (2, 3, 4))
def test_row_tile_kernel_shapes(aq, bits):
    # (N, K): one tile; ragged N; the benchmark's small configuration; K = 512 (two slabs: the least that selects the
    # kernel) and K = 256 (one slab: the streaming kernel)
    for N, K in ((16, 512), (1000, 1280), (4096, 4096), (40, 256), (24, 768)):
        _check(aq, N, K, bits, (1, 2, 3, 5, 8), ("f16", "bf16"), 100 + bits)


def test_row_tile_kernel_limits(aq):
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    # as many row tiles as the kernel takes (four per SM) and one more (streaming kernel), ragged
    for NT in (4 * sms, 4 * sms + 1):
        _check(aq, NT * 16 - 5, 512, 3, (1, 8), ("f16",), 7)
    # 64 slabs along k (the most) and 65
    for K in (64 * 256, 65 * 256):
        _check(aq, 48, K, 2, (1, 4), ("f16", "bf16"), 8)
    # outputs beyond what the fused write takes (M N > 8192): two launches
    _check(aq, 2048, 1024, 4, (4, 5), ("f16",), 9)
