"""aq_linear_noalloc, the entry point for callers that may not allocate device
memory (deadline loops, fixed memory budgets): its output must agree with
aq_linear's on the same inputs, on two calls in a row (the second call finds the
shared scratch array as the first one left it).  Collected last on purpose."""
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


@pytest.mark.parametrize("bits,M,dtype", [(2, 1, "f16"), (3, 8, "f16"), (4, 3, "bf16")])
def test_noalloc_matches_aq_linear_twice(aq, bits, M, dtype):
    tdt = torch.float16 if dtype == "f16" else torch.bfloat16
    N, K = 1000, 1280            # N is not a multiple of 16: the padded rows stay out of y
    W = synth.weights(N, K, 41, bits, outliers=True)
    h = aq.aq_pack(bits, 32, torch.from_numpy(W).cuda())
    d, m, q = O.quantize(W, bits)
    for call in range(2):
        xt = torch.from_numpy(synth.activations(M, K, 41, bits, call)).to(tdt)
        x = xt.cuda()
        y_ref = torch.empty((M, N), dtype=tdt, device="cuda")
        aq.aq_linear(h, x, y_ref)
        y = torch.full((M, N), float("nan"), dtype=tdt, device="cuda")
        aq.aq_linear_noalloc(h, x, y)
        aq.aq_check()
        yo, T = O.linear(d, m, q, xt.to(torch.float64).numpy())
        a, b = y.double().cpu().numpy(), y_ref.double().cpu().numpy()
        assert np.all(np.isfinite(a))
        # each within the library's bound of the exact product, hence within twice the bound of each other
        assert O.linear_excess(a, yo, T).max() <= 1.0
        assert np.all(np.abs(a - b) <= 2 * (2e-3 * T + 1e-5))
    h.free()


def test_noalloc_leaves_device_memory_alone_and_fills_the_scratch_to_its_edge(aq):
    """The property the entry point exists for: after one warm-up call (which looks up the array's address) a burst of
    calls changes neither the free device memory nor anything the caching allocator holds.  The shape is the largest
    the fixed array takes: 8 tokens and N = 16380, padded to 16384 rows, so the last row of the last token is the
    array's last element; the result must still agree with aq_linear's."""
    N, K, M = 16380, 64, 8
    W = synth.weights(N, K, 43, 2)
    h = aq.aq_pack(3, 32, torch.from_numpy(W).cuda())
    xt = torch.from_numpy(synth.activations(M, K, 43, 1)).to(torch.float16)
    x = xt.cuda()
    y = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda")
    y_ref = torch.empty((M, N), dtype=torch.float16, device="cuda")
    aq.aq_linear(h, x, y_ref)
    aq.aq_linear_noalloc(h, x, y)                 # warm-up: first call on the device
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    reserved0 = torch.cuda.memory_reserved()
    for _ in range(20):
        aq.aq_linear_noalloc(h, x, y)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0 and torch.cuda.memory_reserved() == reserved0
    aq.aq_check()
    d, m, q = O.quantize(W, 3)
    yo, T = O.linear(d, m, q, xt.to(torch.float64).numpy())
    a, b = y.double().cpu().numpy(), y_ref.double().cpu().numpy()
    assert O.linear_excess(a, yo, T).max() <= 1.0
    assert np.all(np.abs(a - b) <= 2 * (2e-3 * T + 1e-5))
    h.free()


def test_noalloc_rejects_what_the_fixed_scratch_cannot_hold(aq):
    lib = aq.raw_lib()
    W = torch.from_numpy(synth.weights(32, 64, 42)).cuda()
    h = aq.aq_pack(4, 32, W)
    x = torch.zeros((9, 64), dtype=torch.float16, device="cuda")
    y = torch.zeros((9, 32), dtype=torch.float16, device="cuda")
    assert lib.aq_linear_noalloc(h.raw, x.data_ptr(), y.data_ptr(), 9, aq.AQ_F16, None) == aq.AQ_ERR_UNSUPPORTED
    assert lib.aq_linear_noalloc(h.raw, x.data_ptr(), y.data_ptr(), 0, aq.AQ_F16, None) == aq.AQ_ERR_INVALID_ARG
    h.free()
    big = aq.aq_pack(2, 32, torch.zeros((16400, 32), dtype=torch.float32, device="cuda"))   # N > 16384
    xb = torch.zeros((1, 32), dtype=torch.float16, device="cuda")
    yb = torch.zeros((1, 16400), dtype=torch.float16, device="cuda")
    assert lib.aq_linear_noalloc(big.raw, xb.data_ptr(), yb.data_ptr(), 1, aq.AQ_F16, None) == aq.AQ_ERR_UNSUPPORTED
    torch.cuda.synchronize()
    big.free()
