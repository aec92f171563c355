"""aq_pack_opt (Section 3.3, Eq. 10 and Eq. 11) against the oracle: the exported bytes must be equal."""
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


def _fisher(N, K, seed):
    g = synth.weights(N, K, seed, 1).astype(np.float64)
    return (g * g * 2500.0 + 1e-4).astype(np.float32)      # squared-gradient-like, positive, wide range


@pytest.mark.parametrize("bits", (2, 3, 4))
@pytest.mark.parametrize("shape", ((16, 256), (272, 1280), (100, 96), (512, 4096)))
@pytest.mark.parametrize("with_fisher", (False, True))
def test_bytes_equal_the_oracle(aq, bits, shape, with_fisher):
    N, K = shape
    W = synth.weights(N, K, 61, bits, N, outliers=True)
    F = _fisher(N, K, 62) if with_fisher else None
    h = aq.aq_pack_opt(bits, 32, torch.from_numpy(W).cuda(), None if F is None else torch.from_numpy(F).cuda(), rounds=4)
    got = aq.aq_export(h)
    d, m, q = O.quantize_opt(W, bits, F, rounds=4)
    want = O.pack(d, m, q, bits)
    assert got.size == want.size == O.packed_nbytes(N, K, bits)
    bad = np.flatnonzero(got != want)
    assert bad.size == 0, f"{bad.size} bytes differ, first at {bad[:4]}"
    # and the handle is an ordinary one: dequant is the bit-exact decode of those bytes
    out = torch.empty((N, K), dtype=torch.float16, device="cuda")
    aq.aq_dequant(h, out)
    assert np.array_equal(out.view(torch.int16).cpu().numpy().view(np.uint16), O.dequant(d, m, q, "f16"))
    h.free()


@pytest.mark.parametrize("bits", (2, 3, 4))
def test_zero_rounds_is_plain_packing_and_more_rounds_lower_phi(aq, bits):
    W = synth.weights(64, 512, 63, bits, outliers=True)
    Wd = torch.from_numpy(W).cuda()
    h0, h1 = aq.aq_pack(bits, 32, Wd), aq.aq_pack_opt(bits, 32, Wd, None, rounds=0)
    assert np.array_equal(aq.aq_export(h0), aq.aq_export(h1))
    d0, m0, q0 = O.quantize(W, bits)
    phi = [O.block_phi(W, d0, m0, q0).sum()]
    for rounds in (1, 4):
        d, m, q = O.quantize_opt(W, bits, None, rounds=rounds)
        h = aq.aq_pack_opt(bits, 32, Wd, None, rounds=rounds)
        assert np.array_equal(aq.aq_export(h), O.pack(d, m, q, bits))
        phi.append(O.block_phi(W, d, m, q).sum())
        h.free()
    assert phi[1] < phi[0] and phi[2] <= phi[1] * (1 + 1e-6)
    h0.free(); h1.free()


def test_bad_arguments(aq):
    W = torch.from_numpy(synth.weights(16, 64, 64)).cuda()
    for kw in ({"rounds": -1}, {"rounds": 65}):
        with pytest.raises(aq.AqError):
            aq.aq_pack_opt(4, 32, W, None, **kw)
    with pytest.raises(aq.AqError):
        aq.aq_pack_opt(5, 32, W, None)
