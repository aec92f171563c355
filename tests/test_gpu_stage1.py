"""GPU parity of the inter-tensor stage (RBF kernel matrices, HSIC of Eq. 2, sensitivity of Eq. 5) against the oracle.

Tolerances (derived from the arithmetic, per entry):
  kernel matrix: the GPU forms D = n_i + n_j - 2 G_ij from exact products summed in binary32; with
  gamma = (d/16 + 32) 2^-23 covering the summation of the norms and of the inner product,
  |D_gpu - D| <= 3 gamma (n_i + n_j); the exponent c D then carries that error times c, the rounding of c and of the
  product (2^-21 c D) and expf's 2 ulp, so |K_gpu - K| <= K (3 gamma (n_i + n_j) c + 2^-21 c D + 2^-21) + 1e-37.
  HSIC given the same float32 matrices: binary64 on both sides, 1e-11 of the largest term.
  HSIC end to end: first-order propagation of the per-entry bounds through tr(K_A C K_B C).
"""
import math

import numpy as np
import pytest

from oracle import stage1_oracle as S1
from paper_2605_24011_b200 import synth

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def aq():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2605_24011_b200 import aq as mod
    return mod


def _half(a32, dtype):
    t = torch.from_numpy(np.ascontiguousarray(a32)).to(torch.float16 if dtype == "f16" else torch.bfloat16)
    return t, t.to(torch.float64).numpy()


def _entry_bound(A64, sigma, Kref):
    d = A64.shape[1]
    n = np.einsum("kd,kd->k", A64, A64)
    c = 1.0 / (2.0 * sigma * sigma)
    gamma = (d / 16 + 32) * 2.0**-23
    D = -np.log(np.maximum(Kref, 1e-300)) / c
    return Kref * (3 * gamma * (n[:, None] + n[None, :]) * c + 2.0**-21 * c * D + 2.0**-21) + 1e-37


def _gram_case(aq, K, d, dtype, sigma, seed, pitch=None, A32=None):
    if A32 is None:
        A32 = np.random.default_rng(seed).standard_normal((K, d)).astype(np.float32)
    t, A64 = _half(A32, dtype)
    ref = S1.rbf_gram(A64, sigma)
    if pitch is None:
        G = aq.aq_rbf_gram(t.cuda(), sigma)
    else:
        buf = torch.full((K, pitch), float("nan"), dtype=torch.float32, device="cuda")
        G = aq.aq_rbf_gram(t.cuda(), sigma, G=buf[:, :K])
        assert torch.isnan(buf[:, K:]).all()
    aq.aq_check()
    got = G.double().cpu().numpy()
    assert np.all(np.isfinite(got))
    assert np.array_equal(np.diag(got), np.ones(K))
    assert np.array_equal(got, got.T)
    err = np.abs(got - ref)
    bound = _entry_bound(A64, sigma, ref)
    worst = (err / bound).max()
    assert worst <= 1.0, f"worst error/bound {worst:.3f} at {np.unravel_index((err / bound).argmax(), err.shape)}"
    return got, ref, A64


@pytest.mark.parametrize("dtype", ("f16", "bf16"))
@pytest.mark.parametrize("K,d", ((2, 8), (100, 64), (128, 200), (129, 72), (300, 1024), (515, 4096)))
def test_rbf_gram_shapes(aq, K, d, dtype):
    _gram_case(aq, K, d, dtype, math.sqrt(d), 31)


def test_rbf_gram_row_pitch_and_bandwidths(aq):
    _gram_case(aq, 200, 256, "f16", 16.0, 32, pitch=260)
    _gram_case(aq, 200, 256, "f16", 16.0, 32, pitch=203)     # row pitch not a multiple of four: scalar stores
    _gram_case(aq, 257, 256, "bf16", 4.0, 33)                 # narrow kernel: off-diagonal entries near e^-16
    _gram_case(aq, 257, 256, "bf16", 400.0, 34)               # wide kernel: everything near 1


def test_rbf_gram_duplicates_and_close_points(aq):
    """Equal samples give exactly-cancelling distances (entry 1 within the bound); close pairs stress n_i + n_j - 2G."""
    g = np.random.default_rng(35)
    A = g.standard_normal((160, 512)).astype(np.float32)
    A[1] = A[0]
    A[100] = A[3]
    A[5] = A[4] + 1e-2 * g.standard_normal(512).astype(np.float32)
    got, ref, _ = _gram_case(aq, 160, 512, "f16", 8.0, 0, A32=A)
    assert abs(got[0, 1] - 1.0) < 1e-4 and abs(got[100, 3] - 1.0) < 1e-4


@pytest.mark.parametrize("K,d,dtype", ((2100, 1024, "bf16"), (3000, 520, "f16"), (4096, 256, "bf16"), (5000, 72, "f16")))
def test_rbf_gram_many_samples(aq, K, d, dtype):
    """Several tiles each way, ragged last tile; from about 2900 samples on the CTA-pair kernel (256-wide tiles) runs.
    Oracle on sampled rows only."""
    sigma = math.sqrt(d)
    A32 = np.random.default_rng(36).standard_normal((K, d)).astype(np.float32)
    t, A64 = _half(A32, dtype)
    G = aq.aq_rbf_gram(t.cuda(), sigma)
    aq.aq_check()
    got = G.double().cpu().numpy()
    assert np.all(np.isfinite(got))
    assert np.array_equal(got, got.T) and np.array_equal(np.diag(got), np.ones(K))
    n = np.einsum("kd,kd->k", A64, A64)
    c = 1 / (2 * sigma * sigma)
    for i in sorted({0, 127, 128, 255, 256, 1023, 2047, 2048, K - 257, K - 129, K - 1}):
        diff = A64 - A64[i]
        ref = np.exp(-np.einsum("kd,kd->k", diff, diff) * c)
        bound = ref * (3 * (d / 16 + 32) * 2.0**-23 * (n + n[i]) * c + 2.0**-21 * (-np.log(ref)) + 2.0**-21) + 1e-37
        assert np.all(np.abs(got[i] - ref) <= bound), f"row {i}"


@pytest.mark.parametrize("K", (2, 3, 64, 257, 1000))
def test_hsic_given_the_same_matrices(aq, K):
    g = np.random.default_rng(40 + K)
    KA = S1.rbf_gram(g.standard_normal((K, 6)), 2.0).astype(np.float32)
    KB = S1.rbf_gram(np.tanh(g.standard_normal((K, 3))), 1.0).astype(np.float32)
    out = aq.aq_hsic(torch.from_numpy(KA).cuda(), torch.from_numpy(KB).cuda())
    aq.aq_check()
    ref = S1.hsic(KA.astype(np.float64), KB.astype(np.float64))
    scale = float(np.sum(KA.astype(np.float64) * KB)) / (K - 1) ** 2
    assert abs(out.item() - ref) <= 1e-11 * scale
    # a padded row pitch (here not a multiple of four: another, equally fixed, summation order) agrees to rounding
    pa = torch.zeros((K, K + 5), dtype=torch.float32, device="cuda")
    pb = torch.zeros((K, K + 5), dtype=torch.float32, device="cuda")
    pa[:, :K] = torch.from_numpy(KA)
    pb[:, :K] = torch.from_numpy(KB)
    assert abs(aq.aq_hsic(pa[:, :K], pb[:, :K]).item() - ref) <= 1e-11 * scale
    assert aq.aq_hsic(torch.from_numpy(KA).cuda(), torch.from_numpy(KB).cuda()).item() == out.item()   # reproducible


def test_largest_sample_count(aq):
    """K = AQ_HSIC_MAX_K samples: the kernel matrix on sampled rows, HSIC of two such matrices against the O(K^2)
    form of the oracle (float64 on the same float32 matrices)."""
    K, d = 16384, 64
    g = np.random.default_rng(60)
    A32 = g.standard_normal((K, d)).astype(np.float32)
    B32 = (np.tanh(A32[:, :8] @ g.standard_normal((8, 16)).astype(np.float32)) + 0.3 * g.standard_normal((K, 16)).astype(np.float32))
    (ta, A64), (tb, B64) = _half(A32, "f16"), _half(B32, "bf16")
    GA = aq.aq_rbf_gram(ta.cuda(), 8.0)
    GB = aq.aq_rbf_gram(tb.cuda(), 4.0)
    out = aq.aq_hsic(GA, GB)
    aq.aq_check()
    for (G, X64, sigma) in ((GA, A64, 8.0), (GB, B64, 4.0)):
        dd = X64.shape[1]
        n = np.einsum("kd,kd->k", X64, X64)
        c = 1 / (2 * sigma * sigma)
        for i in (0, 255, 256, 8191, 8192, 16127, 16383):
            got = G[i].double().cpu().numpy()
            diff = X64 - X64[i]
            ref = np.exp(-np.einsum("kd,kd->k", diff, diff) * c)
            bound = ref * (3 * (dd / 16 + 32) * 2.0**-23 * (n + n[i]) * c + 2.0**-21 * (-np.log(np.maximum(ref, 1e-300))) + 2.0**-21) + 1e-37
            assert np.all(np.abs(got - ref) <= bound), f"row {i}"
            assert got[i] == 1.0
    ka, kb = GA.cpu().numpy(), GB.cpu().numpy()
    ref = S1.hsic_large(ka, kb)
    scale = float(np.sum(ka.astype(np.float64) * kb)) / (K - 1) ** 2
    assert abs(out.item() - ref) <= 1e-10 * scale
    assert ref > 0


def test_sensitivity_end_to_end(aq):
    """Eq. 5 from samples: three kernel matrices on the tensor cores, two traces, one combination."""
    K, d_in, d_out, d_act = 384, 512, 1024, 8
    alpha, beta = 0.5, 2.0
    res = {}
    for name, (rel, red) in {"relevant": (0.8, 0.2), "redundant": (0.1, 0.9)}.items():
        X, Z, Y = synth.calibration(K, d_in, d_out, d_act, 50, relevance=rel, redundancy=red)
        (tx, X64), (tz, Z64), (ty, Y64) = _half(X, "f16"), _half(Z, "f16"), _half(Y, "f16")
        sx, sz, sy = math.sqrt(d_in), math.sqrt(d_out), math.sqrt(d_act)
        KX, KZ, KY = aq.aq_rbf_gram(tx.cuda(), sx), aq.aq_rbf_gram(tz.cuda(), sz), aq.aq_rbf_gram(ty.cuda(), sy)
        out = aq.aq_sensitivity(KX, KZ, KY, alpha, beta).cpu().numpy()
        aq.aq_check()
        rX, rZ, rY = S1.rbf_gram(X64, sx), S1.rbf_gram(Z64, sz), S1.rbf_gram(Y64, sy)
        s_ref, hxz, hzy = S1.sensitivity(S1.hsic(rX, rZ), S1.hsic(rZ, rY), alpha, beta), S1.hsic(rX, rZ), S1.hsic(rZ, rY)
        C = S1.centering(K)
        eX, eZ, eY = _entry_bound(X64, sx, rX), _entry_bound(Z64, sz, rZ), _entry_bound(Y64, sy, rY)

        def tol(P, eP, Q, eQ):
            return (np.sum(eP * np.abs(C @ Q @ C)) + np.sum(np.abs(C @ P @ C) * eQ) + np.sum(eP * eQ)) / (K - 1) ** 2 + 1e-11 * abs(np.sum(P * Q)) / (K - 1) ** 2

        t1, t2 = tol(rX, eX, rZ, eZ), tol(rZ, eZ, rY, eY)
        assert abs(out[1] - hxz) <= t1 and abs(out[2] - hzy) <= t2
        assert abs(out[0] - s_ref) <= alpha * t1 + beta * t2 + 1e-15
        assert out[0] == pytest.approx(-alpha * out[1] + beta * out[2], rel=1e-12, abs=1e-18)
        res[name] = out
        assert t1 < 0.05 * hxz and t2 < 0.05 * max(hzy, 1e-5)      # the bound is tight enough to mean something
    # the synthetic knobs do what they say: task relevance raises HSIC(Z, Y), input redundancy raises HSIC(X, Z)
    assert res["relevant"][2] > 3 * res["redundant"][2]
    assert res["redundant"][1] > res["relevant"][1]


def test_stage1_bad_arguments(aq):
    A = torch.zeros((16, 16), dtype=torch.float16, device="cuda")
    G = torch.empty((16, 16), dtype=torch.float32, device="cuda")
    out = torch.empty(3, dtype=torch.float64, device="cuda")
    with pytest.raises(aq.AqError):
        aq.aq_rbf_gram(A, 0.0)
    with pytest.raises(aq.AqError):
        aq.aq_rbf_gram(A[:, :12].contiguous(), 1.0)                     # d not a multiple of 8
    with pytest.raises(aq.AqError):
        aq.aq_rbf_gram(A[:1], 1.0)                                      # one sample
    with pytest.raises(aq.AqError):
        aq.aq_rbf_gram(torch.zeros((16, 16), dtype=torch.float32, device="cuda"), 1.0)
    with pytest.raises(aq.AqError):
        aq.aq_sensitivity(G, G, G, -1.0, 1.0, out=out)
    with pytest.raises(aq.AqError):
        aq.aq_hsic(G[:1, :1], G[:1, :1])
    aq.aq_check()
