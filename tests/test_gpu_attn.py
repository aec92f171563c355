"""Attention of one decoded token over a key/value cache, rotary embedding and cache append, through the C ABI,
against oracle/attn_oracle.py on the same seeded inputs.

Tolerances (derived, not tuned): the softmax weights enter the second tensor-core product rounded to the activation
type (unit roundoff u = 2^-11 for float16, 2^-8 for bfloat16) while the normaliser is summed unrounded, so a float32
output is within u * T of the exact one, T = sum_p softmax_p |V_p| (oracle.attn_bound), plus binary32 noise
(2^-16 T covers the exp2 and the running rescaling over hundreds of tiles); a 16-bit output adds its own rounding,
u |o|.  The rotation is formed from a binary64 angle and two binary32 FMAs: 2^-22 (|a| + |b|) before the output's rounding."""
import numpy as np
import pytest

from oracle import attn_oracle as A

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

U = {"f16": 2.0 ** -11, "bf16": 2.0 ** -8}
TD = {"f16": torch.float16, "bf16": torch.bfloat16, "f32": torch.float32}


@pytest.fixture(scope="module")
def aq():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2605_24011_b200 import aq as mod
    return mod


def _inputs(H, Hkv, Lmax, seed, name, qscale=1.0):
    g = np.random.default_rng(seed)
    tdt = TD[name]
    q = torch.from_numpy((g.standard_normal((H, 128)) * qscale).astype(np.float32)).to(tdt)
    K = torch.from_numpy(g.standard_normal((Hkv, Lmax, 128)).astype(np.float32)).to(tdt)
    Vn = g.standard_normal((Hkv, Lmax, 128)).astype(np.float32)
    Vn[g.random(Vn.shape) < 0.001] *= 20.0           # a few outliers
    V = torch.from_numpy(Vn).to(tdt)
    return q, K, V


def _check(aq, H, Hkv, L, Lmax, name, seed, qscale=1.0, scale=0.0):
    q, K, V = _inputs(H, Hkv, Lmax, seed, name, qscale)
    scratch = torch.empty(aq.aq_attn_scratch_bytes(Hkv), dtype=torch.uint8, device="cuda")
    scratch.fill_(0xAB)                               # its contents must not matter
    qd, Kd, Vd = q.cuda(), K.cuda(), V.cuda()
    ref = A.attn_decode(q.double().numpy(), K.double().numpy(), V.double().numpy(), L, scale if scale > 0 else None)
    T = A.attn_bound(q.double().numpy(), K.double().numpy(), V.double().numpy(), L, scale if scale > 0 else None)
    u = U[name]
    for out_name in ("f32", name):
        out = torch.full((H, 128), float("nan"), dtype=TD[out_name], device="cuda")
        for _ in range(2):                            # twice: the tickets must be back at zero after a call
            aq.aq_attn_decode(qd, Kd, Vd, L, out, scratch, scale)
        aq.aq_check()
        got = out.double().cpu().numpy()
        assert np.all(np.isfinite(got))
        tol = (u + 2.0 ** -16) * T + 1e-6 + (0.0 if out_name == "f32" else u * np.abs(ref))
        err = np.abs(got - ref)
        assert np.all(err <= tol), f"H={H} Hkv={Hkv} L={L} {name}->{out_name}: worst {np.max(err / tol):.3f} tolerances"


@pytest.mark.parametrize("name", ("f16", "bf16"))
def test_attention_shapes(aq, name):
    # one position; inside one tile; one more than a tile; the splits' edges; a full 4096-token cache; ragged L and L_max
    for H, Hkv, L, Lmax in ((32, 32, 1, 64), (32, 32, 31, 64), (32, 32, 33, 64), (32, 32, 128, 128), (32, 32, 129, 4096),
                            (32, 32, 4096, 4096), (32, 32, 1000, 1000), (8, 8, 2047, 2048)):
        _check(aq, H, Hkv, L, Lmax, name, 10 + L)


@pytest.mark.parametrize("name", ("f16", "bf16"))
def test_attention_grouped_queries(aq, name):
    for H, Hkv, L, Lmax in ((32, 8, 1000, 1024), (16, 1, 777, 1024), (64, 4, 300, 512), (2, 1, 5, 8), (48, 16, 2500, 3000)):
        _check(aq, H, Hkv, L, Lmax, name, 20 + L)


def test_attention_peaked_and_flat_scores(aq):
    _check(aq, 32, 32, 1500, 2048, "f16", 31, qscale=6.0)       # scores of standard deviation 6: a few positions dominate
    _check(aq, 32, 32, 1500, 2048, "f16", 32, qscale=0.0)       # zero query: the mean of the values
    _check(aq, 32, 32, 700, 1024, "f16", 33, scale=0.25)        # a scale of the caller's own


def test_rope_and_append_build_the_cache(aq):
    g = np.random.default_rng(40)
    Hkv, H, Lmax, L = 4, 8, 64, 40
    for name in ("f16", "bf16"):
        tdt = TD[name]
        kc = torch.zeros((Hkv, Lmax, 128), dtype=tdt, device="cuda")
        vc = torch.zeros((Hkv, Lmax, 128), dtype=tdt, device="cuda")
        Kref = np.zeros((Hkv, Lmax, 128))
        Vref = np.zeros((Hkv, Lmax, 128))
        for pos in range(L):
            k = torch.from_numpy(g.standard_normal((Hkv, 128)).astype(np.float32)).to(tdt)
            v = torch.from_numpy(g.standard_normal((Hkv, 128)).astype(np.float32)).to(tdt)
            kd = k.cuda()
            aq.aq_rope(kd, pos)
            rk = A.rope(k.double().numpy(), pos)
            got = kd.double().cpu().numpy()
            lim = U[name] * np.abs(rk) + 2.0 ** -22 * (np.abs(k.double().numpy()) + np.abs(np.roll(k.double().numpy(), 64, axis=1))) + 1e-9
            assert np.all(np.abs(got - rk) <= lim), f"rope {name} pos {pos}"
            aq.aq_kv_append(kc, vc, kd, v.cuda(), pos)
            Kref[:, pos] = got                        # what the cache holds is the GPU's rounded rotation
            Vref[:, pos] = v.double().numpy()
        assert np.array_equal(kc.double().cpu().numpy(), Kref) and np.array_equal(vc.double().cpu().numpy(), Vref)
        q = torch.from_numpy(g.standard_normal((H, 128)).astype(np.float32)).to(tdt).cuda()
        aq.aq_rope(q, L - 1)
        out = torch.empty((H, 128), dtype=torch.float32, device="cuda")
        scratch = torch.empty(aq.aq_attn_scratch_bytes(Hkv), dtype=torch.uint8, device="cuda")
        aq.aq_attn_decode(q, kc, vc, L, out, scratch)
        aq.aq_check()
        qn = q.double().cpu().numpy()
        ref, T = A.attn_decode(qn, Kref, Vref, L), A.attn_bound(qn, Kref, Vref, L)
        assert np.all(np.abs(out.double().cpu().numpy() - ref) <= (U[name] + 2.0 ** -16) * T + 1e-6)


def test_rope_float32_and_large_positions(aq):
    g = np.random.default_rng(41)
    x = g.standard_normal((5, 128)).astype(np.float32)
    for pos, theta in ((0, 10000.0), (1, 10000.0), (4095, 10000.0), (100000, 500000.0)):
        xd = torch.from_numpy(x.copy()).cuda()
        aq.aq_rope(xd, pos, theta)
        ref = A.rope(x.astype(np.float64), pos, theta)
        lim = 2.0 ** -22 * (np.abs(x) + np.abs(np.roll(x, 64, axis=1))) + 1e-12
        assert np.all(np.abs(xd.double().cpu().numpy() - ref) <= lim), f"pos {pos}"
    # another head dimension (the rotation alone is not tied to 128)
    y = g.standard_normal((3, 64)).astype(np.float32)
    yd = torch.from_numpy(y.copy()).cuda()
    aq.aq_rope(yd, 77)
    assert np.allclose(yd.double().cpu().numpy(), A.rope(y.astype(np.float64), 77), atol=1e-5)


def test_attention_rejects_bad_arguments(aq):
    lib = aq.raw_lib()
    q = torch.zeros((32, 128), dtype=torch.float16, device="cuda")
    kc = torch.zeros((32, 64, 128), dtype=torch.float16, device="cuda")
    out = torch.zeros((32, 128), dtype=torch.float32, device="cuda")
    sc = torch.zeros(aq.aq_attn_scratch_bytes(32), dtype=torch.uint8, device="cuda")
    def call(H=32, Hkv=32, D=128, L=10, Lmax=64, dt=aq.AQ_F16, odt=aq.AQ_F32, nbytes=None, qp=None, M=1):
        return lib.aq_attn_decode(qp if qp is not None else q.data_ptr(), kc.data_ptr(), kc.data_ptr(), out.data_ptr(), M, H, Hkv, D, L, Lmax,
                                  0.0, dt, odt, sc.data_ptr(), sc.numel() if nbytes is None else nbytes, None)
    assert call() == aq.AQ_OK
    assert call(L=0) == aq.AQ_ERR_INVALID_ARG and call(L=65) == aq.AQ_ERR_INVALID_ARG
    assert call(H=33) == aq.AQ_ERR_INVALID_ARG                  # not a multiple of the key/value heads
    assert call(D=64) == aq.AQ_ERR_UNSUPPORTED
    assert call(H=34, Hkv=2) == aq.AQ_ERR_UNSUPPORTED           # 17 query heads per key/value head
    assert call(H=8, Hkv=4, M=9) == aq.AQ_ERR_UNSUPPORTED       # 2 x 9 rows
    assert call(M=0) == aq.AQ_ERR_INVALID_ARG and call(M=4, L=3) == aq.AQ_ERR_INVALID_ARG
    assert call(dt=aq.AQ_F32) == aq.AQ_ERR_UNSUPPORTED
    assert call(nbytes=1024) == aq.AQ_ERR_INVALID_ARG
    assert call(qp=q.data_ptr() + 2) == aq.AQ_ERR_INVALID_ARG
    assert lib.aq_kv_append(kc.data_ptr(), kc.data_ptr(), q.data_ptr(), q.data_ptr(), 32, 128, 64, 64, aq.AQ_F16, None) == aq.AQ_ERR_INVALID_ARG
    assert lib.aq_rope(q.data_ptr(), 32, 127, 3, 10000.0, aq.AQ_F16, None) == aq.AQ_ERR_INVALID_ARG
    torch.cuda.synchronize()
    aq.aq_check()


@pytest.mark.parametrize("name", ("f16", "bf16"))
def test_attention_of_several_new_tokens(aq, name):
    """M new tokens in one call (the decode path's 1..8, and up to 16 rows of heads x tokens): each sees the positions up
    to its own.  Includes contexts shorter than a tile, so that some rows see nothing in some warps' tiles."""
    for M, H, Hkv, L, Lmax in ((8, 32, 32, 1000, 1024), (16, 32, 32, 4096, 4096), (8, 16, 8, 333, 512), (4, 32, 8, 2049, 4096),
                               (3, 8, 8, 3, 64), (8, 8, 8, 9, 64), (2, 64, 8, 130, 256), (5, 6, 2, 37, 40)):
        g = np.random.default_rng(50 + M + L)
        tdt = TD[name]
        q = torch.from_numpy(g.standard_normal((M, H, 128)).astype(np.float32)).to(tdt)
        K = torch.from_numpy(g.standard_normal((Hkv, Lmax, 128)).astype(np.float32)).to(tdt)
        V = torch.from_numpy(g.standard_normal((Hkv, Lmax, 128)).astype(np.float32)).to(tdt)
        scratch = torch.empty(aq.aq_attn_scratch_bytes(Hkv), dtype=torch.uint8, device="cuda")
        out = torch.full((M, H, 128), float("nan"), dtype=torch.float32, device="cuda")
        aq.aq_attn_decode(q.cuda(), K.cuda(), V.cuda(), L, out, scratch)
        aq.aq_check()
        qn, Kn, Vn = q.double().numpy(), K.double().numpy(), V.double().numpy()
        ref, T = A.attn_decode_tokens(qn, Kn, Vn, L), A.attn_bound_tokens(qn, Kn, Vn, L)
        got = out.double().cpu().numpy()
        assert np.all(np.isfinite(got))
        tol = (U[name] + 2.0 ** -16) * T + 1e-6
        assert np.all(np.abs(got - ref) <= tol), f"M={M} H={H} Hkv={Hkv} L={L} {name}: worst {np.max(np.abs(got - ref) / tol):.3f}"
