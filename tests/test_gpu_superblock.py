"""Super-block format on the GPU against the oracle: pack bytes, import / export round trip, dequant bits, the linear on
both paths, and a stack pass (the handle is an ordinary one for every kernel of the hot path)."""
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


@pytest.mark.parametrize("bits", BITS)
@pytest.mark.parametrize("shape", ((16, 256), (37, 768), (300, 1024), (1, 4096)))
def test_pack_sb_bytes_dequant_and_linear(aq, bits, shape):
    N, K = shape
    W = synth.weights(N, K, 301, bits, outliers=True)
    h = aq.aq_pack_sb(bits, torch.from_numpy(W).cuda())
    D, Dm, Mn, u, v, q = O.quantize_sb(W, bits)
    want = O.pack_sb(D, Dm, Mn, u, v, q, bits)
    got = aq.aq_export_sb(h)
    assert got.size == want.size == O.packed_nbytes_sb(N, K, bits) == aq.aq_info(h)["packed_bytes"]
    assert np.array_equal(got, want), "super-block bytes differ from the oracle"
    d, m = O.sb_block_params(D, Dm, Mn, u, v)
    assert np.array_equal(aq.aq_export(h), O.pack(d, m, q, bits))          # the plain form carries the decoded parameters
    for name, tdt in (("f16", torch.float16), ("bf16", torch.bfloat16), ("f32", torch.float32)):
        out = torch.empty((N, K), dtype=tdt, device="cuda")
        aq.aq_dequant(h, out)
        ref = O.dequant(d, m, q, name)
        a = out.cpu().numpy().view(np.uint32) if name == "f32" else out.view(torch.int16).cpu().numpy().view(np.uint16)
        assert np.array_equal(a, ref), f"dequant {name} not bit-exact"
    for M, tdt in ((1, torch.float16), (7, torch.bfloat16), (40, torch.bfloat16), (130, torch.float16)):
        xt = torch.from_numpy(synth.activations(M, K, 301, M)).to(tdt)
        y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        aq.aq_linear(h, xt.cuda(), y)
        aq.aq_check()
        yo, T = O.linear(d, m, q, xt.to(torch.float64).numpy())
        assert O.linear_excess(y.double().cpu().numpy(), yo, T).max() <= 1.0
    # import of the exported bytes gives the same handle contents
    h2 = aq.aq_import_sb(bits, N, K, got)
    assert np.array_equal(aq.aq_export_sb(h2), want) and np.array_equal(aq.aq_export(h2), aq.aq_export(h))
    h.free(); h2.free()


def test_sb_rejections(aq):
    lib = aq.raw_lib()
    import ctypes as C
    W = torch.zeros((16, 288), dtype=torch.float32, device="cuda")       # K not a multiple of 256
    out = C.c_void_p()
    assert lib.aq_pack_sb(2, 32, 8, W.data_ptr(), 16, 288, None, C.byref(out)) == aq.AQ_ERR_INVALID_ARG
    W = torch.zeros((16, 256), dtype=torch.float32, device="cuda")
    assert lib.aq_pack_sb(2, 32, 4, W.data_ptr(), 16, 256, None, C.byref(out)) == aq.AQ_ERR_UNSUPPORTED
    h = aq.aq_pack(2, 32, W)
    n = C.c_size_t()
    assert lib.aq_export_sb(h.raw, None, 0, C.byref(n)) == aq.AQ_ERR_INVALID_ARG     # a plain handle has no super-block form
    h.free()


def test_sb_handles_in_a_stack(aq):
    """A tiny block stack whose matrices are super-block handles, M = 1 and M = 40: same per-op parity as plain ones."""
    from paper_2605_24011_b200 import programs
    from stack_check import check_program
    shapes = synth.tiny_layer(256, 512)
    layers, quant = [], {}
    for l in range(2):
        L = {"shape": {}}
        for i, (name, N, K) in enumerate(shapes):
            W = synth.weights(N, K, 303, l, i)
            b = (2, 3, 4)[(l + i) % 3]
            L[name] = aq.aq_pack_sb(b, torch.from_numpy(W).cuda())
            L["shape"][name] = (N, K)
            D, Dm, Mn, u, v, q = O.quantize_sb(W, b)
            d, m = O.sb_block_params(D, Dm, Mn, u, v)
            quant[(l, name)] = (d, m, q)
        layers.append(L)
    prog, out_buf, names = programs.block_program(layers)
    for M, tdt in ((1, torch.float16), (40, torch.bfloat16)):
        ws = torch.empty(prog.workspace_bytes(M), dtype=torch.uint8, device="cuda")
        x0 = torch.from_numpy(synth.activations(M, 256, 303, M)).to(tdt).cuda()
        out = torch.empty((M, 256), dtype=tdt, device="cuda")
        aq.aq_stack_forward(prog, x0, out, out_buf, M, ws)
        aq.aq_check()
        check_program(prog, names, ws, M, tdt, quant)
