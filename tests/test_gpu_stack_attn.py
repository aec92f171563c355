"""aq_stack_forward_attn: a stack of transformer blocks decoded with the attention in its place (q, k, v -> rotation,
cache append, attention over the cache -> W_o ...), through the C ABI.

Checked teacher-forced, like the plain stack: every linear against the oracle applied to the input the GPU staged
(tests/stack_check.py); every attention step against the oracle applied to what the GPU's own q, k, v buffers and caches
hold: the rows appended to the caches are the rounded rotation of the float32 k and the rounded v, the attention output
is softmax attention of the rounded rotated q over the GPU's caches.  The oracle's q may differ from the GPU's by one
rounding of the activation type (the rotation runs in binary32 there, binary64 here), which moves an output by up to
about u * T more, T = sum_p softmax_p |V_p|: hence (2 u + 2^-16) T."""
import numpy as np
import pytest

from oracle import aq_oracle as O
from oracle import attn_oracle as A
from paper_2605_24011_b200 import synth
from stack_check import check_program

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

U = {torch.float16: 2.0 ** -11, torch.bfloat16: 2.0 ** -8}


@pytest.fixture(scope="module")
def aq():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2605_24011_b200 import aq as mod
    return mod


def _model(aq, hidden, kv_width, inter, n_layers, seed):
    shapes = (("q", hidden, hidden), ("k", kv_width, hidden), ("v", kv_width, hidden), ("o", hidden, hidden),
              ("gate", inter, hidden), ("up", inter, hidden), ("down", hidden, inter))
    layers, quant = [], {}
    for l in range(n_layers):
        L = {"shape": {}}
        for i, (name, N, K) in enumerate(shapes):
            W = synth.weights(N, K, seed, l, i)
            b = (2, 3, 4)[(l + i) % 3]
            L[name] = aq.aq_pack(b, 32, torch.from_numpy(W).cuda())
            L["shape"][name] = (N, K)
            quant[(l, name)] = O.quantize(W, b)
        layers.append(L)
    return layers, quant


def _round(a, tdt):
    return torch.from_numpy(np.asarray(a, dtype=np.float32)).to(tdt).double().numpy()


@pytest.mark.parametrize("tdt", (torch.float16, torch.bfloat16))
@pytest.mark.parametrize("hidden,kv_width", ((256, 256), (512, 256)))
def test_blocks_with_attention(aq, tdt, hidden, kv_width):
    from paper_2605_24011_b200 import programs
    H, Hkv, Lmax, n_layers = hidden // 128, kv_width // 128, 96, 2
    layers, quant = _model(aq, hidden, kv_width, 416, n_layers, 60 + hidden)
    prog, out_buf, names, attn = programs.block_program_attn(layers, H, Hkv)
    g = np.random.default_rng(61)
    u = U[tdt]
    caches = []
    for t in attn:
        kc = torch.from_numpy(g.standard_normal((Hkv, Lmax, 128)).astype(np.float32)).to(tdt).cuda()
        vc = torch.from_numpy(g.standard_normal((Hkv, Lmax, 128)).astype(np.float32)).to(tdt).cuda()
        t["k_cache"], t["v_cache"] = kc, vc
        caches.append((kc.clone(), vc.clone()))
    pos = 37
    for M in (4, 1, 8):     # three calls in a row: the cache grows by M each time
        ws = torch.empty(prog.workspace_bytes(M), dtype=torch.uint8, device="cuda")
        scratch = torch.empty(aq.aq_stack_attn_scratch_bytes(H, Hkv, M), dtype=torch.uint8, device="cuda")
        x0 = torch.from_numpy(synth.activations(M, hidden, 62, M)).to(tdt).cuda()
        out = torch.empty((M, hidden), dtype=tdt, device="cuda")
        aq.aq_stack_forward_attn(prog, attn, pos, x0, out, out_buf, M, ws, scratch)
        aq.aq_check()
        check_program(prog, names, ws, M, tdt, quant)
        for li, t in enumerate(attn):
            q = aq.stack_buffer(prog, ws, M, t["q_buf"]).double().cpu().numpy().reshape(M, H, 128)
            k = aq.stack_buffer(prog, ws, M, t["k_buf"]).double().cpu().numpy().reshape(M, Hkv, 128)
            v = aq.stack_buffer(prog, ws, M, t["v_buf"]).double().cpu().numpy().reshape(M, Hkv, 128)
            Kg, Vg = t["k_cache"].double().cpu().numpy(), t["v_cache"].double().cpu().numpy()
            K0, V0 = caches[li][0].double().cpu().numpy(), caches[li][1].double().cpu().numpy()
            # rows outside pos .. pos + M - 1 are untouched
            keep = np.ones(Lmax, dtype=bool)
            keep[pos:pos + M] = False
            assert np.array_equal(Kg[:, keep], K0[:, keep]) and np.array_equal(Vg[:, keep], V0[:, keep])
            qr = np.empty_like(q)
            for m in range(M):
                rk = A.rope(k[m], pos + m)
                lim = u * np.abs(rk) + 2.0 ** -22 * (np.abs(k[m]) + np.abs(np.roll(k[m], 64, axis=1))) + 1e-9
                assert np.all(np.abs(Kg[:, pos + m] - rk) <= lim), f"layer {li} token {m}: appended key"
                assert np.array_equal(Vg[:, pos + m], _round(v[m], tdt)), f"layer {li} token {m}: appended value"
                qr[m] = _round(A.rope(q[m], pos + m), tdt)
            ref = A.attn_decode_tokens(qr, Kg, Vg, pos + M)
            T = A.attn_bound_tokens(qr, Kg, Vg, pos + M)
            got = aq.stack_buffer(prog, ws, M, t["dst_buf"]).double().cpu().numpy().reshape(M, H, 128)
            tol = (2 * u + 2.0 ** -16) * T + 1e-6
            assert np.all(np.abs(got - ref) <= tol), f"layer {li} M={M}: attention off by {np.max(np.abs(got - ref) / tol):.3f} tolerances"
            caches[li] = (t["k_cache"].clone(), t["v_cache"].clone())
        # the rounded output is the last buffer rounded
        last = aq.stack_buffer(prog, ws, M, out_buf)
        assert torch.equal(out, last.to(tdt))
        pos += M
    for L in layers:
        for nm in ("q", "k", "v", "o", "gate", "up", "down"):
            L[nm].free()


def test_rejects_bad_attention_steps(aq):
    from paper_2605_24011_b200 import programs
    layers, _ = _model(aq, 256, 256, 416, 1, 70)
    prog, out_buf, names, attn = programs.block_program_attn(layers, 2, 2)
    kc = torch.zeros((2, 64, 128), dtype=torch.float16, device="cuda")
    attn[0]["k_cache"] = attn[0]["v_cache"] = kc
    M = 1
    ws = torch.empty(prog.workspace_bytes(M), dtype=torch.uint8, device="cuda")
    scratch = torch.empty(aq.aq_stack_attn_scratch_bytes(2, 2, 8), dtype=torch.uint8, device="cuda")
    x0 = torch.zeros((8, 256), dtype=torch.float16, device="cuda")
    out = torch.empty((8, 256), dtype=torch.float16, device="cuda")

    def status(a, pos=3, M=1):
        try:
            aq.aq_stack_forward_attn(prog, a, pos, x0[:M], out[:M], out_buf, M, torch.empty(prog.workspace_bytes(M), dtype=torch.uint8, device="cuda"), scratch)
        except aq.AqError as e:
            return e.status
        return aq.AQ_OK

    assert status(attn) == aq.AQ_OK
    bad = [dict(attn[0], after_op=1)]                   # in the middle of the q | k | v phase
    assert status(bad) == aq.AQ_ERR_INVALID_ARG
    bad = [dict(attn[0], dst_buf=attn[0]["q_buf"])]     # a buffer that an op writes
    assert status(bad) == aq.AQ_ERR_INVALID_ARG
    bad = [dict(attn[0], after_op=0)]                   # k and v are not written yet
    assert status(bad) == aq.AQ_ERR_INVALID_ARG
    assert status(attn, pos=64) == aq.AQ_ERR_INVALID_ARG            # past the end of the cache
    bad = [dict(attn[0], n_heads=4)]                    # widths do not match
    assert status(bad) == aq.AQ_ERR_INVALID_ARG
    torch.cuda.synchronize()
    aq.aq_check()
    for nm in ("q", "k", "v", "o", "gate", "up", "down"):
        layers[0][nm].free()
    del ws


def test_token_replayed_from_a_cuda_graph(aq):
    """After one eager call with the same arguments the whole token (for these two blocks: three stretches of linears,
    two preparation and two attention kernels, one cast) records into a CUDA graph; a replay rewrites the same cache rows
    and must reproduce the eager result bit for bit where the arithmetic has one order (the caches and the rounded
    rotation) and within the linears' tolerance elsewhere (their sums are atomic adds)."""
    from paper_2605_24011_b200 import programs
    layers, quant = _model(aq, 256, 256, 416, 2, 80)
    prog, out_buf, names, attn = programs.block_program_attn(layers, 2, 2)
    g = np.random.default_rng(81)
    for t in attn:
        t["k_cache"] = torch.from_numpy(g.standard_normal((2, 64, 128)).astype(np.float32)).half().cuda()
        t["v_cache"] = torch.from_numpy(g.standard_normal((2, 64, 128)).astype(np.float32)).half().cuda()
    M, pos = 2, 20
    ws = torch.empty(prog.workspace_bytes(M), dtype=torch.uint8, device="cuda")
    scratch = torch.empty(aq.aq_stack_attn_scratch_bytes(2, 2, M), dtype=torch.uint8, device="cuda")
    x0 = torch.from_numpy(synth.activations(M, 256, 82, M)).half().cuda()
    out = torch.empty((M, 256), dtype=torch.float16, device="cuda")
    aq.aq_stack_forward_attn(prog, attn, pos, x0, out, out_buf, M, ws, scratch)
    aq.aq_check()
    eager = out.clone()
    k_eager = [t["k_cache"].clone() for t in attn]
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            aq.aq_stack_forward_attn(prog, attn, pos, x0, out, out_buf, M, ws, scratch)
    torch.cuda.synchronize()
    for _ in range(2):
        out.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        aq.aq_check()
        check_program(prog, names, ws, M, torch.float16, quant)
        assert torch.all(torch.isfinite(out))
        # first block's appended keys depend on the program input alone: identical; the output agrees to a few roundings
        assert torch.equal(attn[0]["k_cache"], k_eager[0])
        assert torch.allclose(out.float(), eager.float(), rtol=2e-2, atol=2e-2)
    for L in layers:
        for nm in ("q", "k", "v", "o", "gate", "up", "down"):
            L[nm].free()
