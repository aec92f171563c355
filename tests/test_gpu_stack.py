"""aq_stack_forward against the oracle, op by op (teacher-forced)."""
import numpy as np
import pytest

from oracle import aq_oracle as O
from paper_2605_24011_b200 import synth
from stack_check import check_program

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def aq():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2605_24011_b200 import aq as mod
    return mod


def _build_layers(aq, layer_shapes, n_layers, bits_list, seed, outliers=True):
    layers, quant = [], {}
    i = 0
    for l in range(n_layers):
        L = {"shape": {}}
        for (name, N, K) in layer_shapes:
            W = synth.weights(N, K, seed, l, i, outliers=outliers)
            b = bits_list[i]
            L[name] = aq.aq_pack(b, 32, torch.from_numpy(W).cuda())
            L["shape"][name] = (N, K)
            quant[(l, name)] = O.quantize(W, b)
            i += 1
        layers.append(L)
    return layers, quant


@pytest.mark.parametrize("M,dtype", [(1, "f16"), (3, "f16"), (8, "f16"), (2, "bf16"), (50, "bf16"), (300, "bf16")])
def test_tiny_block_stack(aq, M, dtype):
    from paper_2605_24011_b200 import programs
    tdt = torch.float16 if dtype == "f16" else torch.bfloat16
    shapes = synth.tiny_layer(256, 416)
    n_layers = 3
    sizes = [N * K for _ in range(n_layers) for (_, N, K) in shapes]
    bits = synth.draw_bits(sizes, 3.0, 5)
    layers, quant = _build_layers(aq, shapes, n_layers, bits, 31)
    prog, out_buf, names = programs.block_program(layers)
    ws = torch.empty(prog.workspace_bytes(M), dtype=torch.uint8, device="cuda")
    x0 = torch.from_numpy(synth.activations(M, 256, 31, M)).to(tdt).cuda()
    out = torch.empty((M, 256), dtype=tdt, device="cuda")
    aq.aq_stack_forward(prog, x0, out, out_buf, M, ws)
    aq.aq_check()
    worst, worst_in = check_program(prog, names, ws, M, tdt, quant)
    # buffer 0 is the widened input; `out` is the rounded last residual
    assert torch.equal(aq.stack_buffer(prog, ws, M, 0), x0.float())
    assert torch.equal(out, aq.stack_buffer(prog, ws, M, out_buf).to(tdt))
    # values stayed finite and non-trivial
    assert float(out.float().abs().max()) > 0 and bool(torch.isfinite(out.float()).all())


@pytest.mark.parametrize("M,dtype", [(1, "f16"), (8, "f16"), (40, "bf16")])
@pytest.mark.parametrize("shapes", ("tiny", "expert_like"))
def test_independent_inputs_program(aq, M, dtype, shapes):
    """The second reading of a "linear stack": no chain, every linear reads the program input (or the first block's
    q / silu(gate) * up where its K differs); per-op parity as for the chained program."""
    from paper_2605_24011_b200 import programs
    tdt = torch.float16 if dtype == "f16" else torch.bfloat16
    layer = synth.tiny_layer(256, 416) if shapes == "tiny" else [("q", 512, 256), ("k", 64, 256), ("v", 64, 256), ("o", 256, 512),
                                                                 ("gate", 416, 256), ("up", 416, 256), ("down", 256, 416)]
    n_layers = 3
    sizes = [N * K for _ in range(n_layers) for (_, N, K) in layer]
    bits = synth.draw_bits(sizes, 3.0, 7)
    layers, quant = _build_layers(aq, layer, n_layers, bits, 33)
    prog, out_buf, names = programs.independent_program(layers)
    assert sorted(names) == sorted((l, nm) for l in range(n_layers) for (nm, _, _) in layer)
    ws = torch.empty(prog.workspace_bytes(M), dtype=torch.uint8, device="cuda")
    x0 = torch.from_numpy(synth.activations(M, 256, 33, M)).to(tdt).cuda()
    out = torch.empty((M, prog.buf_width[out_buf]), dtype=tdt, device="cuda")
    aq.aq_stack_forward(prog, x0, out, out_buf, M, ws)
    aq.aq_check()
    check_program(prog, names, ws, M, tdt, quant)


@pytest.mark.parametrize("M", (1, 8))
def test_config2_llama_mlp_3bit(aq, M):
    """gate/up 4096 -> 11008, down 11008 -> 4096, 3-bit, x fp16 N(0,1), SiLU(gate)*up in fp32."""
    from paper_2605_24011_b200 import programs
    H, I = 4096, 11008
    mats, quant = {}, {}
    for i, (name, N, K) in enumerate((("gate", I, H), ("up", I, H), ("down", H, I))):
        W = synth.weights(N, K, 2, i)
        mats[name] = aq.aq_pack(3, 32, torch.from_numpy(W).cuda())
        quant[(0, name)] = O.quantize(W, 3)
        assert aq.aq_info(mats[name])["packed_bytes"] == 22_544_384
    prog, out_buf, names = programs.mlp_program(mats["gate"], mats["up"], mats["down"], H, I)
    ws = torch.empty(prog.workspace_bytes(M), dtype=torch.uint8, device="cuda")
    x0 = torch.from_numpy(synth.activations(M, H, 2, M)).to(torch.float16).cuda()
    out = torch.empty((M, H), dtype=torch.float16, device="cuda")
    aq.aq_stack_forward(prog, x0, out, out_buf, M, ws)
    aq.aq_check()
    check_program(prog, names, ws, M, torch.float16, quant)


def test_bad_programs_are_rejected(aq):
    from paper_2605_24011_b200 import programs
    W = torch.from_numpy(synth.weights(64, 64, 3)).cuda()
    h = aq.aq_pack(4, 32, W)
    ops = [{"w": h, "src": 0, "dst": 1}]
    assert aq.Program([64, 64], ops).workspace_bytes(1) > 0
    assert aq.Program([64, 32], ops).workspace_bytes(1) == 0          # width mismatch
    assert aq.Program([64, 64], [{"w": h, "src": 1, "dst": 1}]).workspace_bytes(1) == 0   # reads unwritten
    assert aq.Program([64, 64], ops).workspace_bytes(0) == 0
    assert aq.Program([64, 64], ops).workspace_bytes(aq.AQ_MAX_M + 1) == 0
    h.free()
