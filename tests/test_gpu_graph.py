"""aq_stack_forward recorded into a CUDA graph and replayed: every replay must pass the same per-op parity against
the oracle as an eager call (a replay runs with the arguments of the recording, so nothing in the library may depend on
per-launch host state), on the decode path (one cooperative kernel) and on the prefill path (grouped tensor-core launches)."""
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


@pytest.mark.parametrize("M,dtype", [(1, "f16"), (8, "f16"), (50, "bf16"), (300, "bf16"), (600, "bf16")])
def test_replayed_stack_matches_oracle(aq, M, dtype):
    from paper_2605_24011_b200 import programs
    tdt = torch.float16 if dtype == "f16" else torch.bfloat16
    shapes = synth.tiny_layer(256, 416)
    sizes = [N * K for _ in range(2) for (_, N, K) in shapes]
    bits = synth.draw_bits(sizes, 3.0, 6)
    layers, quant, i = [], {}, 0
    for l in range(2):
        L = {"shape": {}}
        for (name, N, K) in shapes:
            W = synth.weights(N, K, 41, l, i, outliers=True)
            L[name] = aq.aq_pack(bits[i], 32, torch.from_numpy(W).cuda())
            L["shape"][name] = (N, K)
            quant[(l, name)] = O.quantize(W, bits[i])
            i += 1
        layers.append(L)
    prog, out_buf, names = programs.block_program(layers)
    ws = torch.zeros(prog.workspace_bytes(M), dtype=torch.uint8, device="cuda")
    x0 = torch.from_numpy(synth.activations(M, 256, 41, M)).to(tdt).cuda()
    out = torch.empty((M, 256), dtype=tdt, device="cuda")
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(stream):
        aq.aq_stack_forward(prog, x0, out, out_buf, M, ws)      # eager: builds the library's cached tables
        aq.aq_check(stream)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            aq.aq_stack_forward(prog, x0, out, out_buf, M, ws)
    for rep in range(3):
        x_new = torch.from_numpy(synth.activations(M, 256, 42 + rep, M)).to(tdt).cuda()
        x0.copy_(x_new)
        ws.zero_()
        out.zero_()
        graph.replay()
        torch.cuda.synchronize()
        aq.aq_check()
        check_program(prog, names, ws, M, tdt, quant)
        assert torch.equal(aq.stack_buffer(prog, ws, M, 0), x_new.float())
        assert torch.equal(out, aq.stack_buffer(prog, ws, M, out_buf).to(tdt))
