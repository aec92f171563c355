"""Failure detection of the whole-program decode kernel, exercised on a healthy GPU: a table built with the testing
hook `aq_debug_decode_hold` makes the first phase that reads another op's output wait for one contribution more than
will ever arrive.  Every CTA's wait must run out after the (shortened) limit, the kernel must drain and return with the
context intact, `aq_check` must report AQ_ERR_TIMEOUT exactly once, and the next ordinary call on the same handles and
workspace must pass parity.  Nothing here traps, faults or spins without bound."""
import time

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


@pytest.mark.parametrize("M", (1, 4))
def test_bounded_wait_runs_out_and_the_next_call_is_clean(aq, M):
    from paper_2605_24011_b200 import programs
    shapes = synth.tiny_layer(256, 416)
    layers, quant = [], {}
    for l in range(2):
        L = {"shape": {}}
        for i, (name, N, K) in enumerate(shapes):
            W = synth.weights(N, K, 55, l, i)
            b = (2, 3, 4)[(l + i) % 3]
            L[name] = aq.aq_pack(b, 32, torch.from_numpy(W).cuda())
            L["shape"][name] = (N, K)
            quant[(l, name)] = O.quantize(W, b)
        layers.append(L)
    prog, out_buf, names = programs.block_program(layers)
    ws = torch.empty(prog.workspace_bytes(M), dtype=torch.uint8, device="cuda")
    x0 = torch.from_numpy(synth.activations(M, 256, 55, M)).to(torch.float16).cuda()
    out = torch.empty((M, 256), dtype=torch.float16, device="cuda")
    aq.aq_check()                                     # nothing pending from earlier tests
    try:
        aq.aq_set_wait_limit_ns(5_000_000)            # 5 ms instead of 2 s
        aq.aq_debug_decode_hold(True)
        t0 = time.time()
        aq.aq_stack_forward(prog, x0, out, out_buf, M, ws)
        with pytest.raises(aq.AqError) as err:
            aq.aq_check()
        took = time.time() - t0
        assert err.value.status == aq.AQ_ERR_TIMEOUT
        assert took < 1.5, f"the kernel took {took:.2f} s to give up on a 5 ms limit"
        aq.aq_check()                                 # the record was cleared: no second report
    finally:
        aq.aq_debug_decode_hold(False)
        aq.aq_set_wait_limit_ns(0)
    # the context is intact and the same handles and workspace give a correct pass
    aq.aq_stack_forward(prog, x0, out, out_buf, M, ws)
    aq.aq_check()
    check_program(prog, names, ws, M, torch.float16, quant)
    assert bool(torch.isfinite(out.float()).all())
