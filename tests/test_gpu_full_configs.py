"""The full-size workloads, in the launch configuration the benchmark times, checked
on sampled outputs: for every matrix of the stack a seeded sample of its rows is kept
when it is packed, the oracle re-quantises exactly those rows, and the matching output
columns of every op are compared (teacher-forced, all or sampled token rows)."""
import numpy as np
import pytest

from oracle import aq_oracle as O
from stack_check import check_program

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def aq():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2605_24011_b200 import aq as mod
    return mod


def _sampled(samples):
    cache = {}

    def quantised(layer, name, cols):
        key = (layer, name)
        if key not in cache:
            rows, W, bits = samples[key]
            cache[key] = O.quantize(np.ascontiguousarray(W), bits)
        return cache[key]

    def cols_of(layer, name):
        return samples[(layer, name)][0]

    return quantised, cols_of


def _token_rows(M, n, seed):
    if M <= n:
        return list(range(M))
    fixed = {0, M - 1, min(255, M - 1), min(256, M - 1)}
    rng = np.random.default_rng(seed)
    while len(fixed) < n:
        fixed.add(int(rng.integers(0, M)))
    return sorted(fixed)


def _run(aq, prog, out_buf, names, samples, M, dtype, width, key, kind="normal", token_rows=32):
    from paper_2605_24011_b200 import workloads
    ws = torch.empty(prog.workspace_bytes(M), dtype=torch.uint8, device="cuda")
    x0 = workloads.activations_device(M, width, dtype, *key, kind=kind)
    out = torch.empty((M, width), dtype=dtype, device="cuda")
    aq.aq_stack_forward(prog, x0, out, out_buf, M, ws)
    aq.aq_check()
    quantised, cols_of = _sampled(samples)
    worst, worst_in = check_program(prog, names, ws, M, dtype, quantised, rows=_token_rows(M, token_rows, 11), cols_of=cols_of)
    assert bool(torch.isfinite(out.float()).all())
    return worst, worst_in


def test_config3_full_7b_decode_stack(aq):
    """32 layers x {q,k,v,o,gate,up,down}, per-matrix 2/3/4-bit (mean 2.5), 0.1% x20 outliers, M = 1 and 8, fp16.
    Every output of the first and of the last layer is checked (all 4096 / 11008 rows of their matrices: a unit dealt
    to the wrong CTA or op would show there), 48 sampled rows per matrix in between.  The oracle re-quantises
    2 x 202 M weights for this: the test takes about twenty seconds."""
    from paper_2605_24011_b200 import workloads
    prog, out_buf, names, samples, info = workloads.llama7b_decode_stack(n_layers=32, seed=0, sample_rows=48, full_layers=(0, 31))
    assert abs(info["mean_code_bits"] - 2.5) <= 0.005
    assert info["weights"] == 6_476_005_376
    _run(aq, prog, out_buf, names, samples, 1, torch.float16, 4096, (3, 0))
    _run(aq, prog, out_buf, names, samples, 8, torch.float16, 4096, (3, 8))


def test_config4_full_7b_prefill_stack(aq):
    """The same stack at M = 512: 256 vision-like rows + 256 text rows, bf16."""
    from paper_2605_24011_b200 import workloads
    prog, out_buf, names, samples, info = workloads.llama7b_decode_stack(n_layers=32, seed=0, sample_rows=32)
    _run(aq, prog, out_buf, names, samples, 512, torch.bfloat16, 4096, (4, 0), kind="vision_text")


def test_config5_gemma_backbone_and_expert(aq):
    """Gemma-2B-shaped backbone (mean 3.0 bits) at M = 768 bf16, then the 4-bit action expert at M = 50."""
    from paper_2605_24011_b200 import workloads
    prog, out_buf, names, samples, info = workloads.gemma2b_stack(n_layers=18, seed=0, sample_rows=32)
    assert abs(info["mean_code_bits"] - 3.0) <= 0.005
    assert info["weights"] == 1_981_808_640
    _run(aq, prog, out_buf, names, samples, 768, torch.bfloat16, 2048, (5, 0))
    del prog
    prog, out_buf, names, samples, info = workloads.expert_stack(n_layers=18, seed=0, sample_rows=32)
    assert info["weights"] == 311_427_072
    for step in range(2):   # flow-matching steps run the same program on new activations
        _run(aq, prog, out_buf, names, samples, 50, torch.bfloat16, 1024, (6, step))
