"""aq_allocate_bits (host entry point of libaq, no GPU needed) against the oracle's greedy solver of Eq. 6:
the chosen bit-widths are integers decided by binary64 comparisons that both sides evaluate with the same
operations in the same order, so they must be equal everywhere."""
import numpy as np
import pytest

from oracle import stage1_oracle as S1
from paper_2605_24011_b200 import synth


@pytest.fixture(scope="module")
def aq():
    from paper_2605_24011_b200 import aq as mod
    return mod


def _stack(layer, n_layers):
    numel = np.array([N * K for (_, N, K) in layer] * n_layers, dtype=np.int64)
    layer_of = np.repeat(np.arange(n_layers), len(layer)).astype(np.int32)
    return numel, layer_of


@pytest.mark.parametrize("budget", (2.0, 2.25, 2.5, 3.0, 3.5, 4.0))
def test_allocation_equals_oracle_on_the_7b_stack(aq, budget):
    numel, layer_of = _stack(synth.llama7b_layer(), 32)
    S = synth.sensitivities(32, 7, 1)
    bits, obj = aq.aq_allocate_bits(S, numel, layer_of, [2, 3, 4], budget)
    ref, _ = S1.allocate_bits(S, numel, layer_of, [2, 3, 4], budget)
    assert np.array_equal(bits, ref)
    assert S1.mean_bits(bits, numel) <= budget
    assert obj == pytest.approx(S1.objective(S, ref, layer_of), rel=1e-13)


@pytest.mark.parametrize("seed", range(12))
def test_allocation_equals_oracle_on_random_problems(aq, seed):
    g = np.random.default_rng(seed)
    n_layers, per = int(g.integers(1, 9)), int(g.integers(1, 8))
    n = n_layers * per
    S = synth.sensitivities(n_layers, per, 2, seed)
    numel = g.integers(1, 5000, n).astype(np.int64) * 32
    layer_of = g.permutation(np.repeat(np.arange(n_layers), per)).astype(np.int32)
    types = [[2, 3, 4], [2, 4], [3, 4, 6, 8], [4]][seed % 4]
    budget = float(types[0] + g.random() * (types[-1] - types[0] + 0.2))
    bits, _ = aq.aq_allocate_bits(S, numel, layer_of, types, budget)
    ref, _ = S1.allocate_bits(S, numel, layer_of, types, budget)
    assert np.array_equal(bits, ref)


def test_allocation_errors(aq):
    S, numel, layer_of = [1.0, 2.0], [32, 32], [0, 1]
    with pytest.raises(aq.AqError) as e:
        aq.aq_allocate_bits(S, numel, layer_of, [2, 3, 4], 1.5)
    assert e.value.status == aq.AQ_ERR_RANGE
    for bad in (dict(types=[3, 2]), dict(types=[2, 2]), dict(numel=[32, 0]), dict(layer_of=[0, -1]), dict(S=[1.0, float("nan")])):
        kw = dict(S=S, numel=numel, layer_of=layer_of, types=[2, 3, 4])
        kw.update(bad)
        with pytest.raises(aq.AqError) as e:
            aq.aq_allocate_bits(kw["S"], kw["numel"], kw["layer_of"], kw["types"], 3.0)
        assert e.value.status == aq.AQ_ERR_INVALID_ARG
