"""Builders for the benchmark / full-size test workloads: seeded synthetic
weights generated on the GPU, packed through the C ABI, wired into programs.

Only plumbing lives here (generate, pack, free, wire).  For full-size stacks
the float32 weights exist on the device one matrix at a time; a few rows per
matrix can be copied to the host before the matrix is freed so that a CPU
check can re-quantise exactly those rows.
"""
from __future__ import annotations

import numpy as np

from . import aq, programs, synth


def _flat(key):
    for k in key:
        if isinstance(k, (tuple, list)):
            yield from _flat(k)
        else:
            yield int(k) & 0xFFFFFFFF


def _seed(*key) -> int:
    return int(np.random.SeedSequence(list(_flat(key))).generate_state(1)[0])


def build_stack(layer_shapes, n_layers, bits, key, outliers=False, sample_rows=0, device="cuda", full_layers=()):
    """Pack n_layers blocks.  bits: one width per matrix, in order.
    Returns (layers, samples, stats): layers for programs.block_program;
    samples[(layer, name)] = (row indices, float32 rows, bits) when sample_rows > 0; for the layers
    listed in full_layers every row is kept."""
    import torch
    layers, samples = [], {}
    weights = packed = device_bytes = 0
    i = 0
    rs = np.random.default_rng(_seed(0x5A, key))
    for l in range(n_layers):
        L = {"shape": {}}
        for (name, N, K) in layer_shapes:
            W = synth.weights_device(N, K, _seed(key, l, i), outliers=outliers, device=device)
            if sample_rows:
                rows = np.sort(rs.choice(N, size=min(sample_rows, N), replace=False))
                if l in full_layers:
                    rows = np.arange(N)
                samples[(l, name)] = (rows, W[torch.from_numpy(rows).to(device)].cpu().numpy(), bits[i])
            h = aq.aq_pack(bits[i], 32, W)
            torch.cuda.current_stream().synchronize()
            del W
            L[name] = h
            L["shape"][name] = (N, K)
            weights += N * K
            packed += N * K * (bits[i] + 1) // 8
            i += 1
        layers.append(L)
    info = {"weights": weights, "packed_bytes": packed,
            "mean_code_bits": float(sum(b * N * K for b, (_, _, N, K) in zip(bits, synth.stack_shapes(layer_shapes, n_layers))) / weights)}
    return layers, samples, info


def llama7b_decode_stack(n_layers=32, seed=0, sample_rows=0, full_layers=()):
    """The 7B-class decoder linear stack: per-matrix widths from {2,3,4} with a
    parameter-weighted mean of 2.5 bits, N(0,0.02) weights with 0.1 % x20 outliers."""
    shapes = synth.llama7b_layer()
    sizes = [N * K for (_, _, N, K) in synth.stack_shapes(shapes, n_layers)]
    bits = synth.draw_bits(sizes, 2.5, seed)
    layers, samples, info = build_stack(shapes, n_layers, bits, (3, seed), outliers=True, sample_rows=sample_rows,
                                        full_layers=full_layers)
    prog, out_buf, names = programs.block_program(layers)
    info["bits"] = bits
    info["layers"] = layers   # the packed matrices, for other wirings of the same stack (programs.independent_program)
    return prog, out_buf, names, samples, info


def gemma2b_stack(n_layers=18, seed=0, sample_rows=0):
    shapes = synth.gemma2b_layer()
    sizes = [N * K for (_, _, N, K) in synth.stack_shapes(shapes, n_layers)]
    bits = synth.draw_bits(sizes, 3.0, seed)
    layers, samples, info = build_stack(shapes, n_layers, bits, (5, seed), sample_rows=sample_rows)
    prog, out_buf, names = programs.block_program(layers)
    info["bits"] = bits
    return prog, out_buf, names, samples, info


def expert_stack(n_layers=18, seed=0, sample_rows=0):
    shapes = synth.expert_layer()
    bits = [4] * (n_layers * len(shapes))
    layers, samples, info = build_stack(shapes, n_layers, bits, (6, seed), sample_rows=sample_rows)
    prog, out_buf, names = programs.block_program(layers)
    info["bits"] = bits
    return prog, out_buf, names, samples, info


def activations_device(M, K, dtype, *key, kind="normal"):
    import torch
    return torch.from_numpy(synth.activations(M, K, *key, kind=kind)).to(dtype).cuda()
