"""Per-op, teacher-forced check of an aq_stack_forward run against the oracle.

For every op the oracle (1) re-forms the input vector from the GPU's float32
source buffers in float64 and compares it with the rounded vector the GPU
actually staged, then (2) applies the linear to that staged vector and
compares with the GPU's output buffer under the per-element bound
|dy| <= 2e-3 * sum|x w| + 1e-5.  Errors therefore do not compound.
"""
import numpy as np
import torch

from oracle import aq_oracle as O
from paper_2605_24011_b200 import aq


def check_program(prog, names, ws, M, dtype, quantised, rows=None, cols_sample=None, rng=None, cols_of=None):
    """quantised: dict (layer, name) -> (d, m, q) oracle codes of that matrix,
    or a callable (layer, name, row_idx) -> (d, m, q) restricted to rows.
    rows: token rows to check (default all).  cols_sample: number of output
    columns to sample per op (default all); cols_of(layer, name) gives the output
    columns to check instead (the rows of W that were kept at packing time).
    Returns worst normalised error."""
    ulp = 2.0 ** -10 if dtype == torch.float16 else 2.0 ** -7
    tiny = 2.0 ** -24 if dtype == torch.float16 else 1e-37     # spacing of binary16 subnormals
    rows = list(range(M)) if rows is None else rows
    worst = 0.0
    worst_in = 0.0
    for i, op in enumerate(prog.ops):
        src = aq.stack_buffer(prog, ws, M, op["src"]).double().cpu().numpy()[rows]
        in_op = op.get("in_op", aq.AQ_IN_PLAIN)
        if in_op == aq.AQ_IN_RMSNORM:
            want = src * O.rms_scale(src)
            tol = ulp * np.abs(want) + 4e-7 * np.abs(want) + tiny
        elif in_op == aq.AQ_IN_SILU_MUL:
            src2 = aq.stack_buffer(prog, ws, M, op["src2"]).double().cpu().numpy()[rows]
            want = O.silu_mul(src, src2)
            # fp32 expf / divide / multiply: a few ulp of binary32 before the rounding to half
            tol = ulp * np.abs(want) + 2e-6 * np.abs(want) + tiny
        else:
            want = src
            tol = ulp * np.abs(want) + tiny
        x_gpu = aq.stack_input(prog, ws, M, i, dtype).double().cpu().numpy()[rows]
        err_in = np.abs(x_gpu - want) / tol
        worst_in = max(worst_in, float(err_in.max()))
        assert err_in.max() <= 1.0, f"op {i} {names[i]}: staged input off by {err_in.max():.2f} tolerances"

        key = names[i]
        N = prog.buf_width[op["dst"]]
        if cols_of is not None:
            cols = np.asarray(cols_of(key[0], key[1]))
        elif cols_sample is not None and cols_sample < N:
            cols = np.sort(rng.choice(N, size=cols_sample, replace=False))
        else:
            cols = np.arange(N)
        d, m, q = quantised(key[0], key[1], cols) if callable(quantised) else tuple(a[cols] for a in quantised[key])
        y, T = O.linear(d, m, q, x_gpu)
        dst = aq.stack_buffer(prog, ws, M, op["dst"]).double().cpu().numpy()[rows][:, cols]
        slack = 0.0
        if op.get("out_op", aq.AQ_OUT_STORE) == aq.AQ_OUT_ADD:
            res = aq.stack_buffer(prog, ws, M, op["res"]).double().cpu().numpy()[rows][:, cols]
            y = y + res
            slack = 2.0 ** -22 * (np.abs(res) + np.abs(y))     # the float32 additions into the residual
        ex = np.abs(dst - y) / (2e-3 * T + 1e-5 + slack)
        worst = max(worst, float(ex.max()))
        assert ex.max() <= 1.0, f"op {i} {names[i]}: worst normalised error {ex.max():.3f}"
    return worst, worst_in
