"""Wiring of transformer-block linears into an aq_stack_t program.

No arithmetic lives here: the module lists which packed matrix reads which
activation buffer.  Per block (Section 3: W_Q, W_K, W_V, W_O, W_gate, W_up,
W_down), with h the residual stream:

    q, k, v = W_{q,k,v} rmsnorm(h)         (k, v are written out as a KV-cache
                                            write would be; attention itself is
                                            outside this library and q stands in
                                            for its output)
    h1 = h + W_o q
    g, u = W_{gate,up} rmsnorm(h1)
    h2 = h1 + W_down (silu(g) * u)
"""
from __future__ import annotations

from . import aq

ORDER = ("q", "k", "v", "o", "gate", "up", "down")


def block_program(layers):
    """layers: list of dicts name -> Handle with keys q,k,v,o,gate,up,down and
    'shape' name -> (N, K).  Returns (Program, out_buf, op_names)."""
    first = layers[0]["shape"]
    widths = [first["q"][1]]          # buffer 0: the input residual stream
    ops, names = [], []
    h = 0

    def new_buf(w):
        widths.append(w)
        return len(widths) - 1

    for li, L in enumerate(layers):
        sh = L["shape"]
        bq, bk, bv = new_buf(sh["q"][0]), new_buf(sh["k"][0]), new_buf(sh["v"][0])
        for nm, b in (("q", bq), ("k", bk), ("v", bv)):
            ops.append({"w": L[nm], "src": h, "dst": b, "in_op": aq.AQ_IN_RMSNORM})
            names.append((li, nm))
        h1 = new_buf(sh["o"][0])
        ops.append({"w": L["o"], "src": bq, "dst": h1, "in_op": aq.AQ_IN_PLAIN, "out_op": aq.AQ_OUT_ADD, "res": h})
        names.append((li, "o"))
        bg, bu = new_buf(sh["gate"][0]), new_buf(sh["up"][0])
        for nm, b in (("gate", bg), ("up", bu)):
            ops.append({"w": L[nm], "src": h1, "dst": b, "in_op": aq.AQ_IN_RMSNORM})
            names.append((li, nm))
        h2 = new_buf(sh["down"][0])
        ops.append({"w": L["down"], "src": bg, "src2": bu, "dst": h2, "in_op": aq.AQ_IN_SILU_MUL,
                    "out_op": aq.AQ_OUT_ADD, "res": h1})
        names.append((li, "down"))
        h = h2
    return aq.Program(widths, ops), h, names


def mlp_program(gate, up, down, hidden, inter):
    """gate/up -> silu*up -> down, no norm and no residual (a bare MLP block)."""
    widths = [hidden, inter, inter, hidden]
    ops = [
        {"w": gate, "src": 0, "dst": 1, "in_op": aq.AQ_IN_PLAIN},
        {"w": up, "src": 0, "dst": 2, "in_op": aq.AQ_IN_PLAIN},
        {"w": down, "src": 1, "src2": 2, "dst": 3, "in_op": aq.AQ_IN_SILU_MUL},
    ]
    return aq.Program(widths, ops), 3, [(0, "gate"), (0, "up"), (0, "down")]
