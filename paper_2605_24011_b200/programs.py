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


def block_program_attn(layers, n_heads, n_kv_heads):
    """block_program with the attention in its place: W_o reads a buffer that the attention step of
    aq_stack_forward_attn fills from q, k, v and the caches.  Returns (Program, out_buf, op_names, attn), attn being
    the list of attention steps without their caches (keys after_op, q_buf, k_buf, v_buf, dst_buf, n_heads, n_kv_heads)."""
    first = layers[0]["shape"]
    widths = [first["q"][1]]
    ops, names, attn = [], [], []
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
        ba = new_buf(sh["q"][0])                      # the attention's output: no op writes it
        attn.append({"after_op": len(ops) - 1, "q_buf": bq, "k_buf": bk, "v_buf": bv, "dst_buf": ba, "n_heads": n_heads,
                     "n_kv_heads": n_kv_heads})
        h1 = new_buf(sh["o"][0])
        ops.append({"w": L["o"], "src": ba, "dst": h1, "in_op": aq.AQ_IN_PLAIN, "out_op": aq.AQ_OUT_ADD, "res": h})
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
    return aq.Program(widths, ops), h, names, attn


def mlp_program(gate, up, down, hidden, inter):
    """gate/up -> silu*up -> down, no norm and no residual (a bare MLP block)."""
    widths = [hidden, inter, inter, hidden]
    ops = [
        {"w": gate, "src": 0, "dst": 1, "in_op": aq.AQ_IN_PLAIN},
        {"w": up, "src": 0, "dst": 2, "in_op": aq.AQ_IN_PLAIN},
        {"w": down, "src": 1, "src2": 2, "dst": 3, "in_op": aq.AQ_IN_SILU_MUL},
    ]
    return aq.Program(widths, ops), 3, [(0, "gate"), (0, "up"), (0, "down")]


def independent_program(layers):
    """The same matrices without the chain: every linear whose K equals the input width reads the program input as it
    is; the others read the first block's outputs of that width (o: q; down: silu(gate) * up).  Nothing is normalised
    or added and every output goes to a buffer of its own, so after the first block nothing waits for anything: the
    streaming upper bound of the chained program.  Ops that share an input and sit together form one phase; the order
    keeps phases at three matrices: gate up q | down | k v o in the first block, q k v | down | o gate up after it.
    Returns (Program, out_buf, op_names)."""
    hidden = layers[0]["shape"]["q"][1]
    widths = [hidden]
    ops, names = [], []
    first = {}   # name -> output buffer of that matrix in the first block

    def new_buf(w):
        widths.append(w)
        return len(widths) - 1

    for li, L in enumerate(layers):
        sh = L["shape"]
        order = ("gate", "up", "q", "down", "k", "v", "o") if li == 0 else ("q", "k", "v", "down", "o", "gate", "up")
        for nm in order:
            N, K = sh[nm]
            op = {"w": L[nm], "dst": new_buf(N), "in_op": aq.AQ_IN_PLAIN, "src": 0}
            if nm == "down":
                op.update({"src": first["gate"], "src2": first["up"], "in_op": aq.AQ_IN_SILU_MUL})
            elif K != hidden:
                op["src"] = first["q"]
            ops.append(op)
            names.append((li, nm))
            first.setdefault(nm, op["dst"])
    return aq.Program(widths, ops), ops[-1]["dst"], names
