"""Seeded random operator DAGs in the manner of the paper's graph construction (Algorithm 1).

A graph grows one operator at a time from an initial input node; after each growth step the
data flow is checked (operator must fit the shape of its operands, §3.2) and an invalid step is
rolled back and redrawn.  Topological diversity comes from letting a binary operator take, with
probability one half, an earlier node of matching shape as its second operand (a random
connection / path merge) instead of a fresh input.  Operators are drawn uniformly from eleven
names; the number of operators is uniform on 3..8.

Only text and sampling laws are produced here; no operator is evaluated.
"""
from __future__ import annotations

import math

from . import tensors

OPS = ("add", "mul", "relu", "gelu", "sigmoid", "exp", "broadcast_bias", "row_softmax", "row_layernorm", "row_sum", "gemm")
ROWS = (1024, 4096, 16384)
COLS = (256, 1024, 4096)
GEMM_N = (1024, 4096)


class _Draws:
    def __init__(self, seed, attempt):
        self.u = tensors.uniform(seed, 1000 + attempt, 256)
        self.i = 0

    def next(self):
        v = self.u[self.i]
        self.i += 1
        return v

    def choice(self, seq):
        return seq[min(int(self.next() * len(seq)), len(seq) - 1)]


def make_dag(seed: int, attempt: int = 0, rows: int | None = None):
    """Returns (spec_text, laws, meta).  ``rows`` overrides the drawn row count (same graph, fewer rows)."""
    d = _Draws(seed, attempt)
    n_ops = 3 + min(int(d.next() * 6), 5)
    r_drawn = d.choice(ROWS)
    c = d.choice(COLS)
    r = rows if rows is not None else r_drawn
    lines = ["hct 1", f"input x0 f32 [{r},{c}]"]
    laws = {"x0": {"kind": "normal", "mean": 0.0, "std": 1.0}}
    nodes = [("x0", (r, c))]   # every tensor a later binary op may connect to
    cur, cur_shape = "x0", (r, c)
    n_in, n_node, rollbacks = 1, 0, 0
    body = []

    def fresh(shape, law):
        nonlocal n_in
        name = f"x{n_in}"
        n_in += 1
        lines.append(f"input {name} f32 [{','.join(str(s) for s in shape)}]")
        laws[name] = law
        return name

    std_normal = {"kind": "normal", "mean": 0.0, "std": 1.0}
    made = 0
    while made < n_ops:
        op = d.choice(OPS)
        full = cur_shape[1] > 1
        # data-flow validity: row operators and GEMM need a full-width [R,C] operand
        if op in ("row_softmax", "row_layernorm", "row_sum", "gemm", "broadcast_bias") and not full:
            rollbacks += 1
            continue
        name = f"n{n_node}"
        if op in ("relu", "sigmoid", "exp"):
            body.append(f"node {name} = {op}({cur})")
            shape = cur_shape
        elif op == "gelu":
            body.append(f"node {name} = gelu_tanh({cur})")
            shape = cur_shape
        elif op in ("add", "mul"):
            other = None
            if d.next() < 0.5:
                cands = [n for n, s in nodes if s == cur_shape and n != cur]
                if cands:
                    other = d.choice(cands)
            if other is None:
                other = fresh(cur_shape, std_normal)
                nodes.append((other, cur_shape))
            body.append(f"node {name} = {op}({cur}, {other})")
            shape = cur_shape
        elif op == "broadcast_bias":
            bias = fresh((cur_shape[1],), std_normal)
            body.append(f"node {name} = add({cur}, {bias})")
            shape = cur_shape
        elif op == "row_softmax":
            body.append(f"node {name} = row_softmax({cur})")
            shape = cur_shape
        elif op == "row_layernorm":
            ga = fresh((cur_shape[1],), {"kind": "normal", "mean": 1.0, "std": 0.1})
            be = fresh((cur_shape[1],), {"kind": "normal", "mean": 0.0, "std": 0.1})
            body.append(f"node {name} = row_layernorm({cur}, {ga}, {be}, eps=1e-5)")
            shape = cur_shape
        elif op == "row_sum":
            body.append(f"node {name} = row_sum({cur})")
            shape = (cur_shape[0], 1)
        else:  # gemm: K = current columns, N drawn, weight ~ N(0, 1/K)
            n_out = d.choice(GEMM_N)
            k = cur_shape[1]
            w = fresh((k, n_out), {"kind": "normal", "mean": 0.0, "std": 1.0 / math.sqrt(k)})
            body.append(f"node {name} = gemm({cur}, {w})")
            shape = (cur_shape[0], n_out)
        n_node += 1
        made += 1
        cur, cur_shape = name, shape
        nodes.append((name, shape))
    lines += body
    lines.append(f"output {cur} f32")
    meta = {"seed": seed, "attempt": attempt, "rows": r_drawn, "cols": c, "n_ops": n_ops, "rollbacks": rollbacks}
    return "\n".join(lines) + "\n", laws, meta
