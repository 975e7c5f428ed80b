"""Seeded operator DAGs grown with every step of the paper's graph construction (Algorithm 1).

Where ``random_dag`` keeps the algorithm's validity check and a minimal form of its random
connections, this generator follows its whole loop and yields branching graphs with several
outputs.  One round of the loop:

  1. candidate node expansion: a non-empty random subset of the current tips (nodes nobody
     consumes yet) each receive a new operator node.  The operator is drawn among those of the
     pool whose use count in this graph is still below ``ceil(P_op * |pool|)`` (the usage cap);
  2. one of three actions, chosen at random, adds topological diversity:
       (a) random connection: a fresh-input operand of an existing binary node n_j is rewired to an
           earlier computed node n_i of the same shape; n_j is drawn with probability proportional
           to one plus its number of computed operands (in-degree, smoothed so that nodes fed only
           by inputs can be chosen at all),
       (b) branch: one node receives two new consumers,
       (c) merge: all tips of one shape are folded into a single node by additions;
  3. data-flow validity: an operator that does not fit its operand's shape is rolled back and
     redrawn; nodes are only ever wired to earlier nodes, so the graph stays acyclic; every tip
     left at the end becomes an output, so no computed node dangles.

The loop ends once the graph has more than ``N_max`` operator nodes or is deeper than ``D_max``.
Only text and sampling laws are produced here; no operator is evaluated.
"""
from __future__ import annotations

import math

from . import tensors

UNARY = ("relu", "gelu_tanh", "sigmoid", "tanh", "exp", "abs")
BINARY = ("add", "sub", "mul", "max")
ROW = ("row_softmax", "row_layernorm", "row_sum", "row_max")
ORDER = ("row_sort", "row_topk")          # logic-intensive operators
POOL = UNARY + BINARY + ("broadcast_bias",) + ROW + ORDER + ("gemm",)
COLS = (128, 512, 2048)
GEMM_N = (256, 1024)
ROWS = (1024, 4096)
MAX_OUTPUTS = 3

_STD = {"kind": "normal", "mean": 0.0, "std": 1.0}


class _Draws:
    def __init__(self, seed, attempt):
        self.u = tensors.uniform(seed, 2000 + attempt, 4096)
        self.i = 0

    def next(self):
        v = self.u[self.i % len(self.u)]
        self.i += 1
        return float(v)

    def below(self, n):
        return min(int(self.next() * n), n - 1)

    def choice(self, seq):
        return seq[self.below(len(seq))]

    def weighted(self, seq, weights):
        x = self.next() * sum(weights)
        for item, wgt in zip(seq, weights):
            x -= wgt
            if x < 0:
                return item
        return seq[-1]


class _Node:
    def __init__(self, name, op, args, shape, depth, attrs=""):
        self.name, self.op, self.args, self.shape, self.depth, self.attrs = name, op, list(args), shape, depth, attrs
        self.fresh = []      # positions in args that hold an input created for this node alone (same shape as the node)


def grow_graph(seed: int, attempt: int = 0, rows: int | None = None, p_op: float = 0.25):
    """Returns (spec_text, laws, meta).  ``rows`` overrides the drawn row count (same graph, fewer rows)."""
    d = _Draws(seed, attempt)
    n_max = 6 + d.below(9)          # 6..14 operator nodes
    d_max = 4 + d.below(5)          # depth 4..8
    r_drawn = d.choice(ROWS)
    c0 = d.choice(COLS)
    r = rows if rows is not None else r_drawn
    cap = math.ceil(p_op * len(POOL))
    usage = {op: 0 for op in POOL}
    inputs = {"x0": ((r, c0), _STD)}    # name -> (shape, law); insertion order is the input order
    order = []                          # operator nodes in creation (= topological) order
    by_name = {}
    consumers = {"x0": 0}
    shapes = {"x0": (r, c0)}
    depth = {"x0": 0}
    counters = {"in": 1, "node": 0, "rollbacks": 0, "connections": 0, "branches": 0, "merges": 0}

    def fresh(shape, law):
        name = f"x{counters['in']}"
        counters["in"] += 1
        inputs[name] = (shape, law)
        shapes[name] = shape
        depth[name] = 0
        consumers[name] = 0
        return name

    def emit(op, args, shape, attrs=""):
        name = f"n{counters['node']}"
        counters["node"] += 1
        nd = _Node(name, op, args, shape, 1 + max(depth[a] for a in args), attrs)
        order.append(nd)
        by_name[name] = nd
        shapes[name], depth[name], consumers[name] = shape, nd.depth, 0
        for a in args:
            consumers[a] += 1
        return nd

    def expand(src):
        """Attach one operator node to ``src``; invalid draws are rolled back and redrawn."""
        shape = shapes[src]
        full = shape[1] > 1
        for _ in range(32):
            allowed = [op for op in POOL if usage[op] < cap]
            if not allowed:
                allowed = list(UNARY)
            op = d.choice(allowed)
            if op in ROW + ORDER + ("gemm", "broadcast_bias") and not full:
                counters["rollbacks"] += 1      # operator does not fit the operand's shape
                continue
            usage[op] += 1
            if op in UNARY:
                return emit(op, [src], shape)
            if op in BINARY:
                cols = [n.name for n in order if n.shape == (shape[0], 1) and n.name != src]
                if full and cols and d.next() < 0.25:
                    return emit(op, [src, d.choice(cols)], shape)       # column broadcast of an earlier reduction
                other = fresh(shape, _STD)
                nd = emit(op, [src, other], shape)
                nd.fresh.append(1)
                return nd
            if op == "broadcast_bias":
                return emit("add", [src, fresh((shape[1],), _STD)], shape)
            if op == "row_layernorm":
                ga = fresh((shape[1],), {"kind": "normal", "mean": 1.0, "std": 0.1})
                be = fresh((shape[1],), {"kind": "normal", "mean": 0.0, "std": 0.1})
                return emit(op, [src, ga, be], shape, ", eps=1e-5")
            if op == "row_softmax":
                return emit(op, [src], shape)
            if op in ("row_sum", "row_max"):
                return emit(op, [src], (shape[0], 1))
            if op == "row_sort":
                return emit(op, [src], shape, ", descending=1" if d.next() < 0.5 else "")
            if op == "row_topk":
                k = d.choice([kk for kk in (8, 32, 128) if kk < shape[1]] or [shape[1]])
                return emit(op, [src], (shape[0], k), f", k={k}")
            n_out = d.choice(GEMM_N)
            w = fresh((shape[1], n_out), {"kind": "normal", "mean": 0.0, "std": 1.0 / math.sqrt(shape[1])})
            return emit("gemm", [src, w], (shape[0], n_out))
        return emit("relu", [src], shape)

    def tips():
        t = [n.name for n in order if consumers[n.name] == 0]
        return t if t else ["x0"]

    def merge(names):
        acc = names[0]
        for other in names[1:]:
            acc = emit("add", [acc, other], shapes[acc]).name
        counters["merges"] += 1
        return acc

    while True:
        current = tips()
        chosen = [t for t in current if d.next() < 0.5] or [d.choice(current)]
        for t in chosen:
            expand(t)
        action = d.below(3)
        if action == 0:
            targets = [n for n in order if n.fresh]
            if targets:
                nj = d.weighted(targets, [1 + sum(a in by_name for a in n.args) for n in targets])
                idx = order.index(nj)
                cands = [n.name for n in order[:idx] if n.shape == nj.shape and n.name not in nj.args]
                if cands:
                    ni = d.choice(cands)
                    pos = nj.fresh.pop()
                    dropped = nj.args[pos]
                    nj.args[pos] = ni
                    consumers[ni] += 1
                    del inputs[dropped]
                    nj.depth = 1 + max(depth[a] for a in nj.args)
                    # depths downstream of n_j may have grown
                    for n in order[idx:]:
                        n.depth = 1 + max(depth[a] for a in n.args)
                        depth[n.name] = n.depth
                    counters["connections"] += 1
        elif action == 1 and order:
            src = d.choice(order).name
            expand(src)
            expand(src)
            counters["branches"] += 1
        elif action == 2:
            groups = {}
            for t in tips():
                groups.setdefault(shapes[t], []).append(t)
            multi = [g for g in groups.values() if len(g) > 1]
            if multi:
                merge(d.choice(multi))
        if len(order) > n_max or max(n.depth for n in order) > d_max:
            break

    # every remaining tip is an output; tips of one shape are merged first while there are too many
    while True:
        groups = {}
        for t in tips():
            groups.setdefault(shapes[t], []).append(t)
        if sum(len(g) for g in groups.values()) <= MAX_OUTPUTS:
            break
        multi = [g for g in groups.values() if len(g) > 1]
        if not multi:
            break
        merge(max(multi, key=len))
    outs = tips()

    lines = ["hct 1"]
    for name, (shape, _) in inputs.items():
        lines.append(f"input {name} f32 [{','.join(str(s) for s in shape)}]")
    for n in order:
        lines.append(f"node {n.name} = {n.op}({', '.join(n.args)}{n.attrs})")
    for o in outs:
        lines.append(f"output {o} f32")
    laws = {name: law for name, (_, law) in inputs.items()}
    meta = {"seed": seed, "attempt": attempt, "rows": r_drawn, "cols": c0, "n_nodes": len(order), "depth": max(n.depth for n in order),
            "n_max": n_max, "d_max": d_max, "outputs": len(outs), "usage_cap": cap, "max_usage": max(usage.values()),
            **{k: counters[k] for k in ("rollbacks", "connections", "branches", "merges")}}
    return "\n".join(lines) + "\n", laws, meta
