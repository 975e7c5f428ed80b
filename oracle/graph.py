"""Oracle-side reader of the operator-DAG spec text (test infrastructure only).

A computation graph is a DAG whose nodes are computations and whose edges are
data flow (paper §3.2).  This reader enforces the validity rules stated there:
every operand must already be defined (so the graph is acyclic and nothing
dangles), operator types must agree with operand shapes and dtypes, and every
node must reach an output.
"""
from __future__ import annotations

import re
from dataclasses import dataclass, field


class SpecError(ValueError):
    pass


UNARY = ("relu", "gelu_tanh", "gelu_erf", "sigmoid", "exp", "tanh", "sqrt", "sin", "cos", "neg", "abs", "log", "rsqrt", "square",
         "reciprocal")
BINARY = ("add", "sub", "mul", "div", "max", "min")
ROW_TO_ROW = ("row_softmax",)
ROW_TO_COL = ("row_sum", "row_mean", "row_max", "row_min", "row_argmax", "row_argmin")


@dataclass
class Node:
    name: str
    op: str            # "input" or an operator name
    args: list         # operand names (str) or float literals
    attrs: dict
    shape: tuple
    dtype: str         # storage dtype for inputs; "f32" for computed nodes


@dataclass
class Graph:
    nodes: dict = field(default_factory=dict)   # name -> Node, insertion order = evaluation order
    inputs: list = field(default_factory=list)
    outputs: list = field(default_factory=list)  # (name, dtype)
    output_layouts: dict = field(default_factory=dict)  # name -> "nhwc" for outputs declared channels-last


_NAME = re.compile(r"^[A-Za-z_][A-Za-z0-9_]*$")


def _broadcast(a, b, where):
    ra, rb = list(a), list(b)
    n = max(len(ra), len(rb))
    ra = [1] * (n - len(ra)) + ra
    rb = [1] * (n - len(rb)) + rb
    out = []
    for x, y in zip(ra, rb):
        if x == y or y == 1:
            out.append(x)
        elif x == 1:
            out.append(y)
        else:
            raise SpecError(f"{where}: shapes {tuple(a)} and {tuple(b)} do not broadcast")
    return tuple(out)


def _split_args(s, where):
    parts = [p.strip() for p in s.split(",")] if s.strip() else []
    pos, attrs = [], {}
    for p in parts:
        if not p:
            raise SpecError(f"{where}: empty argument")
        if "=" in p:
            k, v = (t.strip() for t in p.split("=", 1))
            attrs[k] = v
        else:
            if attrs:
                raise SpecError(f"{where}: positional argument after keyword")
            pos.append(p)
    return pos, attrs


def parse(text: str) -> Graph:
    g = Graph()
    lines = text.splitlines()
    seen_header = False
    for ln, raw in enumerate(lines, 1):
        line = raw.split("#", 1)[0].strip()
        if not line:
            continue
        where = f"line {ln}"
        if not seen_header:
            if line.split() != ["hct", "1"]:
                raise SpecError(f"{where}: expected header 'hct 1'")
            seen_header = True
            continue
        kw = line.split(None, 1)[0]
        if kw == "input":
            m = re.match(r"^input\s+(\S+)\s+(\S+)\s*\[([^\]]*)\]\s*(\S*)$", line)
            if not m:
                raise SpecError(f"{where}: malformed input")
            name, dtype, dims, layout = m.groups()
            if layout not in ("", "nchw", "nhwc"):
                raise SpecError(f"{where}: unknown layout {layout!r}")
            if not _NAME.match(name) or name in g.nodes:
                raise SpecError(f"{where}: bad or duplicate name {name!r}")
            if dtype not in ("f32", "bf16"):
                raise SpecError(f"{where}: unknown dtype {dtype!r}")
            try:
                shape = tuple(int(t) for t in dims.split(","))
            except ValueError:
                raise SpecError(f"{where}: malformed shape") from None
            if not 1 <= len(shape) <= 4 or any(d < 0 for d in shape):
                raise SpecError(f"{where}: rank must be 1..4 and extents non-negative")
            if layout == "nhwc" and (len(shape) != 4 or dtype != "bf16"):
                raise SpecError(f"{where}: nhwc needs a bf16 input of rank 4")
            # the layout word only says how the device buffer is ordered; values are always handed over as [N,C,H,W]
            g.nodes[name] = Node(name, "input", [], {"layout": layout or "nchw"}, shape, dtype)
            g.inputs.append(name)
        elif kw == "node":
            m = re.match(r"^node\s+(\S+)\s*=\s*([A-Za-z_0-9]+)\s*\((.*)\)$", line)
            if not m:
                raise SpecError(f"{where}: malformed node")
            name, op, argstr = m.groups()
            if not _NAME.match(name) or name in g.nodes:
                raise SpecError(f"{where}: bad or duplicate name {name!r}")
            pos, attrs = _split_args(argstr, where)
            g.nodes[name] = _infer(g, name, op, pos, attrs, where)
        elif kw == "output":
            toks = line.split()
            if len(toks) not in (2, 3, 4):
                raise SpecError(f"{where}: malformed output")
            name = toks[1]
            dtype = toks[2] if len(toks) >= 3 else "f32"
            layout = toks[3] if len(toks) == 4 else "nchw"
            if layout not in ("nchw", "nhwc"):
                raise SpecError(f"{where}: unknown layout {layout!r}")
            if name not in g.nodes:
                raise SpecError(f"{where}: output {name!r} is not defined")
            if dtype not in ("f32", "bf16"):
                raise SpecError(f"{where}: unknown dtype {dtype!r}")
            if g.nodes[name].op == "input":
                raise SpecError(f"{where}: an input cannot be an output")
            if name in [o for o, _ in g.outputs]:
                raise SpecError(f"{where}: duplicate output")
            if layout == "nhwc":
                if len(g.nodes[name].shape) != 4:
                    raise SpecError(f"{where}: nhwc needs an output of rank 4")
                g.output_layouts[name] = "nhwc"    # a matter of the caller's buffer only: values and extents stay [N,C,H,W]
            g.outputs.append((name, dtype))
        else:
            raise SpecError(f"{where}: unknown statement {kw!r}")
    if not seen_header:
        raise SpecError("empty spec")
    if not g.outputs:
        raise SpecError("no output")
    # a channels-last input may only be the activation operand of a convolution
    for node in g.nodes.values():
        for pos, a in enumerate(node.args):
            if isinstance(a, str) and g.nodes[a].attrs.get("layout") == "nhwc" and not (node.op == "conv2d" and pos == 0):
                raise SpecError(f"input {a!r} is declared nhwc and may only be the first operand of conv2d")
    # every node and every input must reach an output (no dangling nodes)
    live = set()
    stack = [o for o, _ in g.outputs]
    while stack:
        n = stack.pop()
        if n in live:
            continue
        live.add(n)
        stack.extend(a for a in g.nodes[n].args if isinstance(a, str))
    for n in g.nodes:
        if n not in live:
            raise SpecError(f"node {n!r} does not reach any output")
    return g


def _operand(g, tok, where, allow_literal):
    if tok in g.nodes:
        return tok
    try:
        v = float(tok)
    except ValueError:
        raise SpecError(f"{where}: operand {tok!r} is not defined") from None
    if not allow_literal:
        raise SpecError(f"{where}: literal not allowed here")
    return v


def _int_attr(attrs, key, default, where):
    if key not in attrs:
        return default
    try:
        return int(attrs[key])
    except ValueError:
        raise SpecError(f"{where}: attribute {key} must be an integer") from None


def _infer(g, name, op, pos, attrs, where):
    def shape_of(a):
        return g.nodes[a].shape

    def only_attrs(*allowed):
        for k in attrs:
            if k not in allowed:
                raise SpecError(f"{where}: unknown attribute {k!r} for {op}")

    if op == "cast_bf16":
        only_attrs()
        if len(pos) != 1:
            raise SpecError(f"{where}: cast_bf16 takes one operand")
        a = _operand(g, pos[0], where, False)
        return Node(name, op, [a], {}, shape_of(a), "bf16")
    if op == "dropout":
        only_attrs("p", "seed")
        if len(pos) != 1:
            raise SpecError(f"{where}: dropout takes one operand")
        a = _operand(g, pos[0], where, False)
        try:
            prob = float(attrs.get("p", "0.5"))
        except ValueError:
            raise SpecError(f"{where}: p must be a number") from None
        seed = _int_attr(attrs, "seed", 0, where)
        if not (0.0 <= prob < 1.0) or seed < 0 or round(prob * 1000.0) >= 1000:
            raise SpecError(f"{where}: dropout needs 0 <= p < 1 and a non-negative seed")
        return Node(name, op, [a], {"p": prob, "seed": seed}, shape_of(a), "f32")
    if op in UNARY:
        only_attrs()
        if len(pos) != 1:
            raise SpecError(f"{where}: {op} takes one operand")
        a = _operand(g, pos[0], where, False)
        return Node(name, op, [a], {}, shape_of(a), "f32")
    if op in BINARY:
        only_attrs()
        if len(pos) != 2:
            raise SpecError(f"{where}: {op} takes two operands")
        a = _operand(g, pos[0], where, True)
        b = _operand(g, pos[1], where, True)
        if not isinstance(a, str) and not isinstance(b, str):
            raise SpecError(f"{where}: at least one operand must be a tensor")
        if isinstance(a, str) and isinstance(b, str):
            shape = _broadcast(shape_of(a), shape_of(b), where)
        else:
            shape = shape_of(a if isinstance(a, str) else b)
        return Node(name, op, [a, b], {}, shape, "f32")
    if op in ROW_TO_ROW or op in ROW_TO_COL:
        only_attrs()
        if len(pos) != 1:
            raise SpecError(f"{where}: {op} takes one operand")
        a = _operand(g, pos[0], where, False)
        s = shape_of(a)
        if len(s) != 2 or s[1] < (1 if op == "row_softmax" else 2):
            raise SpecError(f"{where}: {op} needs a [R,C] operand with enough columns")
        return Node(name, op, [a], {}, s if op in ROW_TO_ROW else (s[0], 1), "f32")
    if op == "reshape":
        only_attrs("rows", "cols")
        if len(pos) != 1:
            raise SpecError(f"{where}: reshape takes one operand")
        a = _operand(g, pos[0], where, False)
        s = shape_of(a)
        if "rows" not in attrs or "cols" not in attrs:
            raise SpecError(f"{where}: reshape needs rows=R, cols=C")
        rows, cols = _int_attr(attrs, "rows", 0, where), _int_attr(attrs, "cols", 0, where)
        n = 1
        for v in s:
            n *= v
        if rows < 1 or cols < 1 or rows * cols != n:
            raise SpecError(f"{where}: reshape of {s} must keep the number of elements")
        return Node(name, op, [a], {"rows": rows, "cols": cols}, (rows, cols), g.nodes[a].dtype)
    if op in ("row_sort", "row_topk", "row_argsort", "row_topk_indices"):
        only_attrs("k") if op.startswith("row_topk") else only_attrs("descending")
        if len(pos) != 1:
            raise SpecError(f"{where}: {op} takes one operand")
        a = _operand(g, pos[0], where, False)
        s = shape_of(a)
        if len(s) != 2:
            raise SpecError(f"{where}: {op} needs a [R,C] operand")
        if op.startswith("row_topk"):
            k = _int_attr(attrs, "k", 1, where)
            if k < 1 or k > s[1]:
                raise SpecError(f"{where}: {op} needs 1 <= k <= C")
            return Node(name, op, [a], {"k": k}, (s[0], k), "f32")
        return Node(name, op, [a], {"descending": _int_attr(attrs, "descending", 0, where)}, s, "f32")
    if op == "permute":
        only_attrs("axes")
        if len(pos) != 1:
            raise SpecError(f"{where}: permute takes one operand")
        a = _operand(g, pos[0], where, False)
        s = shape_of(a)
        ax = attrs.get("axes", "")
        if not 2 <= len(s) <= 4 or len(ax) != len(s) or sorted(ax) != [str(d) for d in range(len(s))]:
            raise SpecError(f"{where}: permute needs rank 2..4 and axes=<a permutation, one digit per axis>")
        axes = tuple(int(c) for c in ax)
        return Node(name, op, [a], {"axes": axes}, tuple(s[d] for d in axes), g.nodes[a].dtype)
    if op == "transpose":
        only_attrs()
        if len(pos) != 1:
            raise SpecError(f"{where}: transpose takes one operand")
        a = _operand(g, pos[0], where, False)
        s = shape_of(a)
        if len(s) != 2:
            raise SpecError(f"{where}: transpose needs a [R,C] operand")
        return Node(name, op, [a], {}, (s[1], s[0]), "f32")
    if op == "row_layernorm":
        only_attrs("eps")
        if len(pos) != 3:
            raise SpecError(f"{where}: row_layernorm takes (x, gamma, beta)")
        a, ga, be = (_operand(g, p, where, False) for p in pos)
        s = shape_of(a)
        if len(s) != 2 or s[1] < 2:
            raise SpecError(f"{where}: row_layernorm needs a [R,C] operand with C >= 2")
        for p in (ga, be):
            if shape_of(p) not in ((s[1],), (1, s[1])):
                raise SpecError(f"{where}: gamma/beta must have shape [C]")
        try:
            eps = float(attrs.get("eps", "1e-5"))
        except ValueError:
            raise SpecError(f"{where}: eps must be a number") from None
        if not eps >= 0:
            raise SpecError(f"{where}: eps must be non-negative")
        return Node(name, op, [a, ga, be], {"eps": eps}, s, "f32")
    if op == "gemm":
        only_attrs("precision")
        if len(pos) != 2:
            raise SpecError(f"{where}: gemm takes (a, b)")
        a, b = (_operand(g, p, where, False) for p in pos)
        sa, sb = shape_of(a), shape_of(b)
        if len(sa) != 2 or len(sb) != 2 or sa[1] != sb[0]:
            raise SpecError(f"{where}: gemm shapes {sa} x {sb} do not contract")
        if g.nodes[a].dtype != g.nodes[b].dtype:
            raise SpecError(f"{where}: gemm operands must have one dtype")
        return Node(name, op, [a, b], dict(attrs), (sa[0], sb[1]), "f32")
    if op == "conv2d":
        only_attrs("stride", "pad", "dilation", "groups")
        if len(pos) != 2:
            raise SpecError(f"{where}: conv2d takes (x, w)")
        a, b = (_operand(g, p, where, False) for p in pos)
        sa, sb = shape_of(a), shape_of(b)
        stride = _int_attr(attrs, "stride", 1, where)
        pad = _int_attr(attrs, "pad", 0, where)
        dil = _int_attr(attrs, "dilation", 1, where)
        groups = _int_attr(attrs, "groups", 1, where)
        # channels and filters are cut into `groups` equal parts; filter k of a part sees only that part's channels
        if (len(sa) != 4 or len(sb) != 4 or stride < 1 or pad < 0 or dil < 1 or groups < 1 or sa[1] != sb[1] * groups
                or sb[0] % groups != 0):
            raise SpecError(f"{where}: conv2d operands {sa}, {sb} are inconsistent")
        if g.nodes[a].dtype != g.nodes[b].dtype:
            raise SpecError(f"{where}: conv2d operands must have one dtype")
        # a filter of R taps spaced `dil` apart spans dil*(R-1)+1 input rows
        eh, ew = sa[2] + 2 * pad - (dil * (sb[2] - 1) + 1), sa[3] + 2 * pad - (dil * (sb[3] - 1) + 1)
        if eh < 0 or ew < 0:
            raise SpecError(f"{where}: conv2d output is empty")
        ho, wo = eh // stride + 1, ew // stride + 1
        return Node(name, op, [a, b], {"stride": stride, "pad": pad, "dilation": dil, "groups": groups}, (sa[0], sb[0], ho, wo), "f32")
    raise SpecError(f"{where}: unknown operator {op!r}")
