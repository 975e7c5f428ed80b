"""First-order forward error bound of a float32 evaluation of an operator DAG (test infrastructure).

The fp32 parity criterion is "relative error at most 1e-5".  That is well defined wherever nothing
cancels.  Where a subtraction-like step cancels (a row sum of mixed signs, x - mean in a layer
normalisation, an addition of opposite signs), NO float32 evaluation can deliver a relative error of
the result: the best it can do is bounded by the rounding of the larger intermediate values.  This
module computes that bound from the oracle's own float64 node values, by the textbook running
error analysis: every operator contributes its own rounding, `c_op * u * |value|` with u = 2^-24,
and passes on the errors of its operands multiplied by the magnitude of its partial derivatives.
Inputs are exact (they are stored in the dtype the device reads).  A sum of n terms is modelled as
a balanced tree: (ceil(log2 n) + 1) * u * sum |x_j| — for a row sum this is the condition number of
the sum, sum_j |x_ij|, times a small multiple of u.

`bound(spec, inputs)` returns name -> array E with  |fp32 result - exact| <~ E  to first order.
The tests grade  |g - r| <= max(1e-5 |r|, SAFETY * E):  strict relative 1e-5 wherever a float32
evaluation can deliver it, and a small multiple of what float32 can resolve elsewhere.
"""
from __future__ import annotations

import math

import numpy as np

import oracle
from oracle import interp

U = 2.0 ** -24          # unit round-off of float32
SAFETY = 2.0            # first-order bounds ignore second-order terms and differences in evaluation order

# own rounding of one operator, in units of u relative to |result|
C_EXACT = 0.0           # selections and sign changes: relu, neg, abs, max, min, data movement
C_ARITH = 1.0           # one correctly rounded operation: add, sub, mul, square
C_DIV = 2.0             # division, reciprocal, roots (reciprocal estimates refined once)
C_FUNC = 4.0            # exponential-family functions (2-ulp unit plus the rounding of a scaled argument)
C_GEMM = 16.0           # fp32 matrix product from three TF32 products: the dropped tail*tail term is 2^-22 |a||b|


def _tree(n):
    return (math.ceil(math.log2(max(n, 2))) + 1) * U


def _sum_rows(x, ex):
    """Bound for s_i = sum_j x_ij: operand errors add, and the tree's roundings scale with sum |x|."""
    return ex.sum(axis=1, keepdims=True) + _tree(x.shape[1]) * np.abs(x).sum(axis=1, keepdims=True)


def _row_extreme(x, ex, largest):
    """max (min) over a row when each element is uncertain by ex: any element whose interval reaches the
    extreme element's interval may win; the result then differs by at most that element's uncertainty."""
    y = x if largest else -x
    top = y.max(axis=1, keepdims=True)
    e_top = np.take_along_axis(ex, y.argmax(axis=1)[:, None], axis=1)
    cand = (y + ex) >= (top - e_top)
    return np.where(cand, ex, 0.0).max(axis=1, keepdims=True)


def _unary(op, x, y, ex):
    ax = np.abs(x)
    if op in ("relu", "neg", "abs"):
        return ex
    if op == "square":
        return 2 * ax * ex + C_ARITH * U * y
    if op == "exp":
        return y * ex + C_FUNC * U * y
    if op == "sigmoid":
        return y * (1 - y) * ex + C_FUNC * U * y
    if op == "tanh":
        return (1 - y * y) * ex + C_FUNC * U * np.abs(y)
    if op == "sqrt":
        return np.where(y > 0, 0.5 / np.maximum(y, 1e-300), 0.0) * ex + C_DIV * U * y
    if op == "rsqrt":
        return 0.5 * y / np.maximum(ax, 1e-300) * ex + C_DIV * U * y
    if op == "reciprocal":
        return y * y * ex + C_DIV * U * np.abs(y)
    if op == "log":
        return ex / np.maximum(ax, 1e-300) + C_FUNC * U * np.abs(y)
    if op == "sin":
        return np.abs(np.cos(x)) * ex + C_FUNC * U * np.abs(y)
    if op == "cos":
        return np.abs(np.sin(x)) * ex + C_FUNC * U * np.abs(y)
    if op in ("gelu_tanh", "gelu_erf"):
        # 0.5 x (1 + t) with t = tanh(.) or erf(.): for negative x the factor 1 + t cancels, so the own
        # rounding of the definition evaluated in float32 is relative to 0.5 |x| |t| as well as to |y|.
        # The float64 oracle evaluates the same formula: its own rounding (2^-52 |x|) is the floor below
        # which no comparison means anything.
        if op == "gelu_tanh":
            t = np.tanh(math.sqrt(2 / math.pi) * (x + 0.044715 * x ** 3))
            dt = (1 - t * t) * math.sqrt(2 / math.pi) * (1 + 3 * 0.044715 * x * x)
        else:
            from scipy.special import erf
            t = erf(x / math.sqrt(2))
            dt = math.sqrt(2 / math.pi) * np.exp(-0.5 * x * x)
        own = C_FUNC * U * (np.abs(y) + 0.5 * ax * np.abs(t))
        slope = np.abs(0.5 * (1 + t) + 0.5 * x * dt)
        return slope * ex + own + 2.0 ** -52 * ax
    raise ValueError(op)


def _binary(op, a, b, y, ea, eb):
    if op in ("add", "sub"):
        return ea + eb + C_ARITH * U * np.abs(y)
    if op == "mul":
        return np.abs(b) * ea + np.abs(a) * eb + C_ARITH * U * np.abs(y)
    if op == "div":
        ib = 1.0 / np.maximum(np.abs(b), 1e-300)
        return ea * ib + np.abs(y) * eb * ib + C_DIV * U * np.abs(y)
    if op in ("max", "min"):
        return np.maximum(ea, eb)
    raise ValueError(op)


def _softmax(x, y, ex):
    # the shift by the row maximum m changes nothing mathematically; what reaches the exponential is the
    # rounding of the difference x - m and of its scaling to base 2, or, when the shift is folded into one
    # multiply-add x * log2(e) - m * log2(e), the rounding of the second product (done only for |m| < 16)
    m = x.max(axis=1, keepdims=True)
    ed = ex + 2 * U * (np.abs(x - m) + np.minimum(np.abs(m), 16.0))
    e = np.exp(x - m)
    ee = e * ed + C_FUNC * U * e
    s = e.sum(axis=1, keepdims=True)
    es = _sum_rows(e, ee)
    return ee / s + y * es / s + C_DIV * U * y


def _layernorm(x, gamma, beta, eps, y, ex, eg, eb):
    c = x.shape[1]
    mu = x.sum(axis=1, keepdims=True) / c
    emu = _sum_rows(x, ex) / c + U * np.abs(mu)
    d = x - mu
    ed = ex + emu + U * np.abs(d)
    v = (d * d).sum(axis=1, keepdims=True) / c
    ev = _sum_rows(d * d, 2 * np.abs(d) * ed + U * d * d) / c + U * v
    r = 1.0 / np.sqrt(v + eps)
    er = 0.5 * r ** 3 * ev + C_DIV * U * r
    g, b = gamma.reshape(1, -1), beta.reshape(1, -1)
    n = d * r
    en = ed * r + np.abs(d) * er + U * np.abs(n)
    return en * np.abs(g) + np.abs(n) * eg.reshape(1, -1) + eb.reshape(1, -1) + U * (np.abs(n * g) + np.abs(y))


def bound(spec, inputs, values=None):
    """name -> first-order bound on |float32 evaluation - exact value| for every node of the graph."""
    g = spec if isinstance(spec, oracle.Graph) else oracle.parse(spec)
    val = values if values is not None else oracle.run_nodes(g, inputs)
    err = {}
    for name, node in g.nodes.items():
        y = val[name]
        if node.op == "input":
            err[name] = np.zeros_like(y)
            continue
        av = [val[a] if isinstance(a, str) else np.float64(a) for a in node.args]
        ae = [err[a] if isinstance(a, str) else np.float64(0.0) for a in node.args]
        op = node.op
        if op == "cast_bf16":
            # an uncertain value may round to the neighbouring bfloat16
            e = np.where(ae[0] > 0, ae[0] + 2.0 ** -8 * np.abs(y), 0.0)
        elif op == "dropout":
            e = np.where(y != 0, ae[0] / (1.0 - node.attrs["p"]), 0.0) + C_ARITH * U * np.abs(y)
        elif op in interp.UNARY:
            e = _unary(op, av[0], y, ae[0])
        elif op in interp.BINARY:
            e = np.broadcast_to(_binary(op, av[0], av[1], y, ae[0], ae[1]), y.shape)
        elif op == "reshape":
            e = ae[0].reshape(y.shape)
        elif op == "transpose":
            e = ae[0].T
        elif op == "permute":
            e = np.transpose(ae[0], node.attrs["axes"])
        elif op in ("row_sort", "row_topk"):
            # values are moved, not changed; an uncertain key may land in a neighbouring slot
            e = np.broadcast_to(ae[0].max(axis=1, keepdims=True), y.shape)
        elif op == "row_softmax":
            e = _softmax(av[0], y, ae[0])
        elif op == "row_sum":
            e = _sum_rows(av[0], ae[0])
        elif op == "row_mean":
            e = _sum_rows(av[0], ae[0]) / av[0].shape[1] + U * np.abs(y)
        elif op in ("row_max", "row_min"):
            e = _row_extreme(av[0], ae[0], op == "row_max")
        elif op in ("row_argmax", "row_argmin", "row_argsort", "row_topk_indices"):
            e = np.zeros_like(y)      # an index: compared exactly (tests give these operators exact operands)
        elif op == "row_layernorm":
            e = _layernorm(av[0], av[1], av[2], node.attrs["eps"], y, ae[0], ae[1], ae[2])
        elif op == "gemm":
            a, b = np.abs(av[0]), np.abs(av[1])
            e = ae[0] @ b + a @ ae[1] + (C_GEMM * U + _tree(a.shape[1])) * (a @ b)
        elif op == "conv2d":
            at = node.attrs
            conv = lambda p, q: interp.conv2d(p, q, at["stride"], at["pad"], at["dilation"], at["groups"])
            a, b = np.abs(av[0]), np.abs(av[1])
            terms = b.shape[1] * b.shape[2] * b.shape[3]
            e = conv(ae[0] + 0 * a, b) + conv(a, ae[1] + 0 * b) + (C_ARITH * U + _tree(terms)) * conv(a, b)
        else:  # pragma: no cover
            raise ValueError(op)
        err[name] = np.asarray(e, dtype=np.float64)
    return err
