"""Float64 interpreter of an operator DAG (test infrastructure only).

Every node is materialised in float64 and evaluated from the operator's plain
definition, in the order the spec lists the nodes.  There is no fusion, no
tiling and no reordering: what the fused GPU kernels must reproduce is exactly
this composition (fusion changes the schedule, not the mathematics).

Operator classes follow the paper's Table 1: elementwise (add, sub, mul, div,
sqrt, sin, cos, relu, ...), reduction (sum, mean, softmax, ...) and
compute-intensive (matmul, conv).
"""
from __future__ import annotations

import math

import numpy as np
from scipy.special import erf as _erf

from .graph import Graph, parse, UNARY, BINARY


# ---- elementwise (Table 1, "Elementwise") ---------------------------------------------------

def relu(x):
    return np.maximum(x, 0.0)


def sigmoid(x):
    return 1.0 / (1.0 + np.exp(-x))


def gelu_tanh(x):
    # 0.5 x (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3)))
    return 0.5 * x * (1.0 + np.tanh(math.sqrt(2.0 / math.pi) * (x + 0.044715 * x * x * x)))


def gelu_erf(x):
    # 0.5 x (1 + erf(x / sqrt 2))
    return 0.5 * x * (1.0 + _erf(x / math.sqrt(2.0)))


_UNARY_FN = {
    "relu": relu, "gelu_tanh": gelu_tanh, "gelu_erf": gelu_erf, "sigmoid": sigmoid,
    "exp": np.exp, "tanh": np.tanh, "sqrt": np.sqrt, "sin": np.sin, "cos": np.cos,
    "neg": np.negative, "abs": np.abs, "log": np.log, "rsqrt": lambda x: 1.0 / np.sqrt(x), "square": lambda x: x * x,
    "reciprocal": lambda x: 1.0 / x,
}
_BINARY_FN = {
    "add": np.add, "sub": np.subtract, "mul": np.multiply, "div": np.divide,
    "max": np.maximum, "min": np.minimum,
}


def cast_bf16(x):
    """Rounds to bfloat16, nearest even: the value is first taken to float32 (the width every computed
    value has on the device), then its low 16 bits are rounded away."""
    u = np.asarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    r = ((u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))) >> np.uint64(16)) << np.uint64(16)
    y = r.astype(np.uint32).view(np.float32).astype(np.float64)
    return np.where(np.isfinite(x), y, x)


def dropout_keep_mask(shape, seed: int, p: float):
    """Which elements inverted dropout keeps (the paper's first case study, Section 5.3 "Detailed Case Study").

    The generator is counter based: the element at row-major offset ``i`` draws
    ``h = i + seed``, then ``h ^= h >> 17``, ``h ^= h << 31``, ``h ^= h >> 8`` in
    unsigned 64-bit arithmetic, and its uniform variate is ``(h mod 1000) / 1000``.
    The case study elides the comparison; the reading taken here keeps the element
    when the variate is at least ``p``, decided on integers: ``h mod 1000 >= round(1000 p)``.
    """
    n = int(np.prod(shape))
    h = np.arange(n, dtype=np.uint64) + np.uint64(seed)
    h ^= h >> np.uint64(17)
    h ^= h << np.uint64(31)      # numpy wraps modulo 2^64, as the unsigned arithmetic does
    h ^= h >> np.uint64(8)
    return ((h % np.uint64(1000)) >= np.uint64(round(p * 1000.0))).reshape(shape)


def dropout(x, p: float, seed: int):
    """Kept elements are scaled by 1 / (1 - p), dropped ones are zero."""
    return np.where(dropout_keep_mask(x.shape, seed, p), x / (1.0 - p), 0.0)


# ---- row reductions (Table 1, "Reduction") --------------------------------------------------

def row_sum(x):
    return x.sum(axis=1, keepdims=True)


def row_mean(x):
    return x.sum(axis=1, keepdims=True) / x.shape[1]


def row_max(x):
    return x.max(axis=1, keepdims=True)


def reshape(x, rows, cols):
    # element number t of x in row-major order becomes y[t // cols, t % cols]
    flat = np.ascontiguousarray(x).ravel(order="C")
    y = np.empty((rows, cols), dtype=x.dtype)
    for i in range(rows):
        y[i, :] = flat[i * cols:(i + 1) * cols]
    return y


# ---- logic-intensive operators (Table 1): ordering the values of a row ------------------------

def row_sort(x, descending=False):
    # y[i, :] holds the values of x[i, :] in non-decreasing (non-increasing) order
    y = np.sort(x, axis=1, kind="stable")
    return y[:, ::-1].copy() if descending else y


def row_topk(x, k):
    # the k largest values of every row, largest first
    return row_sort(x, descending=True)[:, :k].copy()


def row_argsort(x, descending=False):
    # y[i, j] = column of the j-th value of row i in non-decreasing (non-increasing) order; among equal
    # values the smaller column comes first in both directions (-0 and +0 are equal).  Returned as floats.
    r, c = x.shape
    y = np.empty((r, c), dtype=np.float64)
    for i in range(r):
        cols = sorted(range(c), key=lambda j: ((-x[i, j] if descending else x[i, j]) + 0.0, j))
        y[i, :] = cols
    return y


def row_topk_indices(x, k):
    # columns of the k largest values of every row, largest first, smaller column first among equal values
    return row_argsort(x, descending=True)[:, :k].copy()


# ---- layout transform (Table 1, "LayoutTransform") ------------------------------------------

def transpose(x):
    # y[j, i] = x[i, j]
    r, c = x.shape
    y = np.empty((c, r), dtype=x.dtype)
    for i in range(r):
        y[:, i] = x[i, :]
    return y


def permute(x, axes):
    # y[o] = x[i] with i[axes[d]] = o[d]: output axis d is input axis axes[d]
    y = np.empty(tuple(x.shape[a] for a in axes), dtype=x.dtype)
    for o in np.ndindex(*y.shape):
        i = [0] * x.ndim
        for d, a in enumerate(axes):
            i[a] = o[d]
        y[o] = x[tuple(i)]
    return y


def row_min(x):
    return x.min(axis=1, keepdims=True)


def row_argmax(x):
    # column of the largest element of each row, the first one among equals (Table 1, "argmax"), as a float
    return np.argmax(x, axis=1).reshape(-1, 1).astype(np.float64)


def row_argmin(x):
    return np.argmin(x, axis=1).reshape(-1, 1).astype(np.float64)


def row_softmax(x):
    # y_ij = exp(x_ij - m_i) / sum_j exp(x_ij - m_i), m_i the row maximum
    e = np.exp(x - x.max(axis=1, keepdims=True))
    return e / e.sum(axis=1, keepdims=True)


def row_layernorm(x, gamma, beta, eps):
    # mu_i = mean_j x_ij ; v_i = mean_j (x_ij - mu_i)^2 (biased) ;
    # y_ij = (x_ij - mu_i) / sqrt(v_i + eps) * gamma_j + beta_j
    mu = x.sum(axis=1, keepdims=True) / x.shape[1]
    d = x - mu
    v = (d * d).sum(axis=1, keepdims=True) / x.shape[1]
    return d / np.sqrt(v + eps) * gamma.reshape(1, -1) + beta.reshape(1, -1)


# ---- contractions (Table 1, "ComputeIntensive") ---------------------------------------------

def gemm(a, b):
    # C_ij = sum_k A_ik B_kj for row-major A[M,K], B[K,N]
    return np.matmul(a, b)


def conv2d(x, w, stride, pad, dilation=1, groups=1):
    """Y[n,k,h,w] = sum_{c,r,s} X[n,c,h*stride-pad+r*dilation, w*stride-pad+s*dilation] * Wt[k,c,r,s].

    Cross-correlation over an NCHW input with zeros outside the image, as in
    the paper's convolution case study (input row h - P + kh, column w - P + kw,
    taps outside the image contribute nothing; output index ((n*K+k)*H+h)*W+w).
    For each tap (r, s) the strided window of the zero-padded input is
    contracted over channels with the tap's [K,C] weight slice.

    With ``groups`` = G the C input channels and the K filters are cut into G
    equal consecutive parts, Wt is [K, C/G, R, S], and the filters of part g
    sum over the channels of part g only (G = C: one filter plane per channel,
    the depthwise operator class of the paper's model workloads).
    """
    n, c, h, wd = x.shape
    k, cg, kr, ks = w.shape
    assert c == cg * groups and k % groups == 0
    kg = k // groups
    ho = (h + 2 * pad - dilation * (kr - 1) - 1) // stride + 1
    wo = (wd + 2 * pad - dilation * (ks - 1) - 1) // stride + 1
    xp = np.zeros((n, c, h + 2 * pad, wd + 2 * pad), dtype=x.dtype)
    xp[:, :, pad:pad + h, pad:pad + wd] = x
    y = np.zeros((n, k, ho, wo), dtype=x.dtype)
    for g in range(groups):
        xg = xp[:, g * cg:(g + 1) * cg]
        wg = w[g * kg:(g + 1) * kg]
        for r in range(kr):
            for s in range(ks):
                r0, s0 = r * dilation, s * dilation
                win = xg[:, :, r0:r0 + (ho - 1) * stride + 1:stride, s0:s0 + (wo - 1) * stride + 1:stride]
                y[:, g * kg:(g + 1) * kg] += np.einsum("nchw,kc->nkhw", win, wg[:, :, r, s], optimize=True)
    return y


# ---- interpreter ----------------------------------------------------------------------------

def run_nodes(spec, inputs: dict, dtype=np.float64, gemm_fn=None) -> dict:
    """Evaluate every node; returns name -> array for all nodes (inputs included).

    ``inputs`` maps input names to arrays already widened to float64 (the
    stored float32 / bfloat16 values, exactly).  ``dtype`` is float64 for every
    expected value; float32 is accepted only to study how a graph reacts to
    single-precision evaluation (the sweep's conditioning check), never as a
    reference; ``gemm_fn`` replaces the matrix product in such a study.
    """
    g = spec if isinstance(spec, Graph) else parse(spec)
    val = {}
    for name, node in g.nodes.items():
        if node.op == "input":
            a = np.asarray(inputs[name], dtype=dtype)
            if tuple(a.shape) != tuple(node.shape):
                raise ValueError(f"input {name}: expected shape {node.shape}, got {a.shape}")
            val[name] = a
            continue
        args = [val[a] if isinstance(a, str) else float(a) for a in node.args]
        op = node.op
        if op == "cast_bf16":
            out = cast_bf16(args[0])
        elif op == "dropout":
            out = dropout(args[0], node.attrs["p"], node.attrs["seed"])
        elif op in UNARY:
            out = _UNARY_FN[op](args[0])
        elif op in BINARY:
            out = _BINARY_FN[op](args[0], args[1])
            out = np.broadcast_to(out, node.shape)
        elif op == "reshape":
            out = reshape(args[0], node.attrs["rows"], node.attrs["cols"])
        elif op == "row_sort":
            out = row_sort(args[0], bool(node.attrs["descending"]))
        elif op == "row_topk":
            out = row_topk(args[0], node.attrs["k"])
        elif op == "row_argsort":
            out = row_argsort(args[0], bool(node.attrs["descending"]))
        elif op == "row_topk_indices":
            out = row_topk_indices(args[0], node.attrs["k"])
        elif op == "transpose":
            out = transpose(args[0])
        elif op == "permute":
            out = permute(args[0], node.attrs["axes"])
        elif op == "row_softmax":
            out = row_softmax(args[0])
        elif op == "row_sum":
            out = row_sum(args[0])
        elif op == "row_mean":
            out = row_mean(args[0])
        elif op == "row_max":
            out = row_max(args[0])
        elif op == "row_min":
            out = row_min(args[0])
        elif op == "row_argmax":
            out = row_argmax(args[0])
        elif op == "row_argmin":
            out = row_argmin(args[0])
        elif op == "row_layernorm":
            out = row_layernorm(args[0], args[1], args[2], node.attrs["eps"])
        elif op == "gemm":
            out = (gemm_fn or gemm)(args[0], args[1])
        elif op == "conv2d":
            out = conv2d(args[0], args[1], node.attrs["stride"], node.attrs["pad"], node.attrs["dilation"], node.attrs["groups"])
        else:  # pragma: no cover - parse() rejects unknown operators
            raise ValueError(op)
        assert tuple(out.shape) == tuple(node.shape), (name, out.shape, node.shape)
        val[name] = np.asarray(out, dtype=dtype)
    return val


def run(spec, inputs: dict) -> dict:
    """Evaluate the graph; returns output name -> float64 array (no output rounding)."""
    g = spec if isinstance(spec, Graph) else parse(spec)
    val = run_nodes(g, inputs)
    return {name: val[name] for name, _ in g.outputs}
